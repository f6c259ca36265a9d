// Mean-pooled key pyramid (Eq. "mean pyramid", Sec. 3.2).
//
// Level 1 is one streaming pass over k (HBM-bound: N*Hkv*d elements read once); the levels above
// it together hold about M_1/(g-1) nodes per (b, h) and are pooled by one more launch in which a
// CTA owns one (b, h, 16-byte column slice) and walks the levels bottom-up, so no level needs a
// grid-wide barrier: every node it reads was written by the same CTA.
#include "pisa_common.cuh"
#include "tc_utils.cuh"
#include "tma_map.cuh"

namespace pisa {

// Level 1 as a TMA pipeline: one persistent CTA per SM walks (b, leaf, h) units; a unit's C x d slab of
// keys (rows d*es bytes long, one token apart) is one 4-D tile load (this GPU's memory, no multicast)
// into a ring of shared-memory stages, so that several slabs per SM are in flight at all times; eight
// consumer warps take column sums from shared memory in a fixed order (fp32) while the next slabs land.
constexpr int kPyrConsumers = 256;
constexpr int kPyrThreads = kPyrConsumers + 32;

template <typename T>
__global__ void __launch_bounds__(kPyrThreads, 1)
pyramid_level1_tma_kernel(Geometry geo, const __grid_constant__ CUtensorMap tm, T* __restrict__ pyr, int n_units,
                          int stages, int stage_bytes, int32_t* status) {
  extern __shared__ __align__(128) uint8_t smem_pyr[];
  __shared__ uint64_t full[8], empty[8];
  __shared__ float red[2][16][128];                 // [parity][row group][column]
  __shared__ volatile int s_fail;
  uint8_t* slabs = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_pyr) + 127) & ~(uintptr_t)127);
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { tc::mbar_init(&full[i], 1); tc::mbar_init(&empty[i], kPyrConsumers / 32); }
    s_fail = 0;
    tc::mbar_fence_init();
  }
  __syncthreads();
  const int d = geo.d, C = geo.C;
  if (warp == kPyrConsumers / 32) {
    // ------------------------------------------------ producer: one thread issues the tile loads
    if ((tid & 31) == 0) {
      tc::tma_prefetch_desc(&tm);
      int i = 0;
      for (int u = blockIdx.x; u < n_units && !s_fail; u += gridDim.x, ++i) {
        const int s = i % stages;
        if (i >= stages && !tc::mbar_wait_bounded(&empty[s], (uint32_t)((i / stages - 1) & 1))) { s_fail = 1; break; }
        const int h = u % geo.Hkv, leaf = (u / geo.Hkv) % geo.M[1], b = u / (geo.Hkv * geo.M[1]);
        tc::mbar_arrive_expect_tx(&full[s], (uint32_t)stage_bytes);
        tc::tma_load_4d(tc::smem_u32(slabs + (size_t)s * stage_bytes), &tm, &full[s], 0, h, leaf * C, b);
      }
    }
  } else {
    // ------------------------------------------------ consumers: column sums in a fixed order
    constexpr int EPW = 4 / (int)sizeof(T);                 // elements per 32-bit word
    const int Wd = d / EPW;                                 // words per row (a power of two, 16..128)
    const int w = tid % Wd, rg = tid / Wd, RG = kPyrConsumers / Wd;
    int i = 0;
    for (int u = blockIdx.x; u < n_units; u += gridDim.x, ++i) {
      const int s = i % stages;
      // a wait that gives up is agreed on at the barrier below, so that all consumers leave together
      const bool ok = !s_fail && tc::mbar_wait_bounded(&full[s], (uint32_t)((i / stages) & 1));
      if (!ok) s_fail = 1;
      const uint32_t* slab = reinterpret_cast<const uint32_t*>(slabs + (size_t)s * stage_bytes);
      float a0 = 0.f, a1 = 0.f;
#pragma unroll 8
      for (int r = rg; ok && r < C; r += RG) {
        const uint32_t x = slab[r * Wd + w];
        if (EPW == 2) { a0 += __uint_as_float(x << 16); a1 += __uint_as_float(x & 0xFFFF0000u); }
        else a0 += __uint_as_float(x);
      }
      __syncwarp();
      if ((tid & 31) == 0) tc::mbar_arrive(&empty[s]);       // this warp has read its share of the slab
      float* rr = red[i & 1][rg];
      if (EPW == 2) { rr[2 * w] = a0; rr[2 * w + 1] = a1; } else rr[w] = a0;
      asm volatile("bar.sync 1, %0;" ::"n"(kPyrConsumers) : "memory");
      if (s_fail) break;
      if (tid < d) {
        float sum = 0.f;
        for (int g2 = 0; g2 < RG; ++g2) sum += red[i & 1][g2][tid];
        const int h = u % geo.Hkv, leaf = (u / geo.Hkv) % geo.M[1], b = u / (geo.Hkv * geo.M[1]);
        const int cnt = min(C, geo.N - leaf * C);
        pyr[geo.level_off[1] + (((long long)b * geo.Hkv + h) * geo.M[1] + leaf) * d + tid] =
            Elem<T>::from_float(sum / (float)cnt);
      }
    }
  }
  __syncthreads();
  if (s_fail && tid == 0 && status != nullptr) atomicExch(status, (int)PISA_ERR_TIMEOUT);
}

// One CTA per (leaf block, h, b).  Thread (cx, ry): 16-byte column chunk cx, rows ry, ry+RY, ...
template <typename T, int RY>
__global__ void __launch_bounds__(256) pyramid_level1_kernel(Geometry geo, const T* __restrict__ k,
                                                             T* __restrict__ pyr) {
  constexpr int V = Elem<T>::kVec;
  extern __shared__ float red[];             // [RY][d]
  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int chunks = geo.d / V;
  const int cx = threadIdx.x % chunks, ry = threadIdx.x / chunks;
  const int lo = i * geo.C;
  const int hi = min(lo + geo.C, geo.N);
  float acc[V];
#pragma unroll
  for (int e = 0; e < V; ++e) acc[e] = 0.f;
  if (ry < RY) {
    const T* base = k + (long long)b * geo.ks[0] + (long long)h * geo.ks[2] + cx * V;
    for (int r = lo + ry; r < hi; r += RY) {
      float x[V];
      Elem<T>::load_chunk(base + (long long)r * geo.ks[1], x);
#pragma unroll
      for (int e = 0; e < V; ++e) acc[e] += x[e];
    }
#pragma unroll
    for (int e = 0; e < V; ++e) red[ry * geo.d + cx * V + e] = acc[e];
  }
  __syncthreads();
  // fixed-order reduction over the RY row groups: thread t sums column t
  for (int col = threadIdx.x; col < geo.d; col += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < RY; ++r) s += red[r * geo.d + col];
    const float mean = s / (float)(hi - lo);
    T* dst = pyr + geo.level_off[1] + (((long long)b * geo.Hkv + h) * geo.M[1] + i) * geo.d + col;
    *dst = Elem<T>::from_float(mean);
  }
}

// One CTA per (16-byte column chunk, h, b); loops l = 2..L.
template <typename T>
__global__ void __launch_bounds__(256) pyramid_upper_kernel(Geometry geo, T* __restrict__ pyr) {
  constexpr int V = Elem<T>::kVec;
  const int cx = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  for (int l = 2; l <= geo.L; ++l) {
    const T* below = pyr + geo.level_off[l - 1] + ((long long)b * geo.Hkv + h) * geo.M[l - 1] * geo.d + cx * V;
    T* cur = pyr + geo.level_off[l] + ((long long)b * geo.Hkv + h) * geo.M[l] * geo.d + cx * V;
    for (int i = threadIdx.x; i < geo.M[l]; i += blockDim.x) {
      const int lo = i * geo.g, hi = min(lo + geo.g, geo.M[l - 1]);
      float acc[V];
#pragma unroll
      for (int e = 0; e < V; ++e) acc[e] = 0.f;
      for (int r = lo; r < hi; ++r) {
        float x[V];
        Elem<T>::load_chunk(below + (long long)r * geo.d, x);
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] += x[e];
      }
      const float inv = 1.f / (float)(hi - lo);
#pragma unroll
      for (int e = 0; e < V; ++e) cur[(long long)i * geo.d + e] = Elem<T>::from_float(acc[e] * inv);
    }
    __syncthreads();   // level l is complete for this column slice before level l+1 reads it
  }
}

// the TMA pipeline applies when a slab is one tile (C <= 256 rows) that leaves room for two stages,
// and the row words split evenly over the consumers
template <typename T>
static bool level1_tma(const Geometry& g, const T* k, T* pyr, int32_t* status, cudaStream_t s, int* st_out) {
  const int es = (int)sizeof(T);
  const int Wd = g.d * es / 4;
  const size_t stage_bytes = (size_t)g.C * g.d * es;
  if (g.C > 256 || g.d > 128 || Wd < 16 || Wd > 128 || (Wd & (Wd - 1)) || (kPyrConsumers / Wd) > 16) return false;
  if (stage_bytes % 128 != 0 || 2 * stage_bytes > 192 * 1024) return false;
  if ((long long)g.B * g.Hkv * g.M[1] > 0x7fffffffLL) return false;
  int stages = (int)((192 * 1024) / stage_bytes);
  if (stages > 8) stages = 8;
  CUtensorMap tm;
  const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.Hkv, (uint64_t)g.N, (uint64_t)g.B};
  const uint64_t strides[4] = {(uint64_t)es, (uint64_t)g.ks[2] * es, (uint64_t)g.ks[1] * es, (uint64_t)g.ks[0] * es};
  const uint32_t box[4] = {(uint32_t)g.d, 1u, (uint32_t)g.C, 1u};
  if (!tma::make_map(&tm, es, 4, k, dims, strides, box, false)) return false;
  const size_t smem = (size_t)stages * stage_bytes + 128;
  if (cudaFuncSetAttribute(pyramid_level1_tma_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  const int n_units = g.B * g.Hkv * g.M[1];
  const int grid = n_units < num_sms() ? n_units : num_sms();
  pyramid_level1_tma_kernel<T><<<grid, kPyrThreads, smem, s>>>(g, tm, pyr, n_units, stages, (int)stage_bytes, status);
  *st_out = check_launch("pyramid_level1_tma");
  return true;
}

template <typename T>
static int launch_pyramid_t(const Geometry& g, const T* k, T* pyr, int32_t* status, cudaStream_t s) {
  constexpr int V = Elem<T>::kVec;
  constexpr int RY = 8;
  const int chunks = g.d / V;
  int threads = chunks * RY;
  if (threads > 256) return PISA_ERR_UNSUPPORTED;
  if (threads < 32) threads = 32;
  int st = PISA_OK;
  if (!level1_tma<T>(g, k, pyr, status, s, &st)) {
    dim3 grid1(g.M[1], g.Hkv, g.B);
    pyramid_level1_kernel<T, RY><<<grid1, threads, RY * g.d * sizeof(float), s>>>(g, k, pyr);
    st = check_launch("pyramid_level1");
  }
  if (st != PISA_OK) return st;
  if (g.L >= 2) {
    dim3 grid2(chunks, g.Hkv, g.B);
    pyramid_upper_kernel<T><<<grid2, 256, 0, s>>>(g, pyr);
    st = check_launch("pyramid_upper");
  }
  return st;
}

int launch_pyramid(const Geometry& g, int dtype, const void* k, void* pyramid, int32_t* status, cudaStream_t s) {
  if (dtype == PISA_BF16)
    return launch_pyramid_t<__nv_bfloat16>(g, (const __nv_bfloat16*)k, (__nv_bfloat16*)pyramid, status, s);
  return launch_pyramid_t<float>(g, (const float*)k, (float*)pyramid, status, s);
}

}  // namespace pisa
