// Microbenchmark: the query gather of the key-block-major tile kernels through the copy engine.
//
// A tile of those kernels is 128 query rows = 32 tokens x G heads of one KV group; the G rows of a token are
// adjacent in q [N, Hq, d], so one token's piece of a 64-element slab is a plain 2-D TMA box of {64 elements,
// G rows} (G = 4: 512 bytes) that lands in the 128-byte-swizzled layout the UMMA descriptors read.  A tile is
// then 64 such loads (32 tokens x 2 slabs of d = 128) instead of 2048 16-byte cp.async copies.  This program
// measures the rate of those small boxes from random tokens of a 16384-token window, one CTA per SM, four tiles
// in flight, with the tile's 64 loads dealt out over 1, 2, 4 or 8 issuing warps, beside the same bytes moved as
// boxes of {64, 128} from consecutive rows (what a dense tile load does; two loads per tile, so that line mostly
// shows what this loop's own per-tile synchronisation allows).  tile::gather4 moves the same unit of work per
// instruction (four rows of 128 bytes), so these rates stand for it as well.
// Own memory only, no multicast.  Every wait is bounded; a wait that runs out sets a flag and the kernel returns.
// Build: nvcc -gencode arch=compute_100a,code=sm_100a -O3 tma_rows.cu -o tma_rows
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <cuda.h>
#include <cuda_runtime.h>

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("cuda error %s at line %d\n", cudaGetErrorString(e_), __LINE__); return 1; } } while (0)

constexpr int kTileBytes = 32768;     // 128 rows x 256 bytes
constexpr int kSlabBytes = 16384;     // 128 rows x 128 bytes (one 64-element slab)
constexpr int kDepth = 4;             // tiles in flight per SM

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  for (;;) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    if (ok) return true;
    if (clock64() - t0 > 2000000000LL) return false;          // about a second
  }
}

// ROWS = 4: the 64 loads of a tile (token, slab) go round the lanes of the nw warps;  ROWS = 128: lane 0 of warp w
// loads whole slabs of 128 consecutive rows starting at token tok[0]'s first row.
template <int ROWS>
__global__ void tma_rows_kernel(const __grid_constant__ CUtensorMap tm, const int* __restrict__ tok, int tiles, int nw,
                                int* fail) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ __align__(8) uint64_t full[kDepth];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int* my = tok + (long long)blockIdx.x * tiles * 32;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kDepth; ++i)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&full[i])), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  for (int t = 0; t < tiles; ++t) {
    const int s = t % kDepth;
    // the stage's previous tile must have landed before it is overwritten (all warps wait: they all write it)
    if (t >= kDepth && !wait_bounded(&full[s], (uint32_t)((t / kDepth - 1) & 1))) { atomicExch(fail, 1); return; }
    __syncthreads();                                  // every warp has seen the stage free
    if (threadIdx.x == 0)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&full[s])), "r"(kTileBytes) : "memory");
    __syncthreads();                                  // expect_tx is posted before any byte can complete
    uint8_t* dst = smem + s * kTileBytes;
    if (ROWS == 4) {
      // the tile's 64 loads (32 tokens x 2 slabs) are dealt out over the nw * 32 lanes
      const int per = nw >= 2 ? 64 / nw : 32;        // loads per warp and round
      for (int i = warp * per + lane; lane < per && i < 64; i += nw * per) {
        const int tk = i & 31, sl = i >> 5;
        const int row = my[t * 32 + tk] * 32;        // first of the token's 4 adjacent rows (32 heads per token)
        asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                     ::"r"(smem_u32(dst + sl * kSlabBytes + tk * 512)), "l"(&tm), "r"(smem_u32(&full[s])), "r"(sl * 64), "r"(row)
                     : "memory");
      }
    } else if (lane == 0) {
      const int row = my[t * 32] * 32;
      for (int sl = warp; sl < 2; sl += nw)
        asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                     ::"r"(smem_u32(dst + sl * kSlabBytes)), "l"(&tm), "r"(smem_u32(&full[s])), "r"(sl * 64), "r"(row)
                     : "memory");
    }
  }
  // drain: the last kDepth tiles
  for (int t = (tiles > kDepth ? tiles - kDepth : 0); t < tiles; ++t)
    if (!wait_bounded(&full[t % kDepth], (uint32_t)((t / kDepth) & 1))) { atomicExch(fail, 1); return; }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <int ROWS>
static int run(const char* name, EncodeTiledFn enc, void* q, long long rows, const int* tok, int tiles, int nw, int* fail,
               int sms, double clk_hz) {
  CUtensorMap tm;
  const cuuint64_t gdim[2] = {128, (cuuint64_t)rows}, gstride[1] = {256};
  const cuuint32_t box[2] = {64, ROWS}, estr[2] = {1, 1};
  if (enc(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, q, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
    printf("tensor map encode failed\n");
    return 1;
  }
  cudaEvent_t a, b;
  CK(cudaEventCreate(&a)); CK(cudaEventCreate(&b));
  CK(cudaFuncSetAttribute(tma_rows_kernel<ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDepth * kTileBytes));
  tma_rows_kernel<ROWS><<<sms, nw * 32, kDepth * kTileBytes>>>(tm, tok, tiles, nw, fail);
  CK(cudaDeviceSynchronize());
  CK(cudaEventRecord(a));
  tma_rows_kernel<ROWS><<<sms, nw * 32, kDepth * kTileBytes>>>(tm, tok, tiles, nw, fail);
  CK(cudaEventRecord(b));
  CK(cudaDeviceSynchronize());
  int f = 0;
  CK(cudaMemcpy(&f, fail, sizeof(f), cudaMemcpyDeviceToHost));
  if (f) { printf("%s: a wait ran out\n", name); return 1; }
  float ms = 0.f;
  CK(cudaEventElapsedTime(&ms, a, b));
  const double bytes = (double)sms * tiles * kTileBytes;
  printf("%-44s %8.3f ms %6.2f TB/s %6.1f B/clk/SM\n", name, ms, bytes / ms * 1e-9, bytes / sms / (ms * 1e-3 * clk_hz));
  return 0;
}

int main() {
  int dev = 0, sms = 0, khz = 0;
  CK(cudaGetDevice(&dev));
  CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  CK(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
  const double clk = khz * 1e3;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (qres != cudaDriverEntryPointSuccess || fn == nullptr) { printf("no tensor map encoder\n"); return 1; }
  EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(fn);
  const int tiles = 512, window = 16384;
  const long long ntok = 131072;
  uint8_t* q;
  CK(cudaMalloc(&q, ntok * 8192));                    // q of 32 heads x 128 x bf16 per token: 1.07 GB
  CK(cudaMemset(q, 1, ntok * 8192));
  std::vector<int> h((size_t)sms * tiles * 32);
  srand(1);
  for (int c = 0; c < sms; ++c)
    for (int t = 0; t < tiles; ++t)
      for (int i = 0; i < 32; ++i) h[((size_t)c * tiles + t) * 32 + i] = (t * 8 / tiles) * window + rand() % (window - 4);
  int *tok, *fail;
  CK(cudaMalloc(&tok, h.size() * sizeof(int)));
  CK(cudaMemcpy(tok, h.data(), h.size() * sizeof(int), cudaMemcpyHostToDevice));
  CK(cudaMalloc(&fail, sizeof(int)));
  CK(cudaMemset(fail, 0, sizeof(int)));
  printf("SMs %d, SM clock %.0f MHz (bytes per clock use this clock)\n", sms, clk * 1e-6);
  if (run<4>("TMA boxes of 4 rows x 128 B, 1 warp", enc, q, ntok * 32, tok, tiles, 1, fail, sms, clk)) return 1;
  if (run<4>("TMA boxes of 4 rows x 128 B, 2 warps", enc, q, ntok * 32, tok, tiles, 2, fail, sms, clk)) return 1;
  if (run<4>("TMA boxes of 4 rows x 128 B, 4 warps (16 lanes)", enc, q, ntok * 32, tok, tiles, 4, fail, sms, clk)) return 1;
  if (run<4>("TMA boxes of 4 rows x 128 B, 8 warps (8 lanes)", enc, q, ntok * 32, tok, tiles, 8, fail, sms, clk)) return 1;
  if (run<128>("TMA boxes of 128 rows x 128 B", enc, q, ntok * 32, tok, tiles, 2, fail, sms, clk)) return 1;
  return 0;
}
