// Mean-pooled key pyramid (Eq. "mean pyramid", Sec. 3.2).
//
// Level 1 is one streaming pass over k (HBM-bound: N*Hkv*d elements read once).  A CTA owns a subtree
// of g^s consecutive leaves of one (b, h): it pools their keys (every thread keeps eight 16-byte loads
// in flight), keeps the rounded summaries in shared memory and pools the s levels above them there, so
// that the levels holding most of the upper nodes cost no second pass.  The few levels above the
// subtrees are pooled by one more small launch in which a CTA owns one (b, h, 16-byte column slice)
// and walks the levels bottom-up (no grid-wide barrier: every node it reads was written by itself
// or by the first launch).  Tile loads by the TMA engine were measured for the level-1 slabs (one
// 4-D tile of C rows x d*2 bytes per leaf, four 32 KB stages per SM) and were slower than plain
// 16-byte loads: rows of 256 bytes cost the engine a request each.
#include "pisa_common.cuh"

namespace pisa {

// One CTA per (subtree of `span` = g^s leaves, h, b): level 1 from the raw keys, levels 2 .. 1+s from the
// stored (rounded) summaries below them, as the definition pools them.
constexpr int kSubMaxLeaves = 8;
constexpr int kSubRowGroups = 16;
template <typename T>
__global__ void __launch_bounds__(256) pyramid_subtree_kernel(Geometry geo, const T* __restrict__ k,
                                                              T* __restrict__ pyr, int s_levels, int span) {
  constexpr int V = Elem<T>::kVec;
  __shared__ float red[kSubRowGroups][128];
  __shared__ float node[2][kSubMaxLeaves][128];      // stored values of the level being pooled / produced
  const int sub = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int d = geo.d, chunks = d / V;
  const int cx = threadIdx.x % chunks, ry = threadIdx.x / chunks;
  const int RY = min(kSubRowGroups, (int)blockDim.x / chunks);
  const T* base = k + (long long)b * geo.ks[0] + (long long)h * geo.ks[2] + cx * V;
  for (int j = 0; j < span; ++j) {
    const int leaf = sub * span + j;
    if (leaf >= geo.M[1]) break;
    const int lo = leaf * geo.C, hi = min(lo + geo.C, geo.N);
    float acc[V];
#pragma unroll
    for (int e = 0; e < V; ++e) acc[e] = 0.f;
    if (ry < RY) {
      int r = lo + ry;
      for (; r + 7 * RY < hi; r += 8 * RY) {          // eight independent loads in flight per thread
        float x[8][V];
#pragma unroll
        for (int u = 0; u < 8; ++u) Elem<T>::load_chunk(base + (long long)(r + u * RY) * geo.ks[1], x[u]);
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
          for (int e = 0; e < V; ++e) acc[e] += x[u][e];
      }
      for (; r < hi; r += RY) {
        float x[V];
        Elem<T>::load_chunk(base + (long long)r * geo.ks[1], x);
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] += x[e];
      }
#pragma unroll
      for (int e = 0; e < V; ++e) red[ry][cx * V + e] = acc[e];
    }
    __syncthreads();
    for (int col = threadIdx.x; col < d; col += blockDim.x) {       // fixed-order reduction over the row groups
      float sum = 0.f;
      for (int r = 0; r < RY; ++r) sum += red[r][col];
      const T st = Elem<T>::from_float(sum / (float)(hi - lo));
      pyr[geo.level_off[1] + (((long long)b * geo.Hkv + h) * geo.M[1] + leaf) * d + col] = st;
      node[0][j][col] = Elem<T>::to_float(st);
    }
    __syncthreads();
  }
  // levels 2 .. 1 + s_levels inside the subtree
  int width = span;                                   // nodes of the level below inside this subtree
  for (int t = 1; t <= s_levels; ++t) {
    const int l = 1 + t;
    const int below_first = sub * width;              // global index of the subtree's first node one level down
    width /= geo.g;
    const int first = sub * width;
    const float (*src)[128] = node[(t - 1) & 1];
    float (*dst)[128] = node[t & 1];
    for (int e = threadIdx.x; e < width * d; e += blockDim.x) {
      const int i = e / d, col = e % d;
      if (first + i >= geo.M[l]) continue;
      const int c_lo = (first + i) * geo.g, c_hi = min(c_lo + geo.g, geo.M[l - 1]);
      float sum = 0.f;
      for (int r = c_lo; r < c_hi; ++r) sum += src[r - below_first][col];
      const T st = Elem<T>::from_float(sum * (1.f / (float)(c_hi - c_lo)));
      pyr[geo.level_off[l] + (((long long)b * geo.Hkv + h) * geo.M[l] + first + i) * d + col] = st;
      dst[i][col] = Elem<T>::to_float(st);
    }
    __syncthreads();
  }
}

// One CTA per (16-byte column chunk, h, b); loops l = first_level..L.
template <typename T>
__global__ void __launch_bounds__(256) pyramid_upper_kernel(Geometry geo, T* __restrict__ pyr, int first_level) {
  constexpr int V = Elem<T>::kVec;
  const int cx = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  for (int l = first_level; l <= geo.L; ++l) {
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

template <typename T>
static int launch_pyramid_t(const Geometry& g, const T* k, T* pyr, cudaStream_t s) {
  constexpr int V = Elem<T>::kVec;
  const int chunks = g.d / V;
  if (g.d > 128 || chunks * 8 > 256) return PISA_ERR_UNSUPPORTED;
  int threads = chunks * kSubRowGroups;
  if (threads > 256) threads = 256;
  if (threads < 32) threads = 32;
  // subtree depth: the most levels with g^s <= kSubMaxLeaves leaves per CTA that still leave a few CTAs per SM
  int s_levels = 0, span = 1;
  while (span * g.g <= kSubMaxLeaves && 1 + s_levels < g.L &&
         (long long)g.B * g.Hkv * ((g.M[1] + span * g.g - 1) / (span * g.g)) >= 4LL * num_sms()) {
    span *= g.g;
    ++s_levels;
  }
  dim3 grid1((g.M[1] + span - 1) / span, g.Hkv, g.B);
  pyramid_subtree_kernel<T><<<grid1, threads, 0, s>>>(g, k, pyr, s_levels, span);
  int st = check_launch("pyramid_subtree");
  if (st != PISA_OK) return st;
  if (g.L >= 2 + s_levels) {
    dim3 grid2(chunks, g.Hkv, g.B);
    pyramid_upper_kernel<T><<<grid2, 256, 0, s>>>(g, pyr, 2 + s_levels);
    st = check_launch("pyramid_upper");
  }
  return st;
}

int launch_pyramid(const Geometry& g, int dtype, const void* k, void* pyramid, int32_t* status, cudaStream_t s) {
  if (dtype == PISA_BF16)
    return launch_pyramid_t<__nv_bfloat16>(g, (const __nv_bfloat16*)k, (__nv_bfloat16*)pyramid, s);
  (void)status;
  return launch_pyramid_t<float>(g, (const float*)k, (float*)pyramid, s);
}

}  // namespace pisa
