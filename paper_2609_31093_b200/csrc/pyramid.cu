// Mean-pooled key pyramid (Eq. "mean pyramid", Sec. 3.2).
//
// Level 1 is one streaming pass over k (HBM-bound: N*Hkv*d elements read once); the levels above
// it together hold about M_1/(g-1) nodes per (b, h) and are pooled by one more launch in which a
// CTA owns one (b, h, 16-byte column slice) and walks the levels bottom-up, so no level needs a
// grid-wide barrier: every node it reads was written by the same CTA.
#include "pisa_common.cuh"

namespace pisa {

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

template <typename T>
static int launch_pyramid_t(const Geometry& g, const T* k, T* pyr, cudaStream_t s) {
  constexpr int V = Elem<T>::kVec;
  constexpr int RY = 8;
  const int chunks = g.d / V;
  int threads = chunks * RY;
  if (threads > 256) return PISA_ERR_UNSUPPORTED;
  if (threads < 32) threads = 32;
  dim3 grid1(g.M[1], g.Hkv, g.B);
  pyramid_level1_kernel<T, RY><<<grid1, threads, RY * g.d * sizeof(float), s>>>(g, k, pyr);
  int st = check_launch("pyramid_level1");
  if (st != PISA_OK) return st;
  if (g.L >= 2) {
    dim3 grid2(chunks, g.Hkv, g.B);
    pyramid_upper_kernel<T><<<grid2, 256, 0, s>>>(g, pyr);
    st = check_launch("pyramid_upper");
  }
  return st;
}

int launch_pyramid(const Geometry& g, int dtype, const void* k, void* pyramid, cudaStream_t s) {
  if (dtype == PISA_BF16)
    return launch_pyramid_t<__nv_bfloat16>(g, (const __nv_bfloat16*)k, (__nv_bfloat16*)pyramid, s);
  return launch_pyramid_t<float>(g, (const float*)k, (float*)pyramid, s);
}

}  // namespace pisa
