// Per-head softmax denominators of the selected leaf blocks, exact fp32:
//   sel_lse[b, hq, t, s] = log sum_{j in leaf idx[b,h,t,s], j <= t} exp(q[b,t,hq] . k[b,j,h] * scale)
// (Eq. "direct child LSE" at the leaf level with the causal mask of App. B inside the row's own leaf).
// One warp per (b, KV head, token, slot); lanes take keys, online log-sum-exp per head.  This is the
// any-shape version behind pisa_route's sel_lse output; the tensor-core routing emits the same numbers
// from its leaf-scoring tiles instead.
#include <math_constants.h>

#include "pisa_common.cuh"

namespace pisa {

namespace {
constexpr int kWarpsPerCta = 4;

template <typename T>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
sel_lse_simt_kernel(Geometry geo, const T* __restrict__ q, const T* __restrict__ k, const int32_t* __restrict__ idx,
                    float* __restrict__ sel_lse, int32_t* status) {
  constexpr int V = Elem<T>::kVec;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long w = (long long)blockIdx.x * kWarpsPerCta + warp;     // ((b*Hkv + h)*N + t)*K + s
  const long long total = (long long)geo.B * geo.Hkv * geo.N * geo.K;
  if (w >= total) return;
  const int s = (int)(w % geo.K);
  const long long row = w / geo.K;
  const int t = (int)(row % geo.N);
  const int h = (int)((row / geo.N) % geo.Hkv);
  const int b = (int)(row / ((long long)geo.N * geo.Hkv));
  const int leaf = idx[w];
  const int c = t / geo.C;
  bool live = leaf >= 0 && leaf <= c && leaf < geo.M[1];
  if ((geo.debug & PISA_DEBUG_BOUNDS) && leaf != -1 && !live && lane == 0) atomicExch(status, (int)PISA_ERR_BOUNDS);
  const int lo = leaf * geo.C;
  const int hi = live ? min(min(lo + geo.C, geo.N), t + 1) : lo;
  for (int hh = 0; hh < geo.G; ++hh) {
    const T* qrow = q + (long long)b * geo.qs[0] + (long long)t * geo.qs[1] + (long long)(h * geo.G + hh) * geo.qs[2];
    float m = -CUDART_INF_F, ssum = 0.f;
    for (int j = lo + lane; j < hi; j += 32) {
      const T* krow = k + (long long)b * geo.ks[0] + (long long)j * geo.ks[1] + (long long)h * geo.ks[2];
      float z = 0.f;
      for (int e0 = 0; e0 < geo.d; e0 += V) {
        float x[V], y[V];
        Elem<T>::load_chunk(krow + e0, x);
        Elem<T>::load_chunk(qrow + e0, y);
#pragma unroll
        for (int e = 0; e < V; ++e) z = fmaf(x[e], y[e], z);
      }
      z *= geo.scale;
      const float mn = fmaxf(m, z);
      ssum = ssum * expf(m - mn) + expf(z - mn);
      m = mn;
    }
    const float mw = warp_max(m);
    const float part = (ssum > 0.f) ? ssum * expf(m - mw) : 0.f;
    const float tot = warp_sum(part);
    if (lane == 0)
      sel_lse[(((long long)b * geo.Hq + h * geo.G + hh) * geo.N + t) * geo.K + s] =
          (tot > 0.f) ? mw + logf(tot) : -CUDART_INF_F;
  }
}

}  // namespace

int launch_sel_lse_simt(const Geometry& g, int dtype, const void* q, const void* k, const int32_t* idx,
                        float* sel_lse, int32_t* status, cudaStream_t s) {
  const long long total = (long long)g.B * g.Hkv * g.N * g.K;
  const long long ctas = (total + kWarpsPerCta - 1) / kWarpsPerCta;
  if (ctas > 0x7fffffffLL) return PISA_ERR_UNSUPPORTED;
  if (dtype == PISA_BF16)
    sel_lse_simt_kernel<__nv_bfloat16><<<(unsigned)ctas, kWarpsPerCta * 32, 0, s>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, idx, sel_lse, status);
  else
    sel_lse_simt_kernel<float><<<(unsigned)ctas, kWarpsPerCta * 32, 0, s>>>(g, (const float*)q, (const float*)k, idx,
                                                                           sel_lse, status);
  return check_launch("sel_lse_simt");
}

}  // namespace pisa
