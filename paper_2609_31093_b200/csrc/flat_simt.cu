// Flat block selection (Sec. 3.1): the O(N^2/C) reference point for the log-linear claim.
// Every eligible leaf is scored with q . (level-1 summary) * scale; scores are soft-maxed over the
// eligible leaves within each query head, summed over the group's heads (App. C), and the forced
// leaves plus the best of the rest are kept.  One warp per (b, KV head, query token); a streaming
// Top-32 (bitonic merge across lanes) so no score row is ever stored.
#include <math_constants.h>

#include "pisa_common.cuh"

namespace pisa {

namespace {
constexpr int kWarpsPerCta = 4;
constexpr int kBig = 0x7fffffff;

template <typename T, int D, int G>
__device__ __forceinline__ void dot_row(const T* __restrict__ row, const float* __restrict__ qf,
                                        float (&z)[G]) {
  constexpr int V = Elem<T>::kVec;
#pragma unroll
  for (int h = 0; h < G; ++h) z[h] = 0.f;
#pragma unroll 2
  for (int c = 0; c < D / V; ++c) {
    float x[V];
    Elem<T>::load_chunk(row + c * V, x);
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float4* qq = reinterpret_cast<const float4*>(qf + h * D + c * V);
#pragma unroll
      for (int v4 = 0; v4 < V / 4; ++v4) {
        const float4 a = qq[v4];
        z[h] = fmaf(x[4 * v4 + 0], a.x, z[h]);
        z[h] = fmaf(x[4 * v4 + 1], a.y, z[h]);
        z[h] = fmaf(x[4 * v4 + 2], a.z, z[h]);
        z[h] = fmaf(x[4 * v4 + 3], a.w, z[h]);
      }
    }
  }
}

// total order used by Select_K: larger score first, ties to the smaller index
__device__ __forceinline__ bool better(float ua, int ia, float ub, int ib) {
  return (ua > ub) || (ua == ub && ia < ib);
}

// one compare-exchange step of a bitonic network across the warp; `desc_region` says whether this
// lane's region is being sorted best-first
__device__ __forceinline__ void cmpswap(float& u, int& i, int j, bool desc_region, int lane) {
  const float ou = __shfl_xor_sync(0xffffffffu, u, j);
  const int oi = __shfl_xor_sync(0xffffffffu, i, j);
  const bool lower = (lane & j) == 0;
  const bool want_better = (lower == desc_region);
  const bool other_better = better(ou, oi, u, i);
  if (other_better == want_better) { u = ou; i = oi; }
}
}  // namespace

template <typename T, int D, int G>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
flat_simt_kernel(Geometry geo, const T* __restrict__ q, const T* __restrict__ pyr, int32_t* __restrict__ idx) {
  __shared__ __align__(16) float s_q[kWarpsPerCta][G * D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long w = (long long)blockIdx.x * kWarpsPerCta + warp;
  const long long total = (long long)geo.B * geo.Hkv * geo.N;
  if (w >= total) return;
  const int t = (int)(w % geo.N);
  const int h = (int)((w / geo.N) % geo.Hkv);
  const int b = (int)(w / ((long long)geo.N * geo.Hkv));
  const int K = geo.K;
  const int c = t / geo.C;
  int32_t* dst = idx + w * (long long)K;

  if (c + 1 <= K) {                       // at most K eligible leaves: keep all, nothing scored
    for (int s = lane; s < K; s += 32) dst[s] = (s <= c) ? s : -1;
    return;
  }
  float* qf = s_q[warp];
  for (int hh = 0; hh < G; ++hh) {
    const T* row = q + (long long)b * geo.qs[0] + (long long)t * geo.qs[1] + (long long)(h * G + hh) * geo.qs[2];
    for (int e = lane; e < D; e += 32) qf[hh * D + e] = Elem<T>::to_float(row[e]);
  }
  __syncwarp();
  const T* lvl1 = pyr + geo.level_off[1] + ((long long)b * geo.Hkv + h) * geo.M[1] * D;

  // pass 1: per-head softmax normaliser over the eligible leaves 0..c
  float m[G], l[G];
#pragma unroll
  for (int hh = 0; hh < G; ++hh) { m[hh] = -CUDART_INF_F; l[hh] = 0.f; }
  for (int i = lane; i <= c; i += 32) {
    float z[G];
    dot_row<T, D, G>(lvl1 + (long long)i * D, qf, z);
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      const float zz = z[hh] * geo.scale;
      const float mn = fmaxf(m[hh], zz);
      l[hh] = l[hh] * expf(m[hh] - mn) + expf(zz - mn);
      m[hh] = mn;
    }
  }
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    const float mw = warp_max(m[hh]);
    const float part = (l[hh] > 0.f) ? l[hh] * expf(m[hh] - mw) : 0.f;
    l[hh] = warp_sum(part);
    m[hh] = mw;
  }

  // pass 2: grouped normalised score of the non-forced leaves 1..c-2, streaming Top-32
  float best_u = -CUDART_INF_F;
  int best_i = kBig;
  for (int i0 = 1; i0 <= c - 2; i0 += 32) {
    const int i = i0 + lane;
    float u = -CUDART_INF_F;
    int ui = kBig;
    if (i <= c - 2) {
      float z[G];
      dot_row<T, D, G>(lvl1 + (long long)i * D, qf, z);
      u = 0.f;
#pragma unroll
      for (int hh = 0; hh < G; ++hh) u += expf(z[hh] * geo.scale - m[hh]) / l[hh];
      ui = i;
    }
    // skip the merge when nothing in this chunk beats the current 32nd best
    const float worst_u = __shfl_sync(0xffffffffu, best_u, 31);
    const int worst_i = __shfl_sync(0xffffffffu, best_i, 31);
    if (__ballot_sync(0xffffffffu, better(u, ui, worst_u, worst_i)) == 0u) continue;
    // sort the chunk best-first
#pragma unroll
    for (int kk = 2; kk <= 32; kk <<= 1) {
#pragma unroll
      for (int j = kk >> 1; j > 0; j >>= 1) cmpswap(u, ui, j, (lane & kk) == 0, lane);
    }
    // best-first list vs reversed chunk: element-wise winner is a bitonic sequence of the top 32
    const float ru = __shfl_sync(0xffffffffu, u, 31 - lane);
    const int ri = __shfl_sync(0xffffffffu, ui, 31 - lane);
    if (better(ru, ri, best_u, best_i)) { best_u = ru; best_i = ri; }
#pragma unroll
    for (int j = 16; j > 0; j >>= 1) cmpswap(best_u, best_i, j, true, lane);
  }

  // forced leaves plus the K - |forced| best, ascending by index
  const int nf = 3;                        // c >= K >= 3 here, so 0, c-1, c are distinct
  int mine = kBig;
  if (lane < K - nf) mine = best_i;
  else if (lane == K - nf) mine = 0;
  else if (lane == K - nf + 1) mine = c - 1;
  else if (lane == K - nf + 2) mine = c;
  float key = -(float)0;                   // sort on the index alone: reuse cmpswap with equal scores
#pragma unroll
  for (int kk = 2; kk <= 32; kk <<= 1) {
#pragma unroll
    for (int j = kk >> 1; j > 0; j >>= 1) cmpswap(key, mine, j, (lane & kk) == 0, lane);
  }
  if (lane < K) dst[lane] = (mine == kBig) ? -1 : mine;
}

template <typename T, int D, int G>
static int launch_tdg(const Geometry& g, const void* q, const void* pyr, int32_t* idx, cudaStream_t s) {
  const long long total = (long long)g.B * g.Hkv * g.N;
  const long long ctas = (total + kWarpsPerCta - 1) / kWarpsPerCta;
  if (ctas > 0x7fffffffLL) return PISA_ERR_UNSUPPORTED;
  flat_simt_kernel<T, D, G><<<(unsigned)ctas, kWarpsPerCta * 32, 0, s>>>(g, (const T*)q, (const T*)pyr, idx);
  return check_launch("flat_simt");
}

template <typename T, int D>
static int launch_td(const Geometry& g, const void* q, const void* pyr, int32_t* idx, cudaStream_t s) {
  switch (g.G) {
    case 1: return launch_tdg<T, D, 1>(g, q, pyr, idx, s);
    case 2: return launch_tdg<T, D, 2>(g, q, pyr, idx, s);
    case 4: return launch_tdg<T, D, 4>(g, q, pyr, idx, s);
    case 8: return launch_tdg<T, D, 8>(g, q, pyr, idx, s);
    case 16: return launch_tdg<T, D, 16>(g, q, pyr, idx, s);
    default: return PISA_ERR_UNSUPPORTED;
  }
}

template <typename T>
static int launch_t(const Geometry& g, const void* q, const void* pyr, int32_t* idx, cudaStream_t s) {
  switch (g.d) {
    case 32: return launch_td<T, 32>(g, q, pyr, idx, s);
    case 64: return launch_td<T, 64>(g, q, pyr, idx, s);
    case 128: return launch_td<T, 128>(g, q, pyr, idx, s);
    default: return PISA_ERR_UNSUPPORTED;
  }
}

int launch_flat_simt(const Geometry& g, int dtype, const void* q, const void* pyramid, int32_t* idx,
                     cudaStream_t s) {
  if (dtype == PISA_BF16) return launch_t<__nv_bfloat16>(g, q, pyramid, idx, s);
  return launch_t<float>(g, q, pyramid, idx, s);
}

}  // namespace pisa
