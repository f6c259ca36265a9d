// Block-sparse attention over the selected leaf blocks, exact-fp32 SIMT path
// (Eq. "selected sparse attention"; causal mask inside selected blocks, App. B).
//
// One warp per (b, KV head, query token) serves the G query heads of the group together, since they
// share one block set (Sec. 3.3).  Scores: one lane per key; P.V: one lane per slice of d.  Online
// softmax over chunks of 32 keys.
#include <math_constants.h>

#include "pisa_common.cuh"

namespace pisa {

namespace {
constexpr int kWarpsPerCta = 4;

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
}  // namespace

template <typename T, int D, int G>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
bsa_simt_kernel(Geometry geo, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                const int32_t* __restrict__ idx, T* __restrict__ out, float* __restrict__ lse) {
  constexpr int DV = D / 32;                  // output dims per lane
  __shared__ __align__(16) float s_q[kWarpsPerCta][G * D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long w = (long long)blockIdx.x * kWarpsPerCta + warp;
  const long long total = (long long)geo.B * geo.Hkv * geo.N;
  if (w >= total) return;
  const int t = (int)(w % geo.N);
  const int h = (int)((w / geo.N) % geo.Hkv);
  const int b = (int)(w / ((long long)geo.N * geo.Hkv));

  float* qf = s_q[warp];
  for (int hh = 0; hh < G; ++hh) {
    const T* row = q + (long long)b * geo.qs[0] + (long long)t * geo.qs[1] + (long long)(h * G + hh) * geo.qs[2];
    for (int e = lane; e < D; e += 32) qf[hh * D + e] = Elem<T>::to_float(row[e]);
  }
  __syncwarp();

  float acc[G][DV];
  float m[G], l[G];
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    m[hh] = -CUDART_INF_F; l[hh] = 0.f;
#pragma unroll
    for (int e = 0; e < DV; ++e) acc[hh][e] = 0.f;
  }
  const T* kb = k + (long long)b * geo.ks[0] + (long long)h * geo.ks[2];
  const T* vb = v + (long long)b * geo.vs[0] + (long long)h * geo.vs[2];
  const int32_t* sel = idx + w * (long long)geo.K;

  for (int slot = 0; slot < geo.K; ++slot) {
    const int blk = sel[slot];
    if (blk < 0 || blk >= geo.M[1]) continue;
    const int lo = blk * geo.C;
    const int hi = min(min(lo + geo.C, geo.N), t + 1);     // causal: keys j <= t only
    for (int j0 = lo; j0 < hi; j0 += 32) {
      const int j = j0 + lane;
      const bool valid = j < hi;
      float z[G], p[G];
      if (valid) {
        dot_row<T, D, G>(kb + (long long)j * geo.ks[1], qf, z);
      } else {
#pragma unroll
        for (int hh = 0; hh < G; ++hh) z[hh] = 0.f;
      }
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        const float zz = valid ? z[hh] * geo.scale : -CUDART_INF_F;
        const float mn = fmaxf(m[hh], warp_max(zz));
        p[hh] = valid ? expf(zz - mn) : 0.f;
        const float alpha = expf(m[hh] - mn);
        l[hh] = l[hh] * alpha + warp_sum(p[hh]);
#pragma unroll
        for (int e = 0; e < DV; ++e) acc[hh][e] *= alpha;
        m[hh] = mn;
      }
      const int cnt = min(32, hi - j0);
      for (int jj = 0; jj < cnt; ++jj) {
        const T* vr = vb + (long long)(j0 + jj) * geo.vs[1] + lane * DV;
        float xv[DV];
#pragma unroll
        for (int e = 0; e < DV; ++e) xv[e] = Elem<T>::to_float(vr[e]);
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          const float ph = __shfl_sync(0xffffffffu, p[hh], jj);
#pragma unroll
          for (int e = 0; e < DV; ++e) acc[hh][e] = fmaf(ph, xv[e], acc[hh][e]);
        }
      }
    }
  }
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    const int hq = h * G + hh;
    const float inv = (l[hh] > 0.f) ? 1.f / l[hh] : 0.f;
    T* orow = out + (long long)b * geo.os[0] + (long long)t * geo.os[1] + (long long)hq * geo.os[2] + lane * DV;
#pragma unroll
    for (int e = 0; e < DV; ++e) orow[e] = Elem<T>::from_float(acc[hh][e] * inv);
    if (lane == 0)
      lse[((long long)b * geo.Hq + hq) * geo.N + t] = (l[hh] > 0.f) ? m[hh] + logf(l[hh]) : -CUDART_INF_F;
  }
}

template <typename T, int D, int G>
static int launch_tdg(const Geometry& g, const void* q, const void* k, const void* v, const int32_t* idx,
                      void* out, float* lse, cudaStream_t s) {
  const long long total = (long long)g.B * g.Hkv * g.N;
  const long long ctas = (total + kWarpsPerCta - 1) / kWarpsPerCta;
  if (ctas > 0x7fffffffLL) return PISA_ERR_UNSUPPORTED;
  bsa_simt_kernel<T, D, G><<<(unsigned)ctas, kWarpsPerCta * 32, 0, s>>>(
      g, (const T*)q, (const T*)k, (const T*)v, idx, (T*)out, lse);
  return check_launch("bsa_simt");
}

template <typename T, int D>
static int launch_td(const Geometry& g, const void* q, const void* k, const void* v, const int32_t* idx,
                     void* out, float* lse, cudaStream_t s) {
  switch (g.G) {
    case 1: return launch_tdg<T, D, 1>(g, q, k, v, idx, out, lse, s);
    case 2: return launch_tdg<T, D, 2>(g, q, k, v, idx, out, lse, s);
    case 4: return launch_tdg<T, D, 4>(g, q, k, v, idx, out, lse, s);
    case 8: return launch_tdg<T, D, 8>(g, q, k, v, idx, out, lse, s);
    case 16: return launch_tdg<T, D, 16>(g, q, k, v, idx, out, lse, s);
    default: return PISA_ERR_UNSUPPORTED;
  }
}

template <typename T>
static int launch_t(const Geometry& g, const void* q, const void* k, const void* v, const int32_t* idx,
                    void* out, float* lse, cudaStream_t s) {
  switch (g.d) {
    case 32: return launch_td<T, 32>(g, q, k, v, idx, out, lse, s);
    case 64: return launch_td<T, 64>(g, q, k, v, idx, out, lse, s);
    case 128: return launch_td<T, 128>(g, q, k, v, idx, out, lse, s);
    default: return PISA_ERR_UNSUPPORTED;
  }
}

int launch_bsa_simt(const Geometry& g, int dtype, const void* q, const void* k, const void* v,
                    const int32_t* idx, void* out, float* lse, cudaStream_t s) {
  if (dtype == PISA_BF16) return launch_t<__nv_bfloat16>(g, q, k, v, idx, out, lse, s);
  return launch_t<float>(g, q, k, v, idx, out, lse, s);
}

}  // namespace pisa
