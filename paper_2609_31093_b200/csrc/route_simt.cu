// Coarse-to-fine Top-K routing, one warp per (b, KV head, query token), every level fused in one
// launch (Sec. 3.2 "Coarse-to-fine block selection"; the paper's "per-query" schedule, App. B).
//
// This is the exact-fp32 SIMT path: it serves the fp32 dtype, every shape the tensor-core path does
// not cover, and the cross-check of that path.  The same kernel, stopped after the intermediate
// levels (LEAF = false), is stage 1 of the two-stage schedule (Algorithm 1): it then stores the
// kept level-2 nodes, whose children are the leaf candidates, instead of scoring the leaves.
//
// Per warp state lives in shared memory: the G query vectors in fp32, the sorted candidate list
// (at most g*K entries) and the candidates' grouped scores.  The query-summary score matrix is
// never formed: each candidate's children are read, dotted with the G queries, reduced by the
// block score and dropped.
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

// Running statistics of one head's logits for the three block scores (Sec. 4.3):
// LSE keeps (max, sum exp); mean / mean+var/2 keep shifted first and second moments.
struct Stat {
  float a, b, c;   // LSE: a = max, b = sum exp(z - max).  moments: a = shift, b = S1, c = S2
  int n;
};
__device__ __forceinline__ void stat_init(Stat& s, int mode) {
  s.a = (mode == PISA_SCORE_LSE) ? -CUDART_INF_F : 0.f;
  s.b = 0.f; s.c = 0.f; s.n = 0;
}
__device__ __forceinline__ void stat_add(Stat& s, float z, int mode) {
  if (mode == PISA_SCORE_LSE) {
    const float m = fmaxf(s.a, z);
    s.b = s.b * expf(s.a - m) + expf(z - m);
    s.a = m;
  } else {
    if (s.n == 0) s.a = z;
    const float dz = z - s.a;
    s.b += dz; s.c += dz * dz;
  }
  s.n += 1;
}
__device__ __forceinline__ float stat_finish(const Stat& s, int mode) {
  if (mode == PISA_SCORE_LSE) return s.a + logf(s.b);
  const float inv = 1.f / (float)s.n;
  const float mean_d = s.b * inv;
  if (mode == PISA_SCORE_MEAN) return s.a + mean_d;
  return s.a + mean_d + 0.5f * (s.c * inv - mean_d * mean_d);
}
// Merge the lanes' partial statistics of one head (leaf level: one lane per key).
__device__ __forceinline__ float stat_warp_finish(Stat s, int mode) {
  if (mode == PISA_SCORE_LSE) {
    const float m = warp_max(s.a);
    const float part = (s.n > 0) ? s.b * expf(s.a - m) : 0.f;
    return m + logf(warp_sum(part));
  }
  // re-centre every lane's moments on lane 0's shift, then add
  const float shift = __shfl_sync(0xffffffffu, s.a, 0);
  const float delta = s.a - shift;
  const float s1 = (s.n > 0) ? s.b + (float)s.n * delta : 0.f;
  const float s2 = (s.n > 0) ? s.c + 2.f * delta * s.b + (float)s.n * delta * delta : 0.f;
  const float n = warp_sum((float)s.n), S1 = warp_sum(s1), S2 = warp_sum(s2);
  const float mean_d = S1 / n;
  if (mode == PISA_SCORE_MEAN) return shift + mean_d;
  return shift + mean_d + 0.5f * (S2 / n - mean_d * mean_d);
}

}  // namespace

template <typename T, int D, int G, bool LEAF>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
route_simt_kernel(Geometry geo, const T* __restrict__ q, const T* __restrict__ k,
                  const T* __restrict__ pyr, int32_t* __restrict__ idx, float* __restrict__ margin,
                  int32_t* __restrict__ cand_out) {
  __shared__ __align__(16) float s_q[kWarpsPerCta][G * D];
  __shared__ int s_cand[kWarpsPerCta][2][kMaxCand];
  __shared__ __align__(16) float s_u[kWarpsPerCta][kMaxCand];
  __shared__ float s_cut[kWarpsPerCta][2];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long w = (long long)blockIdx.x * kWarpsPerCta + warp;
  const long long total = (long long)geo.B * geo.Hkv * geo.N;
  if (w >= total) return;
  const int t = (int)(w % geo.N);
  const int h = (int)((w / geo.N) % geo.Hkv);
  const int b = (int)(w / ((long long)geo.N * geo.Hkv));
  const int mode = geo.score_mode;
  const int K = geo.K, g = geo.g, C = geo.C;
  const int c = t / C;

  float* qf = s_q[warp];
  float* u = s_u[warp];
  for (int hh = 0; hh < G; ++hh) {
    const T* row = q + (long long)b * geo.qs[0] + (long long)t * geo.qs[1] + (long long)(h * G + hh) * geo.qs[2];
    for (int e = lane; e < D; e += 32) qf[hh * D + e] = Elem<T>::to_float(row[e]);
  }
  int cur = 0;
  int n = 1;
  if (lane == 0) s_cand[warp][0][0] = 0;
  float min_gap = CUDART_INF_F;
  __syncwarp();

  for (int l = geo.L; l >= 1; --l) {
    int* cand = s_cand[warp][cur];
    int* next = s_cand[warp][cur ^ 1];
    const long long span = geo.span[l];
    const int anc_c = (int)(c / span);
    const int f1 = (c >= 1) ? (int)((c - 1) / span) : 0;
    // eligible candidates: exist and do not start after the query's leaf (sorted list => prefix)
    int nV = 0;
    for (int s0 = 0; s0 < n; s0 += 32) {
      const int s = s0 + lane;
      const bool ok = (s < n) && (cand[s] <= anc_c);
      nV += __popc(__ballot_sync(0xffffffffu, ok));
    }
    const bool prune = nV > K;
    if (LEAF || l > 1) {
      if (prune) {
        if (l > 1) {
          // intermediate level: one lane per candidate, its g child summaries read in-lane
          const T* below = pyr + geo.level_off[l - 1] + ((long long)b * geo.Hkv + h) * geo.M[l - 1] * D;
          for (int s = lane; s < nV; s += 32) {
            const int i = cand[s];
            float score = CUDART_INF_F;            // forced nodes rank first and are never scored
            if (i != 0 && i != f1 && i != anc_c) {
              Stat st[G];
#pragma unroll
              for (int hh = 0; hh < G; ++hh) stat_init(st[hh], mode);
              const int lo = i * g, hi = min(lo + g, geo.M[l - 1]);
              for (int r = lo; r < hi; ++r) {
                float z[G];
                dot_row<T, D, G>(below + (long long)r * D, qf, z);
#pragma unroll
                for (int hh = 0; hh < G; ++hh) stat_add(st[hh], z[hh] * geo.scale, mode);
              }
              score = 0.f;
#pragma unroll
              for (int hh = 0; hh < G; ++hh) score += stat_finish(st[hh], mode);
            }
            u[s] = score;
          }
        } else {
          // leaf level: one candidate at a time, one lane per raw key
          const T* kb = k + (long long)b * geo.ks[0] + (long long)h * geo.ks[2];
          for (int s = 0; s < nV; ++s) {
            const int i = cand[s];
            if (i == 0 || i == f1 || i == anc_c) {
              if (lane == 0) u[s] = CUDART_INF_F;
              continue;
            }
            Stat st[G];
#pragma unroll
            for (int hh = 0; hh < G; ++hh) stat_init(st[hh], mode);
            const int lo = i * C, hi = min(lo + C, geo.N);
            for (int j = lo + lane; j < hi; j += 32) {
              float z[G];
              dot_row<T, D, G>(kb + (long long)j * geo.ks[1], qf, z);
#pragma unroll
              for (int hh = 0; hh < G; ++hh) stat_add(st[hh], z[hh] * geo.scale, mode);
            }
            float score = 0.f;
#pragma unroll
            for (int hh = 0; hh < G; ++hh) score += stat_warp_finish(st[hh], mode);
            if (lane == 0) u[s] = score;
          }
        }
        __syncwarp();
      }
      // Select_K: rank by (score desc, position asc); keep rank < K.  Without pruning keep all.
      int base = 0;
      for (int s0 = 0; s0 < nV; s0 += 32) {
        const int s = s0 + lane;
        bool keep = s < nV;
        if (prune) {
          int rank = 0;
          const float ui = (s < nV) ? u[s] : 0.f;
          for (int j = 0; j < nV; ++j) {
            const float uj = u[j];
            rank += (uj > ui) || (uj == ui && j < s);
          }
          keep = keep && (rank < K);
          if (s < nV && rank == K - 1) s_cut[warp][0] = ui;
          if (s < nV && rank == K) s_cut[warp][1] = ui;
        }
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        const int pos = base + __popc(bal & ((1u << lane) - 1u));
        if (keep) {
          const int i = cand[s];
          if (!LEAF && l == 2) {
            cand_out[w * (long long)K + pos] = i;        // two-stage schedule: kept level-2 nodes
          } else if (l > 1) {
            for (int r = 0; r < g; ++r) next[pos * g + r] = i * g + r;
          } else {
            next[pos] = i;
          }
        }
        base += __popc(bal);
      }
      __syncwarp();
      if (prune) {
        const float a = s_cut[warp][0], bb = s_cut[warp][1];
        if (a < CUDART_INF_F) min_gap = fminf(min_gap, (a - bb) / fmaxf(fabsf(a), 1.f));
      }
      if (!LEAF && l == 2) {
        // stage 1 of the two-stage schedule ends here (Algorithm 1): the leaf level is scored
        // key-block-major by the tensor-core stage
        for (int s = base + lane; s < K; s += 32) cand_out[w * (long long)K + s] = -1;
        if (margin != nullptr && lane == 0) margin[w] = min_gap;
        return;
      }
      n = (l > 1) ? base * g : base;
      cur ^= 1;
    }
  }
  // leaf level done: the kept leaves, ascending, padded with -1
  const int* fin = s_cand[warp][cur];
  int32_t* dst = idx + w * (long long)K;
  for (int s = lane; s < K; s += 32) dst[s] = (s < n) ? fin[s] : -1;
  if (margin != nullptr && lane == 0) margin[w] = min_gap;
}

template <typename T, int D, int G>
static int launch_route_tdg(const Geometry& g, const void* q, const void* k, const void* pyr,
                            int32_t* idx, float* margin, int32_t* cand_out, bool leaf, cudaStream_t s) {
  const long long total = (long long)g.B * g.Hkv * g.N;
  const long long ctas = (total + kWarpsPerCta - 1) / kWarpsPerCta;
  if (ctas > 0x7fffffffLL) return PISA_ERR_UNSUPPORTED;
  if (leaf)
    route_simt_kernel<T, D, G, true><<<(unsigned)ctas, kWarpsPerCta * 32, 0, s>>>(
        g, (const T*)q, (const T*)k, (const T*)pyr, idx, margin, nullptr);
  else
    route_simt_kernel<T, D, G, false><<<(unsigned)ctas, kWarpsPerCta * 32, 0, s>>>(
        g, (const T*)q, (const T*)k, (const T*)pyr, idx, margin, cand_out);
  return check_launch("route_simt");
}

template <typename T, int D>
static int launch_route_td(const Geometry& g, const void* q, const void* k, const void* pyr, int32_t* idx,
                           float* margin, int32_t* cand_out, bool leaf, cudaStream_t s) {
  switch (g.G) {
    case 1: return launch_route_tdg<T, D, 1>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    case 2: return launch_route_tdg<T, D, 2>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    case 4: return launch_route_tdg<T, D, 4>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    case 8: return launch_route_tdg<T, D, 8>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    case 16: return launch_route_tdg<T, D, 16>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    default: return PISA_ERR_UNSUPPORTED;
  }
}

template <typename T>
static int launch_route_t(const Geometry& g, const void* q, const void* k, const void* pyr, int32_t* idx,
                          float* margin, int32_t* cand_out, bool leaf, cudaStream_t s) {
  switch (g.d) {
    case 32: return launch_route_td<T, 32>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    case 64: return launch_route_td<T, 64>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    case 128: return launch_route_td<T, 128>(g, q, k, pyr, idx, margin, cand_out, leaf, s);
    default: return PISA_ERR_UNSUPPORTED;
  }
}

int launch_route_simt(const Geometry& g, int dtype, const void* q, const void* k, const void* pyramid,
                      int32_t* idx, float* margin, cudaStream_t s) {
  if (dtype == PISA_BF16) return launch_route_t<__nv_bfloat16>(g, q, k, pyramid, idx, margin, nullptr, true, s);
  return launch_route_t<float>(g, q, k, pyramid, idx, margin, nullptr, true, s);
}

int launch_route_stage1_simt(const Geometry& g, int dtype, const void* q, const void* pyramid,
                             int32_t* cand_out, float* margin, cudaStream_t s) {
  if (g.L < 2) return PISA_ERR_UNSUPPORTED;
  if (dtype == PISA_BF16)
    return launch_route_t<__nv_bfloat16>(g, q, nullptr, pyramid, nullptr, margin, cand_out, false, s);
  return launch_route_t<float>(g, q, nullptr, pyramid, nullptr, margin, cand_out, false, s);
}

}  // namespace pisa
