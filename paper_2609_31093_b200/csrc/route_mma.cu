// Stage 1 of the two-stage routing schedule (Algorithm 1, levels L..2) for bf16 inputs, one warp per
// (b, KV head, query token), with the candidate scoring on warp-level tensor-core MMAs.
//
// At one level a token scores at most g*K candidates, each from g child summaries, against its own G
// query vectors: a gathered [g*K*g rows] x [d] by [d] x [G] product, far too small and too irregular
// for a CTA-wide UMMA tile but a natural fit for m16n8k16 fragments held in registers.  The child
// summaries are the A operand, loaded straight from global/L2 into fragment registers with 32-byte
// loads (the k index of both operands is permuted identically so that a lane's fragment pieces are
// contiguous in memory: lane (gid, tig) owns 32-byte chunk c8*4 + tig of its row for every group c8 of
// 64 elements, so the four lanes of a row read one whole 128-byte line per load); the G query vectors,
// padded to 8 columns, are the B operand and stay in registers for all levels.  A candidate's g children occupy rows (r, r+8) of consecutive tiles, so
// their logits meet in one lane and the child LSE needs no shuffles; the head sum takes two.
// The selection logic (eligibility, forced nodes, Select_K, expansion) is the SIMT kernel's.
#include <math_constants.h>

#include "mma_frag.cuh"
#include "pisa_common.cuh"

namespace pisa {

using namespace frag;

namespace {

constexpr int kWarpsPerCta = 8;

}  // namespace

// MODE: PISA_SCORE_LSE, _MEAN (mean of the children's logits) or _MEAN_VAR (mean + variance / 2), Sec. 4.3
template <int D, int NT, bool G2, int MODE>
// three CTAs per SM (at most 85 registers) for the narrow fan-in-2 instantiations at d = 128: measured 8.5 ms against
// 8.7 (compiler's choice, 76 registers), 9.3 (64) and 9.7 (128) at the headline shape; four at d = 64 (64 registers:
// 1.54 ms against 2.02 with two, B1 Hq32 Hkv2 d64 N131072 C64 K8)
__global__ void __launch_bounds__(kWarpsPerCta * 32, (G2 && D == 64) ? 4 : (G2 && NT == 1) ? 3 : 1)
route_stage1_mma_kernel(Geometry geo, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ pyr,
                        int32_t* __restrict__ par_out, float* __restrict__ margin) {
  constexpr int C8 = D / 64;              // groups of four 32-byte chunks per row (one chunk per tig)
  __shared__ int s_cand[kWarpsPerCta][2][kMaxCand];
  __shared__ __align__(16) float s_u[kWarpsPerCta][kMaxCand];
  __shared__ float s_cut[kWarpsPerCta][2];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const long long w = (long long)blockIdx.x * kWarpsPerCta + warp;
  const long long total = (long long)geo.B * geo.Hkv * geo.N;
  if (w >= total) return;
  const int t = (int)(w % geo.N);
  const int h = (int)((w / geo.N) % geo.Hkv);
  const int b = (int)(w / ((long long)geo.N * geo.Hkv));
  const int K = geo.K, g = geo.g, G = geo.G;
  const int c = t / geo.C;
  float* u = s_u[warp];

  // B fragments: column n = gid is query head nt*8 + gid (zero beyond G); k permuted as the A loads
  uint32_t bq[NT][C8][8];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int head = nt * 8 + gid;
    const __nv_bfloat16* row = q + (long long)b * geo.qs[0] + (long long)t * geo.qs[1] +
                               (long long)(h * G + head) * geo.qs[2];
#pragma unroll
    for (int c8 = 0; c8 < C8; ++c8) {
      uint4 v0 = make_uint4(0u, 0u, 0u, 0u), v1 = v0;             // query rows are only 16-byte aligned
      if (head < G) { v0 = ldg128(row + (c8 * 4 + tig) * 16); v1 = ldg128(row + (c8 * 4 + tig) * 16 + 8); }
      bq[nt][c8][0] = v0.x; bq[nt][c8][1] = v0.y; bq[nt][c8][2] = v0.z; bq[nt][c8][3] = v0.w;
      bq[nt][c8][4] = v1.x; bq[nt][c8][5] = v1.y; bq[nt][c8][6] = v1.z; bq[nt][c8][7] = v1.w;
    }
  }
  const U32x8 zero8 = {{0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u}};

  // Levels that hold at most K nodes cannot prune: every node that does not start after the query's leaf is
  // kept and expanded.  The walk therefore starts at the highest level with more than K nodes (or at level
  // 2), whose candidates are simply the nodes 0 .. anc(c) (at most g*K of them: the level above holds <= K).
  int l_start = 2;
  for (int l = geo.L; l > 2; --l)
    if (geo.M[l] > K) { l_start = l; break; }
  int cur = 0;
  int n;
  {
    const unsigned span0 = (unsigned)min(geo.span[l_start], (long long)0x7fffffff);
    n = min((int)((unsigned)c / span0), geo.M[l_start] - 1) + 1;
    for (int s = lane; s < n; s += 32) s_cand[warp][0][s] = s;
  }
  float min_gap = CUDART_INF_F;
  __syncwarp();

  for (int l = l_start; l >= 2; --l) {
    int* cand = s_cand[warp][cur];
    int* next = s_cand[warp][cur ^ 1];
    // leaves under a level-l node; c < 2^31, so a span beyond that just means ancestor 0 (32-bit division)
    const unsigned span = (unsigned)min(geo.span[l], (long long)0x7fffffff);
    const int anc_c = (int)((unsigned)c / span);
    const int f1 = (c >= 1) ? (int)((unsigned)(c - 1) / span) : 0;
    int nV = 0;
    for (int s0 = 0; s0 < n; s0 += 32) {
      const int s = s0 + lane;
      const bool ok = (s < n) && (cand[s] <= anc_c);
      nV += __popc(__ballot_sync(0xffffffffu, ok));
    }
    const bool prune = nV > K;
    if (prune) {
      const int Mb = geo.M[l - 1];
      const __nv_bfloat16* below = pyr + geo.level_off[l - 1] + ((long long)b * geo.Hkv + h) * Mb * D;
      for (int k0 = 0; k0 < nV; k0 += 8) {
        const int kap = k0 + gid;
        const bool has = kap < nV;
        const int node = has ? cand[kap] : 0;
        float usum = 0.f;
        if (G2) {
          // fan-in 2: both children of a candidate meet in one lane; LSE(a, b) = max + log(1 + e^-|a-b|)
          const int ch_lo = node * 2, ch_hi = ch_lo + 1;
          const bool ok_hi = has && ch_hi < Mb;
          // rows without a candidate (kap >= nV: node 0) or without a second child (ragged level: the first
          // child again) load valid summaries all the same; their logits are dropped below
          const long long off_hi = (long long)(ok_hi ? ch_hi : ch_lo) * D;
          float accs[NT][4];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) accs[nt][0] = accs[nt][1] = accs[nt][2] = accs[nt][3] = 0.f;
#pragma unroll
          for (int c8 = 0; c8 < C8; ++c8) {         // one 64-element group of the row at a time: 16 live data registers
            const U32x8 lo = ldg256(below + (long long)ch_lo * D + (c8 * 4 + tig) * 16);
            const U32x8 hi = ldg256(below + off_hi + (c8 * 4 + tig) * 16);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
              for (int i = 0; i < 8; i += 2)
                mma_bf16_16816(accs[nt], lo.r[i], hi.r[i], lo.r[i + 1], hi.r[i + 1], bq[nt][c8][i], bq[nt][c8][i + 1]);
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const float (&acc)[4] = accs[nt];
#pragma unroll
            for (int jh = 0; jh < 2; ++jh) {
              const float za = acc[jh] * geo.scale, zb = acc[2 + jh] * geo.scale;
              float sc2;
              if (MODE == PISA_SCORE_LSE) sc2 = fmaxf(za, zb) + __logf(1.f + __expf(-fabsf(za - zb)));
              else sc2 = 0.5f * (za + zb) + ((MODE == PISA_SCORE_MEAN_VAR) ? 0.125f * (za - zb) * (za - zb) : 0.f);
              if (nt * 8 + 2 * tig + jh < G) usum += ok_hi ? sc2 : za;
            }
          }
          if (!has) usum = 0.f;
        } else {
          float m[NT][2], ssum[NT][2], sq[NT][2];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            m[nt][0] = m[nt][1] = -CUDART_INF_F; ssum[nt][0] = ssum[nt][1] = 0.f; sq[nt][0] = sq[nt][1] = 0.f;
          }
          const int nch = has ? min(g, Mb - node * g) : 1;                 // valid children of the candidate
          for (int r0 = 0; r0 < g; r0 += 2) {
            const int ch_lo = node * g + r0, ch_hi = ch_lo + 1;
            const bool ok_lo = has && ch_lo < Mb, ok_hi = has && (r0 + 1 < g) && ch_hi < Mb;
            U32x8 lo[C8], hi[C8];
#pragma unroll
            for (int c8 = 0; c8 < C8; ++c8) {
              lo[c8] = ok_lo ? ldg256(below + (long long)ch_lo * D + (c8 * 4 + tig) * 16) : zero8;
              hi[c8] = ok_hi ? ldg256(below + (long long)ch_hi * D + (c8 * 4 + tig) * 16) : zero8;
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int c8 = 0; c8 < C8; ++c8)
#pragma unroll
                for (int i = 0; i < 8; i += 2)
                  mma_bf16_16816(acc, lo[c8].r[i], hi[c8].r[i], lo[c8].r[i + 1], hi[c8].r[i + 1], bq[nt][c8][i],
                                 bq[nt][c8][i + 1]);
              // acc[0..1]: child lo, heads nt*8 + 2*tig + {0,1};  acc[2..3]: child hi, same heads
#pragma unroll
              for (int jh = 0; jh < 2; ++jh) {
                if (MODE == PISA_SCORE_LSE) {
                  if (ok_lo) lse_add(m[nt][jh], ssum[nt][jh], acc[jh] * geo.scale);
                  if (ok_hi) lse_add(m[nt][jh], ssum[nt][jh], acc[2 + jh] * geo.scale);
                } else {
                  // m: the first child's logit (shift); ssum, sq: first and second moments about it
                  if (r0 == 0) m[nt][jh] = acc[jh] * geo.scale;
                  if (ok_lo) { const float dl = acc[jh] * geo.scale - m[nt][jh]; ssum[nt][jh] += dl; sq[nt][jh] += dl * dl; }
                  if (ok_hi) { const float dl = acc[2 + jh] * geo.scale - m[nt][jh]; ssum[nt][jh] += dl; sq[nt][jh] += dl * dl; }
                }
              }
            }
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int jh = 0; jh < 2; ++jh)
              if (nt * 8 + 2 * tig + jh < G && has) {
                if (MODE == PISA_SCORE_LSE) usum += m[nt][jh] + __logf(ssum[nt][jh]);
                else {
                  const float mu = ssum[nt][jh] / (float)nch;
                  usum += m[nt][jh] + mu +
                          ((MODE == PISA_SCORE_MEAN_VAR) ? 0.5f * fmaxf(sq[nt][jh] / (float)nch - mu * mu, 0.f) : 0.f);
                }
              }
        }
        usum += __shfl_xor_sync(0xffffffffu, usum, 1);
        usum += __shfl_xor_sync(0xffffffffu, usum, 2);
        if (has && tig == 0) u[kap] = (node == 0 || node == f1 || node == anc_c) ? forced_score(kap) : usum;
      }
      if (lane < 4 && nV + lane < kMaxCand) u[nV + lane] = -CUDART_INF_F;     // padding read by the 16-byte loads
      __syncwarp();
    }
    // Select_K: rank by (score desc, position asc); keep rank < K.  Without pruning keep all.
    int rank[kMaxCand / 32];
    const bool sorted = prune && nV <= 64;       // the common case: a sorting network instead of ranks
    bool keep_s[2] = {false, false};
    float cut_a = 0.f, cut_b = 0.f;
    if (sorted) {
      const float u0 = (lane < nV) ? u[lane] : -CUDART_INF_F, u1 = (lane + 32 < nV) ? u[lane + 32] : -CUDART_INF_F;
      warp_select_sorted64(u0, u1, K, lane, keep_s[0], keep_s[1], cut_a, cut_b);
    } else if (prune) {
      warp_select_ranks(u, nV, lane, rank);
    }
    int base = 0;
#pragma unroll
    for (int ch = 0; ch < kMaxCand / 32; ++ch) {
      const int s0 = ch * 32;
      if (s0 >= nV) break;
      const int s = s0 + lane;
      bool keep = s < nV;
      if (sorted) {
        keep = keep && keep_s[ch & 1];
      } else if (prune) {
        keep = keep && (rank[ch] < K);
        if (s < nV && rank[ch] == K - 1) s_cut[warp][0] = u[s];
        if (s < nV && rank[ch] == K) s_cut[warp][1] = u[s];
      }
      const unsigned bal = __ballot_sync(0xffffffffu, keep);
      const int pos = base + __popc(bal & ((1u << lane) - 1u));
      if (keep) {
        const int i = cand[s];
        if (l == 2) {
          par_out[w * (long long)K + pos] = i;
        } else {
          for (int r = 0; r < g; ++r) next[pos * g + r] = i * g + r;
        }
      }
      base += __popc(bal);
    }
    __syncwarp();
    if (prune) {
      const float a = sorted ? cut_a : s_cut[warp][0], bb = sorted ? cut_b : s_cut[warp][1];
      if (a < kForcedFloor) min_gap = fminf(min_gap, (a - bb) / fmaxf(fabsf(a), 1.f));
    }
    if (l == 2) {
      for (int s = base + lane; s < K; s += 32) par_out[w * (long long)K + s] = -1;
      if (margin != nullptr && lane == 0) margin[w] = min_gap;
      return;
    }
    n = base * g;
    cur ^= 1;
  }
}

template <int D, int NT>
static int launch_dn(const Geometry& g, const void* q, const void* pyr, int32_t* par, float* margin, cudaStream_t s) {
  const long long total = (long long)g.B * g.Hkv * g.N;
  const long long ctas = (total + kWarpsPerCta - 1) / kWarpsPerCta;
  if (ctas > 0x7fffffffLL) return PISA_ERR_UNSUPPORTED;
  auto go = [&](auto kern) {
    kern<<<(unsigned)ctas, kWarpsPerCta * 32, 0, s>>>(g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)pyr, par, margin);
  };
  const bool g2 = g.g == 2;
  switch (g.score_mode) {
    case PISA_SCORE_LSE:
      if (g2) go(route_stage1_mma_kernel<D, NT, true, PISA_SCORE_LSE>);
      else go(route_stage1_mma_kernel<D, NT, false, PISA_SCORE_LSE>);
      break;
    case PISA_SCORE_MEAN:
      if (g2) go(route_stage1_mma_kernel<D, NT, true, PISA_SCORE_MEAN>);
      else go(route_stage1_mma_kernel<D, NT, false, PISA_SCORE_MEAN>);
      break;
    default:
      if (g2) go(route_stage1_mma_kernel<D, NT, true, PISA_SCORE_MEAN_VAR>);
      else go(route_stage1_mma_kernel<D, NT, false, PISA_SCORE_MEAN_VAR>);
      break;
  }
  return check_launch("route_stage1_mma");
}

bool route_stage1_mma_supported(const Geometry& g, int dtype) {
  return dtype == PISA_BF16 && (g.d == 64 || g.d == 128) && g.L >= 2 &&
         g.G <= 16;
}

int launch_route_stage1_mma(const Geometry& g, const void* q, const void* pyramid, int32_t* par, float* margin,
                            cudaStream_t s) {
  // the 32-byte loads of the summaries: rows are d*2 >= 128 bytes and the levels start on 256-byte
  // boundaries, so the buffer's own alignment decides
  if ((reinterpret_cast<uintptr_t>(pyramid) & 31u) != 0) return PISA_ERR_INVALID_ARG;
  const bool wide = g.G > 8;
  if (g.d == 128) return wide ? launch_dn<128, 2>(g, q, pyramid, par, margin, s) : launch_dn<128, 1>(g, q, pyramid, par, margin, s);
  if (g.d == 64) return wide ? launch_dn<64, 2>(g, q, pyramid, par, margin, s) : launch_dn<64, 1>(g, q, pyramid, par, margin, s);
  return PISA_ERR_UNSUPPORTED;
}

}  // namespace pisa
