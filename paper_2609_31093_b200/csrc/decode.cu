// Decoding step (Sec. 3.3 "Decoding", App. B "Decode cache"): one new token per sequence, one launch.
//
// A thread-block cluster of eight CTAs (four or two once the batch alone fills the GPU, so that every
// cluster is resident at once) serves one (batch, KV head):
//   1. every CTA walks the intermediate levels L..2 redundantly (identical arithmetic, identical
//      result; the summaries are a few KB): eight warps score eight candidates each per round on
//      m16n8k16 fragments, warp 0 applies Select_K and expands;
//   2. the leaf candidates (at most g*K blocks of C raw keys, the only large read of the selection) are
//      spread over the cluster's warps, one block per warp and round; scores meet in global scratch;
//   3. after a cluster barrier every CTA applies the final Select_K to the same scores;
//   4. attention over the selected blocks: two warps per block (halves of its keys), scores on the
//      same fragments, online softmax, P*V on the FMA pipe; partial (max, sum, output) are merged
//      first inside a CTA through shared memory, then across the cluster through global scratch;
//   5. while the first CTA does the last merge, the last CTA refreshes the cached pyramid along the new
//      token's path: the current leaf's mean over the keys it holds so far, then each ancestor from its
//      stored children (nothing in the same step reads these nodes: the path is forced, never scored).
// Cluster barriers are hardware barriers among co-scheduled CTAs: there is no software spin anywhere.
// Decoding is bound by the key/value bytes it must read (about (g*K + 2*K)*C*d*2 bytes per KV head),
// not by arithmetic, which is why nothing here is a CTA-wide tensor-core tile.
#include <math_constants.h>

#include "mma_frag.cuh"
#include "pisa_common.cuh"

namespace pisa {

using namespace frag;

namespace {

constexpr int kCluMax = 16;             // CTAs per cluster, at most (scratch is laid out for this many)
constexpr int kDecWarps = 8;
constexpr int kDecThreads = kDecWarps * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct DecArgs {
  int pos;                              // position of the new token
  const __nv_bfloat16* q;               // [B, Hq, d]
  const __nv_bfloat16* k;               // caches [B, Ncap, Hkv, d] (strides from the geometry)
  const __nv_bfloat16* v;
  __nv_bfloat16* pyr;                   // cached pyramid, capacity layout
  int32_t* idx;                         // [B, Hkv, K]
  __nv_bfloat16* out;                   // [B, Hq, d]
  float* lse;                           // [B, Hq]
  float* ws_u;                          // [B*Hkv][kMaxCand] leaf scores
  float* ws_part;                       // [B*Hkv][kCluMax][G*d + 2*G] attention partials
};

__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// One logit into a candidate's running score state (Sec. 4.3).  LSE score: (m, acc) = running max and sum
// of exponentials.  Moment scores: m = the shift (the candidate's first logit, set by the caller), acc and
// sq = first and second moments about it.
__device__ __forceinline__ void score_add(int mode, float& m, float& acc, float& sq, float z) {
  if (mode == PISA_SCORE_LSE) lse_add(m, acc, z);
  else { const float dl = z - m; acc += dl; sq += dl * dl; }
}
__device__ __forceinline__ float score_finish(int mode, float m, float acc, float sq, int n) {
  if (mode == PISA_SCORE_LSE) return m + __logf(acc);
  const float mu = acc / (float)n;
  return m + mu + ((mode == PISA_SCORE_MEAN_VAR) ? 0.5f * fmaxf(sq / (float)n - mu * mu, 0.f) : 0.f);
}

// The new token's path in the cached pyramid, by one whole CTA.  Nothing in the same step reads these
// nodes (the path is forced, never scored), so this runs off the critical path, after the CTA's share
// of the attention.  The current leaf's mean takes every loaded key in one round (eight warps, sixteen
// keys each at most per round, a lane owning d/32 columns); the ancestors need one sibling load per
// level and child, all issued before the dependent chain of means starts.
__device__ void refresh_path(const Geometry& geo, const DecArgs& a, int b, int h, float* scratch /* [8][128] */) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = geo.d, dv = d / 32;
  const int c = a.pos / geo.C, t0 = c * geo.C, cnt = a.pos - t0 + 1;
  const __nv_bfloat16* kb = a.k + (long long)b * geo.ks[0] + (long long)h * geo.ks[2] + lane * dv;
  float part[4] = {0.f, 0.f, 0.f, 0.f};
  for (int r0 = warp; r0 < cnt; r0 += kDecWarps * 4) {
    uint2 raw[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = r0 + u * kDecWarps;
      raw[u] = make_uint2(0u, 0u);
      if (r < cnt) {
        const __nv_bfloat16* src = kb + (long long)(t0 + r) * geo.ks[1];
        if (dv == 4) raw[u] = *reinterpret_cast<const uint2*>(src);
        else raw[u].x = *reinterpret_cast<const uint32_t*>(src);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      part[0] += __uint_as_float(raw[u].x << 16);
      part[1] += __uint_as_float(raw[u].x & 0xFFFF0000u);
      part[2] += __uint_as_float(raw[u].y << 16);
      part[3] += __uint_as_float(raw[u].y & 0xFFFF0000u);
    }
  }
  for (int j = 0; j < dv; ++j) scratch[warp * 128 + lane * dv + j] = part[j];
  __syncthreads();
  const int dd = tid;
  if (dd >= d) return;
  float s = 0.f;
  for (int w = 0; w < kDecWarps; ++w) s += scratch[w * 128 + dd];
  const long long bh = (long long)b * geo.Hkv + h;
  // siblings of the path at every level (stored values of completed nodes), all loads first
  float sib[kMaxLevels];
  int nch[kMaxLevels];
  int below = c;
  for (int l = 2; l <= geo.L; ++l) {
    const int node = below / geo.g;
    const int lo = node * geo.g, hi = below;                // valid children: lo .. the path's node
    const __nv_bfloat16* bl = a.pyr + geo.level_off[l - 1] + bh * geo.M[l - 1] * geo.d;
    float acc = 0.f;
    for (int r = lo; r < hi; ++r) acc += __bfloat162float(bl[(long long)r * geo.d + dd]);
    sib[l] = acc;
    nch[l] = hi - lo + 1;
    below = node;
  }
  __nv_bfloat16 cur = __float2bfloat16_rn(s / (float)cnt);
  a.pyr[geo.level_off[1] + (bh * geo.M[1] + c) * geo.d + dd] = cur;
  below = c;
  for (int l = 2; l <= geo.L; ++l) {
    const int node = below / geo.g;
    cur = __float2bfloat16_rn((sib[l] + __bfloat162float(cur)) / (float)nch[l]);
    a.pyr[geo.level_off[l] + (bh * geo.M[l] + node) * geo.d + dd] = cur;
    below = node;
  }
}

// MINB = 1: all registers to one CTA per SM (lowest latency, small batches); MINB = 2: two CTAs per SM so
// that the latency-bound phases of different clusters overlap once the grid exceeds the SM count.
// CLU: CTAs per cluster.  MOM: false = LSE score (the state of the other scores folds away), true = the
// mean / mean + variance scores.
template <int D, int NT, int MINB, int CLU, bool MOM>
__global__ void __cluster_dims__(CLU, 1, 1) __launch_bounds__(kDecThreads, MINB)
decode_step_kernel(Geometry geo, DecArgs a) {
  extern __shared__ float s_part[];                       // [kDecWarps][G*D + 2*G] attention partials
  __shared__ int s_cand[2][kMaxCand];
  __shared__ __align__(16) float s_u[kMaxCand];
  __shared__ int s_sel[kMaxK];
  __shared__ int s_n, s_nsel;
  __shared__ float s_z[kDecWarps][16][16];                // per warp: logits, then probabilities, [key][head]
  __shared__ float s_alpha[kDecWarps][16];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int rank = blockIdx.x;                            // cluster spans the x dimension
  const int bh = blockIdx.y;
  const int b = bh / geo.Hkv, h = bh % geo.Hkv;
  const int K = geo.K, g = geo.g, G = geo.G, C = geo.C;
  const int mode = MOM ? geo.score_mode : (int)PISA_SCORE_LSE;
  const int pos = a.pos;
  const int c = pos / C;
  const int f1 = (c >= 1) ? c - 1 : 0;

  QFrag<D, NT> qf;
  qf.load(a.q + ((long long)b * geo.Hq + (long long)h * G) * D, D, G, lane);

  // ---------------------------------------------------------------- 1. levels L..2
  // Levels whose live nodes (those that do not start after the query's leaf) number at most K keep
  // everything, so the walk starts at the highest level that has more, with every child of the live
  // nodes of the level above as its candidates.
  int l_top = 1;                                            // level of the first candidate list
  for (int l = geo.L; l >= 2; --l) {
    const unsigned sp = (unsigned)min(geo.span[l], (long long)0x7fffffff);
    if ((int)((unsigned)c / sp) + 1 > K) { l_top = l; break; }
  }
  {
    int n_init = 1;                                         // the root, when the walk starts there
    if (l_top < geo.L) {
      const unsigned sp = (unsigned)min(geo.span[l_top + 1], (long long)0x7fffffff);
      n_init = min(((int)((unsigned)c / sp) + 1) * g, geo.M[l_top]);
    }
    for (int s = tid; s < n_init; s += kDecThreads) s_cand[0][s] = s;
    if (tid == 0) s_n = n_init;
  }
  __syncthreads();
  int cur = 0;
  for (int l = l_top; l >= 2; --l) {
    const int* cand = s_cand[cur];
    int* next = s_cand[cur ^ 1];
    const int n = s_n;
    // leaves under a level-l node; c < 2^31, so a span beyond that just means ancestor 0 (32-bit division)
    const unsigned span = (unsigned)min(geo.span[l], (long long)0x7fffffff);
    const int anc_c = (int)((unsigned)c / span);
    const int f1l = (c >= 1) ? (int)((unsigned)(c - 1) / span) : 0;
    int nV = 0;                                           // eligible candidates form a prefix
    for (int s0 = 0; s0 < n; s0 += 32) {
      const int s = s0 + lane;
      nV += __popc(__ballot_sync(0xffffffffu, (s < n) && (cand[s] <= anc_c)));
    }
    const bool prune = nV > K;
    if (prune) {
      const int Mb = geo.M[l - 1];
      const __nv_bfloat16* below = a.pyr + geo.level_off[l - 1] + (long long)bh * Mb * D;
      for (int k0 = warp * 8; k0 < nV; k0 += kDecWarps * 8) {
        const int kap = k0 + gid;
        const bool has = kap < nV;
        const int node = has ? cand[kap] : 0;
        float m[NT][2], ssum[NT][2], sq[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          m[nt][0] = m[nt][1] = -CUDART_INF_F; ssum[nt][0] = ssum[nt][1] = 0.f; sq[nt][0] = sq[nt][1] = 0.f;
        }
        const int nch = has ? min(g, Mb - node * g) : 1;        // valid children of the candidate
        for (int r0 = 0; r0 < g; r0 += 2) {
          const int ch_lo = node * g + r0, ch_hi = ch_lo + 1;
          const bool ok_lo = has && ch_lo < Mb, ok_hi = has && (r0 + 1 < g) && ch_hi < Mb;
          float z[NT][4];
          rows2_dot<D, NT>(qf, ok_lo ? below + (long long)ch_lo * D : nullptr,
                           ok_hi ? below + (long long)ch_hi * D : nullptr, lane, z);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int jh = 0; jh < 2; ++jh) {
              if (mode != PISA_SCORE_LSE && r0 == 0) m[nt][jh] = z[nt][jh] * geo.scale;   // shift: the first child
              if (ok_lo) score_add(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], z[nt][jh] * geo.scale);
              if (ok_hi) score_add(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], z[nt][2 + jh] * geo.scale);
            }
        }
        float usum = 0.f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int jh = 0; jh < 2; ++jh)
            if (nt * 8 + 2 * tig + jh < G && has) usum += score_finish(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], nch);
        usum += __shfl_xor_sync(0xffffffffu, usum, 1);
        usum += __shfl_xor_sync(0xffffffffu, usum, 2);
        if (has && tig == 0) s_u[kap] = (node == 0 || node == f1l || node == anc_c) ? forced_score(kap) : usum;
      }
      if (warp == 0 && lane < 4 && nV + lane < kMaxCand) s_u[nV + lane] = -CUDART_INF_F;
    }
    __syncthreads();
    if (warp == 0) {
      int rank_s[kMaxCand / 32];
      const bool sorted = prune && nV <= 64;
      bool keep_s[2] = {false, false};
      if (sorted) {
        float ca, cb;
        warp_select_sorted64((lane < nV) ? s_u[lane] : -CUDART_INF_F, (lane + 32 < nV) ? s_u[lane + 32] : -CUDART_INF_F,
                             K, lane, keep_s[0], keep_s[1], ca, cb);
      } else if (prune) {
        warp_select_ranks(s_u, nV, lane, rank_s);
      }
      int base = 0;
#pragma unroll
      for (int ch = 0; ch < kMaxCand / 32; ++ch) {
        const int s = ch * 32 + lane;
        bool keep = s < nV;
        if (sorted) keep = keep && (ch < 2) && keep_s[ch & 1];
        else if (prune && ch * 32 < nV) keep = keep && (rank_s[ch] < K);
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        const int p = base + __popc(bal & ((1u << lane) - 1u));
        if (keep) {
          const int i = cand[s];
          for (int r = 0; r < g; ++r) next[p * g + r] = i * g + r;
        }
        base += __popc(bal);
      }
      if (lane == 0) s_n = base * g;
    }
    __syncthreads();
    cur ^= 1;
  }

  // ---------------------------------------------------------------- 2. leaf candidates
  const int* cand1 = s_cand[cur];
  const int n1 = s_n;
  int nV1 = 0;
  for (int s0 = 0; s0 < n1; s0 += 32) {
    const int s = s0 + lane;
    nV1 += __popc(__ballot_sync(0xffffffffu, (s < n1) && (cand1[s] <= c)));
  }
  const bool prune1 = nV1 > K;
  float* wu = a.ws_u + (long long)bh * kMaxCand;
  const __nv_bfloat16* kbh = a.k + (long long)b * geo.ks[0] + (long long)h * geo.ks[2];
  const __nv_bfloat16* vbh = a.v + (long long)b * geo.vs[0] + (long long)h * geo.vs[2];
  if (prune1) {
    for (int ci = rank * kDecWarps + warp; ci < nV1; ci += CLU * kDecWarps) {
      const int leaf = cand1[ci];
      if (leaf == 0 || leaf == f1 || leaf == c) continue;        // forced: never scored
      // a scored leaf lies strictly before the current one: all C keys exist and are visible
      float m[NT][2], ssum[NT][2], sq[NT][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        m[nt][0] = m[nt][1] = -CUDART_INF_F; ssum[nt][0] = ssum[nt][1] = 0.f; sq[nt][0] = sq[nt][1] = 0.f;
      }
      for (int kt = 0; kt < C; kt += 32) {                       // two key tiles in flight per round
        const long long t_lo = (long long)leaf * C + kt + gid;
        RowPair<D> r0, r1;
        r0.load(kbh + t_lo * geo.ks[1], kbh + (t_lo + 8) * geo.ks[1], lane);
        r1.load(kbh + (t_lo + 16) * geo.ks[1], kbh + (t_lo + 24) * geo.ks[1], lane);
        float z[NT][4];
        rows2_dot<D, NT>(qf, r0, z);
        if (mode != PISA_SCORE_LSE && kt == 0) {
          // moment scores: every lane shifts by the logit of the block's first key, which the lanes with
          // gid = 0 (lane = tig) hold for their two heads
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int jh = 0; jh < 2; ++jh) m[nt][jh] = __shfl_sync(0xffffffffu, z[nt][jh] * geo.scale, tig);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int jh = 0; jh < 2; ++jh) {
            score_add(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], z[nt][jh] * geo.scale);
            score_add(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], z[nt][2 + jh] * geo.scale);
          }
        rows2_dot<D, NT>(qf, r1, z);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int jh = 0; jh < 2; ++jh) {
            score_add(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], z[nt][jh] * geo.scale);
            score_add(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], z[nt][2 + jh] * geo.scale);
          }
      }
      float usum = 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int jh = 0; jh < 2; ++jh) {
          // the eight lanes that share tig hold the other keys of the same heads
#pragma unroll
          for (int o = 4; o < 32; o <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m[nt][jh], o);
            const float s2 = __shfl_xor_sync(0xffffffffu, ssum[nt][jh], o);
            const float q2 = __shfl_xor_sync(0xffffffffu, sq[nt][jh], o);
            if (mode == PISA_SCORE_LSE) lse_merge(m[nt][jh], ssum[nt][jh], m2, s2);
            else { ssum[nt][jh] += s2; sq[nt][jh] += q2; }         // same shift in every lane
          }
          if (nt * 8 + 2 * tig + jh < G) usum += score_finish(mode, m[nt][jh], ssum[nt][jh], sq[nt][jh], C);
        }
      usum += __shfl_xor_sync(0xffffffffu, usum, 1);
      usum += __shfl_xor_sync(0xffffffffu, usum, 2);
      if (lane == 0) wu[ci] = usum;
    }
  }
  cluster_barrier();

  // ---------------------------------------------------------------- 3. final Select_K (every CTA)
  if (warp == 0) {
    for (int s = lane; s < kMaxCand; s += 32) {
      float sc = -CUDART_INF_F;
      if (s < nV1 && prune1) {
        const int leaf = cand1[s];
        sc = (leaf == 0 || leaf == f1 || leaf == c) ? forced_score(s) : __ldcg(wu + s);
      }
      s_u[s] = sc;
    }
    __syncwarp();
    int rank_s[kMaxCand / 32];
    const bool sorted = prune1 && nV1 <= 64;
    bool keep_s[2] = {false, false};
    if (sorted) {
      float ca, cb;
      warp_select_sorted64(s_u[lane], s_u[lane + 32], K, lane, keep_s[0], keep_s[1], ca, cb);   // -inf beyond nV1
    } else if (prune1) {
      warp_select_ranks(s_u, nV1, lane, rank_s);
    }
    int base = 0;
#pragma unroll
    for (int ch = 0; ch < kMaxCand / 32; ++ch) {
      const int s = ch * 32 + lane;
      bool keep = s < nV1;
      if (sorted) keep = keep && (ch < 2) && keep_s[ch & 1];
      else if (prune1 && ch * 32 < nV1) keep = keep && (rank_s[ch] < K);
      const unsigned bal = __ballot_sync(0xffffffffu, keep);
      const int p = base + __popc(bal & ((1u << lane) - 1u));
      if (keep) s_sel[p] = cand1[s];
      base += __popc(bal);
    }
    if (lane == 0) s_nsel = base;
    __syncwarp();
    if (rank == 0)
      for (int s = lane; s < K; s += 32) a.idx[(long long)bh * K + s] = (s < base) ? s_sel[s] : -1;
  }
  __syncthreads();

  // ---------------------------------------------------------------- 4. attention
  // warp gw of the cluster takes the half blocks gw, gw + (warps in the cluster), ...: half block sh is
  // keys [half*C/2, (half+1)*C/2) of selected block sh/2; the online softmax state runs across them
  const int gw = rank * kDecWarps + warp;
  const int nsel = s_nsel;
  constexpr int DV = D / 32;                               // output columns per lane
  const int W = G * D + 2 * G;                             // floats per partial: o[G][D], m[G], l[G]
  float o_acc[16][DV];
#pragma unroll
  for (int hh = 0; hh < 16; ++hh)
#pragma unroll
    for (int j = 0; j < DV; ++j) o_acc[hh][j] = 0.f;
  float m_run = -CUDART_INF_F, l_run = 0.f;                // lanes 0..G-1: running max (base 2) / sum of head `lane`
  const float sl2 = geo.scale * kLog2e;
  // clusters of sixteen (opt-in size) split a block in four, so that all 128 warps have a part
  constexpr int SUB = (CLU == 16) ? 4 : 2;
  for (int sh = gw; sh < SUB * nsel; sh += CLU * kDecWarps) {
    const int slot = sh / SUB, half = sh % SUB;
    const int leaf = s_sel[slot];
    const int key0 = leaf * C + half * (C / SUB);
    for (int kt = 0; kt < C / SUB; kt += 16) {
      const int t_lo = key0 + kt + gid, t_hi = t_lo + 8;
      if (key0 + kt > pos) break;                          // the rest of the block lies in the future
      RowPair<D> kr;
      kr.load((t_lo <= pos) ? kbh + (long long)t_lo * geo.ks[1] : nullptr,
              (t_hi <= pos) ? kbh + (long long)t_hi * geo.ks[1] : nullptr, lane);
      // the tile's sixteen value rows (this lane's DV columns of each), in flight during the softmax
      uint32_t vraw[16][DV / 2];
#pragma unroll
      for (int kk = 0; kk < 16; ++kk) {
        const int t = key0 + kt + kk;
#pragma unroll
        for (int j = 0; j < DV / 2; ++j) vraw[kk][j] = 0u;
        if (t <= pos) {                                    // one 8-byte (d = 128) or 4-byte (d = 64) load per row
          const __nv_bfloat16* vr = vbh + (long long)t * geo.vs[1] + lane * DV;
          if (DV == 4) {
            const uint2 x = *reinterpret_cast<const uint2*>(vr);
            vraw[kk][0] = x.x; vraw[kk][DV / 2 - 1] = x.y;
          } else {
            vraw[kk][0] = *reinterpret_cast<const uint32_t*>(vr);
          }
        }
      }
      float z[NT][4];
      rows2_dot<D, NT>(qf, kr, z);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int jh = 0; jh < 2; ++jh) {
          const int head = nt * 8 + 2 * tig + jh;
          if (head < G) {
            s_z[warp][gid][head] = (t_lo <= pos) ? z[nt][jh] * sl2 : -CUDART_INF_F;
            s_z[warp][gid + 8][head] = (t_hi <= pos) ? z[nt][2 + jh] * sl2 : -CUDART_INF_F;
          }
        }
      __syncwarp();
      if (lane < G) {                                      // one lane per head: online softmax over the 16 keys
        float tm = -CUDART_INF_F;
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) tm = fmaxf(tm, s_z[warp][kk][lane]);
        const float mn = fmaxf(m_run, tm);                 // finite: the tile's first key is visible
        const float alpha = ex2f(m_run - mn);
        float ps = 0.f;
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
          const float p = ex2f(s_z[warp][kk][lane] - mn);
          s_z[warp][kk][lane] = p;
          ps += p;
        }
        l_run = l_run * alpha + ps;
        m_run = mn;
        s_alpha[warp][lane] = alpha;
      }
      __syncwarp();
#pragma unroll
      for (int hh = 0; hh < 16; ++hh)
        if (hh < G) {
          const float al = s_alpha[warp][hh];
#pragma unroll
          for (int j = 0; j < DV; ++j) o_acc[hh][j] *= al;
        }
#pragma unroll
      for (int kk = 0; kk < 16; ++kk) {                    // rows after pos hold zeros and weight 0
        float vv[DV];
#pragma unroll
        for (int j = 0; j < DV / 2; ++j) {
          vv[2 * j] = __uint_as_float(vraw[kk][j] << 16);
          vv[2 * j + 1] = __uint_as_float(vraw[kk][j] & 0xFFFF0000u);
        }
#pragma unroll
        for (int hh = 0; hh < 16; ++hh)
          if (hh < G) {
            const float p = s_z[warp][kk][hh];
#pragma unroll
            for (int j = 0; j < DV; ++j) o_acc[hh][j] = fmaf(p, vv[j], o_acc[hh][j]);
          }
      }
      __syncwarp();
    }
  }
  // warp partial -> shared memory: o[G][D], m[G], l[G]
  float* mine = s_part + warp * W;
#pragma unroll
  for (int hh = 0; hh < 16; ++hh)
    if (hh < G)
#pragma unroll
      for (int j = 0; j < DV; ++j) mine[hh * D + lane * DV + j] = o_acc[hh][j];
  if (lane < G) { mine[G * D + lane] = m_run; mine[G * D + G + lane] = l_run; }
  __syncthreads();
  // CTA partial: merge the eight warps
  float* cta_out = a.ws_part + ((long long)bh * kCluMax + rank) * W;
  for (int e = tid; e < G * D + G; e += kDecThreads) {
    const bool is_o = e < G * D;
    const int hh = is_o ? e / D : e - G * D;
    float M = -CUDART_INF_F;
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, s_part[w * W + G * D + hh]);
    float acc = 0.f;
    for (int w = 0; w < kDecWarps; ++w) {
      const float mw = s_part[w * W + G * D + hh];
      if (mw > -CUDART_INF_F) acc += (is_o ? s_part[w * W + e] : s_part[w * W + G * D + G + hh]) * ex2f(mw - M);
    }
    if (is_o) cta_out[e] = acc;
    else { cta_out[G * D + hh] = M; cta_out[G * D + G + hh] = acc; }
  }
  cluster_barrier();
  // the last CTA refreshes the cached pyramid while the first one merges the partials
  if (rank == CLU - 1) refresh_path(geo, a, b, h, &s_z[0][0][0]);
  // the first CTA merges the cluster's partials and writes the token's output
  if (rank == 0) {
    const float* parts = a.ws_part + (long long)bh * kCluMax * W;
    for (int e = tid; e < G * D; e += kDecThreads) {
      const int hh = e / D;
      float M = -CUDART_INF_F;
      for (int r = 0; r < CLU; ++r) M = fmaxf(M, __ldcg(parts + r * W + G * D + hh));
      float acc = 0.f, den = 0.f;
      for (int r = 0; r < CLU; ++r) {
        const float mr = __ldcg(parts + r * W + G * D + hh);
        if (mr > -CUDART_INF_F) {
          const float f = ex2f(mr - M);
          acc += __ldcg(parts + r * W + e) * f;
          den += __ldcg(parts + r * W + G * D + G + hh) * f;
        }
      }
      a.out[((long long)b * geo.Hq + (long long)h * G + hh) * D + (e - hh * D)] = __float2bfloat16_rn(acc / den);
      if (e - hh * D == 0) a.lse[(long long)b * geo.Hq + (long long)h * G + hh] = (M + log2f(den)) * kLn2;
    }
  }
}

template <int D, int NT, int MINB, int CLU, bool MOM>
int launch_dnbm(const Geometry& g, const DecArgs& a, cudaStream_t s) {
  const size_t smem = (size_t)kDecWarps * (g.G * D + 2 * g.G) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(decode_step_kernel<D, NT, MINB, CLU, MOM>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess && CLU > 8)
    e = cudaFuncSetAttribute(decode_step_kernel<D, NT, MINB, CLU, MOM>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  if (e != cudaSuccess) { record_cuda_error("decode_step attr", e); return PISA_ERR_CUDA; }
  decode_step_kernel<D, NT, MINB, CLU, MOM><<<dim3(CLU, (unsigned)(g.B * g.Hkv)), kDecThreads, smem, s>>>(g, a);
  return check_launch("decode_step");
}
template <int D, int NT, int MINB, int CLU>
int launch_dnb(const Geometry& g, const DecArgs& a, cudaStream_t s) {
  return (g.score_mode == PISA_SCORE_LSE) ? launch_dnbm<D, NT, MINB, CLU, false>(g, a, s)
                                          : launch_dnbm<D, NT, MINB, CLU, true>(g, a, s);
}
// How many clusters of this instantiation the GPU holds at once (clusters are placed inside one GPC, so
// this is less than SMs * MINB / CLU); asked of the driver once per instantiation.
template <int D, int NT, int MINB, int CLU>
int max_resident_clusters(const Geometry& g) {
  static int cached = -1;
  if (cached >= 0) return cached;
  const size_t smem = (size_t)kDecWarps * (g.G * D + 2 * g.G) * sizeof(float);
  auto kern = decode_step_kernel<D, NT, MINB, CLU, false>;
  cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (CLU > 8 && cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
    cudaGetLastError();
    cached = 0;
    return 0;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(CLU, 1024);
  cfg.blockDim = dim3(kDecThreads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = CLU; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
  cached = n;
  return n;
}

// The widest cluster whose clusters are all resident at once at one CTA per SM (all registers); beyond
// that clusters of two at two CTAs per SM, in waves once even those do not fit.  Measured at the headline shape, 128K
// context: batch 3 / 4 / 6 / 8 take 82 / 86 / 127 / 130 us this way against 98 / 103 / 143 / 152 us with
// clusters of eight at two CTAs per SM whenever those fit.
template <int D, int NT>
int launch_dn(const Geometry& g, const DecArgs& a, cudaStream_t s) {
  const long long units = (long long)g.B * g.Hkv;
  // sixteen CTAs (a quarter block of at least one 16-key tile per warp) for very few units: measured at
  // 128K context, 4 units 48.7 -> 45.4 us and 2 units 49.3 -> 47.3 us, but 8 units 55.6 -> 57.4 us
  if (g.C >= 64 && units <= 4 && units <= max_resident_clusters<D, NT, 1, 16>(g))
    return launch_dnb<D, NT, 1, 16>(g, a, s);
  if (units <= max_resident_clusters<D, NT, 1, 8>(g)) return launch_dnb<D, NT, 1, 8>(g, a, s);
  if (units <= max_resident_clusters<D, NT, 1, 4>(g)) return launch_dnb<D, NT, 1, 4>(g, a, s);
  if (units <= max_resident_clusters<D, NT, 1, 2>(g)) return launch_dnb<D, NT, 1, 2>(g, a, s);
  // two CTAs per SM: only the narrowest width holds more units than the options above
  return launch_dnb<D, NT, 2, 2>(g, a, s);
}

}  // namespace

bool decode_supported(const Geometry& g, int dtype) {
  return dtype == PISA_BF16 && (g.d == 64 || g.d == 128) && g.G <= 16 &&
         (g.C == 64 || g.C == 128 || g.C == 32) && (long long)g.B * g.Hkv <= 65535;
}

size_t decode_workspace_bytes(const Geometry& g) {
  const size_t bh = (size_t)g.B * g.Hkv;
  return align_up(bh * kMaxCand * sizeof(float), 256) +
         align_up(bh * kCluMax * (size_t)(g.G * g.d + 2 * g.G) * sizeof(float), 256);
}

int launch_decode_step(const Geometry& g, int pos, const void* q, const void* k, const void* v, void* pyramid,
                       int32_t* idx, void* out, float* lse, void* ws, cudaStream_t s) {
  DecArgs a;
  a.pos = pos;
  a.q = (const __nv_bfloat16*)q; a.k = (const __nv_bfloat16*)k; a.v = (const __nv_bfloat16*)v;
  a.pyr = (__nv_bfloat16*)pyramid; a.idx = idx; a.out = (__nv_bfloat16*)out; a.lse = lse;
  a.ws_u = (float*)ws;
  a.ws_part = (float*)((char*)ws + align_up((size_t)g.B * g.Hkv * kMaxCand * sizeof(float), 256));
  const bool wide = g.G > 8;
  if (g.d == 128) return wide ? launch_dn<128, 2>(g, a, s) : launch_dn<128, 1>(g, a, s);
  if (g.d == 64) return wide ? launch_dn<64, 2>(g, a, s) : launch_dn<64, 1>(g, a, s);
  return PISA_ERR_UNSUPPORTED;
}

}  // namespace pisa
