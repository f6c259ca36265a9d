// Flat block selection (Sec. 3.1, App. C) on the tensor cores: the O(N^2/C) reference point.
//
// Every eligible leaf i <= c of a query is scored with s = q . kbar_i * scale (kbar = level-1 summary),
// soft-maxed over the eligible leaves within each query head, summed over the G heads of the group, and
// the forced leaves {0, c-1, c} plus the best K - 3 of the rest are kept.  This is a dense contraction
// [queries x d] . [d x leaves], so it runs query-major on tcgen05:
//
//   work item  = (b, KV head, 2 * (128 / G) consecutive tokens) = two 128-row A tiles (row = token*G + head,
//                contiguous in q: one 4-D TMA tile load per tile and 64-wide K slab);
//   B operand  = 128 consecutive level-1 summaries of the head (2-slab TMA tile loads into a ring), shared by
//                the item's two UMMAs per chunk, which halves the L2 traffic per flop;
//   two passes over the chunks 0 .. ceil((c_max + 1) / 128) - 1: pass 1 builds each row's softmax maximum
//                and denominator online, pass 2 recomputes the logits, normalises, sums the G heads of a
//                token with shuffles and streams the scores through a per-token Top-(K - 3) list in shared
//                memory (replace-the-minimum; equal scores keep the smaller leaf id);
//   roles      = warp 0 TMA producer, warp 1 UMMA issuer, warps 2-9 epilogue (four per A tile, one per
//                TMEM lane quarter); accumulators [2 tiles][128 columns], double buffered = 512 TMEM columns.
//
// No score matrix is ever written; all TMA loads read this GPU's own memory, none is multicast.  Every
// wait is time-bounded and reports PISA_ERR_TIMEOUT through the status word.
#include <math_constants.h>

#include "pisa_common.cuh"
#include "tc_utils.cuh"
#include "tma_map.cuh"

namespace pisa {

using namespace tc;

namespace {

constexpr int kFlatThreads = 320;        // producer warp, UMMA warp, 8 epilogue warps
constexpr int kChunk = 128;              // leaves per chunk (UMMA N)
constexpr int kListStride = 33;          // floats / ints per token list (32 slots + 1 pad: conflict-free)
constexpr float kLog2eF = 1.4426950408889634f;

struct FlatArgs {
  int32_t* idx;            // [B, Hkv, N, K]
  int32_t* status;
  int n_pairs;             // tile pairs per (b, KV head)
  int n_items;             // B * Hkv * n_pairs
  int stages;              // B-operand ring depth
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// item -> (bh, pair): late token ranges (the expensive ones) come first
__device__ __forceinline__ void flat_item(const FlatArgs& a, int BH, int item, int& bh, int& pair) {
  bh = item % BH;
  pair = a.n_pairs - 1 - item / BH;
}
// chunks an item walks per pass: up to the last row's current leaf; none if no row has more than K eligible
__device__ __forceinline__ int flat_chunks(const Geometry& geo, int pair, int tok_per_item) {
  const int t_last = min(geo.N, (pair + 1) * tok_per_item) - 1;
  const int c_max = t_last / geo.C;
  return (c_max + 1 <= geo.K) ? 0 : (c_max + 1 + kChunk - 1) / kChunk;
}

}  // namespace

// One pass-1 update of a row's online (maximum, denominator), base 2, over the first nv of 32 logits.
__device__ __forceinline__ void flat_pass1(const uint32_t (&x)[32], int nv, float sl2, float& m, float& l) {
  float cm = -CUDART_INF_F;
#pragma unroll
  for (int j = 0; j < 32; ++j)
    if (j < nv) cm = fmaxf(cm, __uint_as_float(x[j]));
  const float mn = fmaxf(m, cm * sl2);
  float acc4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int j = 0; j < 32; ++j)
    if (j < nv) acc4[j & 3] += ex2f(fmaf(__uint_as_float(x[j]), sl2, -mn));
  l = l * ex2f(m - mn) + ((acc4[0] + acc4[1]) + (acc4[2] + acc4[3]));
  m = mn;
}

// Pass 2 on one 32-column group: normalised scores of this row, summed over the token's G = 2^LG heads by a
// reduce-scatter among its lanes (lane `head` ends up owning 32 / G consecutive columns, starting at
// col_off), then the owned scores that beat the token's current threshold go through its Top-K' list,
// the token's lanes taking turns.  list_val / list_idx: the token's list; slot 32 holds the threshold /
// (count | position of the minimum << 8).
template <int LG>
__device__ __forceinline__ void flat_pass2(const uint32_t (&x)[32], int nv, float sl2, float m2, int head, int leaf_first,
                                           int leaf_last_cand, bool scored, int Kp, float* list_val, int* list_idx) {
  constexpr int G = 1 << LG, OWN = 32 >> LG;
  float v[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = (j < nv) ? ex2f(fmaf(__uint_as_float(x[j]), sl2, -m2)) : 0.f;
#pragma unroll
  for (int s = 0; s < LG; ++s) {
    const int half = 16 >> s;
    const bool up = ((head >> s) & 1) != 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (j < half) {
        const float keep = up ? v[j + half] : v[j];
        const float send = up ? v[j] : v[j + half];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 1 << s);
      }
    }
  }
  // candidates among the owned columns: leaves 1 .. c - 2 that beat the threshold as it stands now (it only
  // rises, so this is a superset of what will be inserted)
  unsigned mask = 0;
  if (scored) {
    const int meta = list_idx[32];
    const bool full = (meta & 0xFF) >= Kp;
    const float tau = list_val[32];
#pragma unroll
    for (int j = 0; j < OWN; ++j) {
      const int leaf = leaf_first + j;
      if (leaf >= 1 && leaf <= leaf_last_cand && (!full || v[j] > tau)) mask |= 1u << j;
    }
  }
  if (__all_sync(0xffffffffu, mask == 0)) return;
#pragma unroll 1
  for (int turn = 0; turn < G; ++turn) {
    if (head == turn && mask != 0) {
      const int meta = list_idx[32];
      int cnt = meta & 0xFF, pos = meta >> 8;
      float tau = list_val[32];
      while (mask != 0) {
        const int jj = __ffs(mask) - 1;
        mask &= mask - 1;
        float u = v[0];
#pragma unroll
        for (int j = 1; j < OWN; ++j) u = (j == jj) ? v[j] : u;
        if (cnt < Kp || u > tau) {
          const int at = (cnt < Kp) ? cnt : pos;
          list_val[at] = u;
          list_idx[at] = leaf_first + jj;
          if (cnt < Kp) ++cnt;
          if (cnt == Kp) {                       // the list is full: find what to replace next
            tau = CUDART_INF_F;
            int ileaf = -1;
            for (int e = 0; e < Kp; ++e) {
              const float ve = list_val[e];
              const int ie = list_idx[e];
              if (ve < tau || (ve == tau && ie > ileaf)) { tau = ve; pos = e; ileaf = ie; }
            }
          }
        }
      }
      list_idx[32] = cnt | (pos << 8);
      list_val[32] = tau;
    }
    __syncwarp();
  }
}

template <int D, int LG>
__global__ void __launch_bounds__(kFlatThreads, 1)
flat_tc_kernel(Geometry geo, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               FlatArgs a) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int KS = D / 64;
  constexpr int TILE = KS * 128 * 128;             // bytes of one 128-row operand tile (A tile or B chunk)
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                              // [2 tiles][TILE]
  uint8_t* sB = smem + 2 * TILE;                   // [stages][TILE]
  float* l_val = reinterpret_cast<float*>(sB + a.stages * TILE);       // [tokens per item][kListStride]
  constexpr int G = 1 << LG, lgG = LG, tpt = 128 >> LG, tok_per_item = 2 * tpt;
  int* l_idx = reinterpret_cast<int*>(l_val + tok_per_item * kListStride);
  __shared__ uint64_t q_full, q_empty, b_full[4], b_empty[4], t_full[2], t_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_fail;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    mbar_init(&q_full, 1); mbar_init(&q_empty, 1);
    for (int i = 0; i < 4; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&t_full[i], 1); mbar_init(&t_empty[i], 8); }
    s_fail = 0;
    mbar_fence_init();
  }
  if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  const int BH = geo.B * geo.Hkv;
  const int K = geo.K, Kp = K - 3;                 // slots for scored leaves

  if (warp == 0) {
    // ------------------------------------------------ TMA producer (one thread)
    if (lane == 0) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      int it = 0, step = 0;                        // items with work, B-ring steps, both counted per CTA
      for (int item = blockIdx.x; item < a.n_items && !s_fail; item += gridDim.x) {
        int bh, pair;
        flat_item(a, BH, item, bh, pair);
        const int nch = flat_chunks(geo, pair, tok_per_item);
        if (nch == 0) continue;
        const int b = bh / geo.Hkv, h = bh % geo.Hkv;
        if (it > 0 && !mbar_wait_bounded(&q_empty, (uint32_t)((it - 1) & 1))) { s_fail = 1; break; }
        mbar_arrive_expect_tx(&q_full, 2u * TILE);
        for (int r = 0; r < 2; ++r)
          for (int ks = 0; ks < KS; ++ks)
            tma_load_4d(smem_u32(sQ + r * TILE + ks * (128 * 128)), &tm_q, &q_full, ks * 64, h * G,
                        pair * tok_per_item + r * tpt, b);
        for (int st = 0; st < 2 * nch; ++st, ++step) {
          const int s = step % a.stages;
          if (step >= a.stages && !mbar_wait_bounded(&b_empty[s], (uint32_t)((step / a.stages - 1) & 1))) { s_fail = 1; break; }
          mbar_arrive_expect_tx(&b_full[s], (uint32_t)TILE);
          for (int ks = 0; ks < KS; ++ks)
            tma_load_3d(smem_u32(sB + s * TILE + ks * (128 * 128)), &tm_k, &b_full[s], ks * 64, (st % nch) * kChunk, bh);
        }
        ++it;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ UMMA issuer (the warp walks the loop, lane 0 issues)
    const uint32_t idesc = make_idesc_bf16(128, kChunk, 0, 0);
    int it = 0, step = 0;
    for (int item = blockIdx.x; item < a.n_items && !s_fail; item += gridDim.x) {
      int bh, pair;
      flat_item(a, BH, item, bh, pair);
      const int nch = flat_chunks(geo, pair, tok_per_item);
      if (nch == 0) continue;
      bool ok = mbar_wait_bounded(&q_full, (uint32_t)(it & 1));
      for (int st = 0; st < 2 * nch && ok; ++st, ++step) {
        const int s = step % a.stages, buf = step & 1;
        ok = mbar_wait_bounded(&b_full[s], (uint32_t)((step / a.stages) & 1));
        if (ok && step >= 2) ok = mbar_wait_bounded(&t_empty[buf], (uint32_t)(((step >> 1) - 1) & 1));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) {
          tcgen05_fence_after_sync();
          const uint32_t b0 = smem_u32(sB + s * TILE);
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const uint32_t a0 = smem_u32(sQ + r * TILE);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint64_t da = make_smem_desc(a0 + (kk >> 2) * (128 * 128) + (kk & 3) * 32, 0, 1024);
              const uint64_t db = make_smem_desc(b0 + (kk >> 2) * (128 * 128) + (kk & 3) * 32, 0, 1024);
              umma_bf16(tmem + (uint32_t)(buf * 256 + r * 128), da, db, idesc, kk > 0);
            }
          }
          umma_commit(&b_empty[s]);
          umma_commit(&t_full[buf]);
          if (st == 2 * nch - 1) umma_commit(&q_empty);
        }
        __syncwarp();
      }
      if (!ok) { s_fail = 1; break; }
      ++it;
    }
  } else {
    // ------------------------------------------------ epilogue: four warps per A tile, one per TMEM lane quarter
    const int r = (warp - 2) >> 2;                   // A tile of this warp
    const int quarter = warp & 3;                    // TMEM lanes quarter*32 .. +31 (fixed by the warp id)
    const int row = quarter * 32 + lane;             // row inside the tile = token * G + head
    const int tl = row >> lgG, head = row & (G - 1);
    const int ti = r * tpt + tl;                     // token inside the item
    const uint32_t t_base = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(r * 128);
    const float sl2 = geo.scale * kLog2eF;
    const int n_own = 32 >> lgG;                     // columns of a 32-column group this lane owns after the head sum
    int col_off = 0;                                 // ... starting at this offset inside the group
    for (int s = 0; s < lgG; ++s) col_off += ((head >> s) & 1) * (16 >> s);
    float* my_val = l_val + ti * kListStride;
    int* my_idx = l_idx + ti * kListStride;
    int step = 0;
    for (int item = blockIdx.x; item < a.n_items && !s_fail; item += gridDim.x) {
      int bh, pair;
      flat_item(a, BH, item, bh, pair);
      const int nch = flat_chunks(geo, pair, tok_per_item);
      const int t = pair * tok_per_item + ti;
      const bool valid = t < geo.N;
      const int c_row = valid ? t / geo.C : -1;
      const bool scored = valid && (c_row + 1 > K);
      float m = -CUDART_INF_F, l = 0.f, m2 = 0.f;
      if (head == 0) my_idx[32] = 0;                 // list meta: count | position of the minimum << 8
      __syncwarp();
      bool ok = true;
      for (int st = 0; st < 2 * nch; ++st, ++step) {
        const int buf = step & 1;
        const int ch = (st < nch) ? st : st - nch;
        if (!mbar_wait_bounded(&t_full[buf], (uint32_t)((step >> 1) & 1))) { ok = false; break; }
        tcgen05_fence_after_sync();
        if (st == nch) m2 = m + log2f(l);            // pass 2: p = 2^(x - m) / l = 2^(x - m2)
        uint32_t ra[32], rb[32];
        tmem_ld_32x32(t_base + (uint32_t)(buf * 256), ra);
#pragma unroll 1
        for (int c0 = 0; c0 < kChunk; c0 += 64) {            // two 32-column groups per round (ra, then rb)
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t (&cur)[32] = hh ? rb : ra;
            uint32_t (&nxt)[32] = hh ? ra : rb;
            const int cc0 = c0 + hh * 32;
            tmem_ld_wait();
            if (cc0 + 32 < kChunk) {
              tmem_ld_32x32(t_base + (uint32_t)(buf * 256 + cc0 + 32), nxt);
            } else {
              tcgen05_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive(&t_empty[buf]);     // the accumulator has been read out
            }
            const int leaf0 = ch * kChunk + cc0;             // leaf of column 0 of this group
            const int nv = scored ? max(0, min(32, c_row + 1 - leaf0)) : 0;   // eligible columns: leaves <= c_row
            if (st < nch) {
              if (nv > 0) flat_pass1(cur, nv, sl2, m, l);
            } else if (!__all_sync(0xffffffffu, nv == 0)) {
              flat_pass2<LG>(cur, nv, sl2, m2, head, leaf0 + col_off, c_row - 2, scored, Kp, my_val, my_idx);
            }
          }
        }
      }
      if (!ok) { s_fail = 1; break; }
      // write the rows of this warp's tokens: forced leaves + the list, ascending, -1 padded
      __syncwarp();
      const int tok0 = r * tpt + ((quarter * 32) >> lgG);
      for (int k2 = 0; k2 < n_own; ++k2) {                   // 32 / G tokens per warp
        const int tk = tok0 + k2;
        const int tt = pair * tok_per_item + tk;
        if (tt >= geo.N) break;
        const int cc = tt / geo.C;
        int mine = 0x7fffffff;
        if (cc + 1 <= K) {
          if (lane <= cc) mine = lane;
        } else {
          if (lane < Kp) mine = l_idx[tk * kListStride + lane];
          else if (lane == Kp) mine = 0;
          else if (lane == Kp + 1) mine = cc - 1;
          else if (lane == Kp + 2) mine = cc;
        }
#pragma unroll
        for (int kk = 2; kk <= 32; kk <<= 1) {
#pragma unroll
          for (int j = kk >> 1; j > 0; j >>= 1) {
            const int other = __shfl_xor_sync(0xffffffffu, mine, j);
            const bool lower = (lane & j) == 0, asc = (lane & kk) == 0;
            mine = (lower == asc) ? min(mine, other) : max(mine, other);
          }
        }
        if (lane < K) a.idx[((long long)bh * geo.N + tt) * K + lane] = (mine == 0x7fffffff) ? -1 : mine;
      }
      __syncwarp();
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (s_fail && tid == 0) atomicExch(a.status, (int)PISA_ERR_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, 512);
}

bool flat_tc_supported(const Geometry& g, int dtype) {
  if (dtype != PISA_BF16) return false;
  if (g.d != 64 && g.d != 128) return false;
  if (g.G > 16 || g.K > 32) return false;
  for (int i = 0; i < 3; ++i)
    if ((g.qs[i] * 2) % 16 != 0) return false;
  return tma::encoder() != nullptr;
}

template <int D, int LG>
static int launch_flat_tc_dg(const Geometry& g, const void* q, const void* pyramid, int32_t* idx, int32_t* status,
                            cudaStream_t s) {
  const int tpt = 128 / g.G, tok_per_item = 2 * tpt;
  constexpr int TILE = (D / 64) * 128 * 128;
  FlatArgs a;
  a.idx = idx;
  a.status = status;
  a.n_pairs = (g.N + tok_per_item - 1) / tok_per_item;
  const long long items = (long long)g.B * g.Hkv * a.n_pairs;
  if (items > 0x7fffffffLL) return PISA_ERR_UNSUPPORTED;
  a.n_items = (int)items;
  const size_t lists = (size_t)tok_per_item * kListStride * 8;
  a.stages = 4;
  while (a.stages > 2 && (size_t)(2 + a.stages) * TILE + lists + 1024 > 220 * 1024) --a.stages;
  const size_t smem = (size_t)(2 + a.stages) * TILE + lists + 1024;
  CUtensorMap tm_q, tm_k;
  {
    const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.Hq, (uint64_t)g.N, (uint64_t)g.B};
    const uint64_t str[4] = {2, (uint64_t)g.qs[2] * 2, (uint64_t)g.qs[1] * 2, (uint64_t)g.qs[0] * 2};
    const uint32_t box[4] = {64u, (uint32_t)g.G, (uint32_t)tpt, 1u};
    if (!tma::make_map(&tm_q, 2, 4, q, dims, str, box, true)) return PISA_ERR_UNSUPPORTED;
  }
  {
    const __nv_bfloat16* lvl1 = (const __nv_bfloat16*)pyramid + g.level_off[1];
    const uint64_t dims[3] = {(uint64_t)g.d, (uint64_t)g.M[1], (uint64_t)g.B * g.Hkv};
    const uint64_t str[3] = {2, (uint64_t)g.d * 2, (uint64_t)g.M[1] * g.d * 2};
    const uint32_t box[3] = {64u, (uint32_t)kChunk, 1u};
    if (!tma::make_map(&tm_k, 2, 3, lvl1, dims, str, box, true)) return PISA_ERR_UNSUPPORTED;
  }
  cudaError_t e = cudaFuncSetAttribute(flat_tc_kernel<D, LG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { record_cuda_error("flat_tc attr", e); return PISA_ERR_CUDA; }
  const int grid = a.n_items < num_sms() ? a.n_items : num_sms();
  flat_tc_kernel<D, LG><<<grid, kFlatThreads, smem, s>>>(g, tm_q, tm_k, a);
  return check_launch("flat_tc");
}

template <int D>
static int launch_flat_tc_d(const Geometry& g, const void* q, const void* pyramid, int32_t* idx, int32_t* status,
                            cudaStream_t s) {
  switch (g.G) {
    case 1: return launch_flat_tc_dg<D, 0>(g, q, pyramid, idx, status, s);
    case 2: return launch_flat_tc_dg<D, 1>(g, q, pyramid, idx, status, s);
    case 4: return launch_flat_tc_dg<D, 2>(g, q, pyramid, idx, status, s);
    case 8: return launch_flat_tc_dg<D, 3>(g, q, pyramid, idx, status, s);
    case 16: return launch_flat_tc_dg<D, 4>(g, q, pyramid, idx, status, s);
    default: return PISA_ERR_UNSUPPORTED;
  }
}

int launch_flat_tc(const Geometry& g, const void* q, const void* pyramid, int32_t* idx, int32_t* status,
                   cudaStream_t s) {
  if (g.d == 128) return launch_flat_tc_d<128>(g, q, pyramid, idx, status, s);
  return launch_flat_tc_d<64>(g, q, pyramid, idx, status, s);
}

}  // namespace pisa
