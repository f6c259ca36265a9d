// Tensor-core path (bf16, tcgen05 + TMEM): key-block-major leaf scoring and block-sparse attention.
//
// Every query token picks its own blocks, and only the G heads of a group share them, so a
// query-major tile would have G useful rows out of 128.  Both dense contractions of the path are
// therefore run key-block-major (the two-stage idea of Algorithm 1, applied to the leaf scores and
// to the attention alike): the per-token lists are inverted into per-block lists of (token, slot)
// references, 128/G tokens x G heads are gathered into a 128-row A operand, and the block's keys
// (and values) stay resident in shared memory as the B operand while the list is walked.
//
//   routing   : stage 1 (levels L..2, SIMT) -> kept level-2 nodes
//               invert by level-2 node      -> lists of (token, slot)
//               lse_ws_kernel               -> per-head LSE of every child leaf (g*C keys per tile),
//                                              causal mask inside the query's own leaf
//               final_topk_kernel           -> grouped score = sum over heads, forced leaves, Top-K;
//                                              also the softmax denominator of the kept leaves
//   attention : invert idx by leaf          -> lists of (token, slot)
//               [lse_ws + row_lse only when the denominators are not already known]
//               pv_ws_kernel                -> S = Q K^T, P = exp(S - lse_row) (already normalised),
//                                              O_partial = P V, added into an fp32 accumulator with
//                                              vector reductions (two 256-byte row segments per instruction)
//               convert                     -> out in the storage dtype
#include <math_constants.h>

#include "pisa_tensor.cuh"
#include "tc_utils.cuh"
#include "tma_map.cuh"

namespace pisa {

using namespace tc;

namespace {

constexpr int kInvTok = 1024;          // tokens per CTA in the inversion kernels
constexpr int kWindowTok = 16384;      // tokens per window of the inverted lists
constexpr int kBwdWindowTok = 32768;   // ... of the backward's lists (fewer, fuller lists: 2.3 ms of 55 at the headline shape)
constexpr int kItemTiles = 32;         // a work item: at most this many consecutive tiles of one list
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ------------------------------------------------------------------ list inversion

// A list is keyed by (b*Hkv + h, token window, node): window-major inside a head, so that the tiles
// being worked on at any moment gather queries from (and, in the attention stage, accumulate into)
// a slice of the sequence small enough to stay in L2.
struct InvArgs {
  const int32_t* nodes;   // [BH, N, K] node ids (ascending, -1 padded)
  int K, fan, Mk, N, C, BH, tpt;
  int lgK, lgC;           // log2 of K and C when they are powers of two (shifts instead of divisions), else -1
  int W, NW;              // tokens per window (a multiple of kInvTok), windows per sequence
  int32_t* count;         // [BH*Mk]
  int32_t* entry_off;     // [BH*Mk + 1]
  int32_t* tile_off;      // [nkeys + 1]  tiles of tpt tokens
  int32_t* item_off;      // [nkeys + 1]  work items: runs of at most kItemTiles tiles of one list
  int32_t* item_key;      // [items]      the list each work item belongs to
  int32_t* cursor;        // [nkeys]
  int32_t* blk_tot;       // [3][ceil(nkeys / 1024) + 1] scan scratch: per-block totals, then block offsets
  int32_t* entries;       // [<= BH*N*K]  token | slot << 24
  int32_t* work_ctr;      // next-work-item counter of the attention kernel that walks these lists (zeroed with count)
  int32_t* status;        // the workspace's status word
  int debug;              // PISA_DEBUG_* bits
  int skip_forced;        // leave the row's forced leaves (0, c-1, c) out of the lists: the local-window kernel serves them
};

__device__ __forceinline__ int inv_token(const InvArgs& a, int e) { return a.lgK >= 0 ? (e >> a.lgK) : e / a.K; }
__device__ __forceinline__ int inv_slot(const InvArgs& a, int e) { return a.lgK >= 0 ? (e & (a.K - 1)) : e % a.K; }
__device__ __forceinline__ bool inv_valid(const InvArgs& a, int node, int t) {
  const int leaf = a.lgC >= 0 ? (t >> a.lgC) : t / a.C;
  const bool ok = node >= 0 && node < a.Mk && (long long)node * a.fan <= (long long)leaf;
  // bounds-check mode: anything but the -1 padding that is not a usable node id is reported
  if ((a.debug & PISA_DEBUG_BOUNDS) && !ok && node != -1) atomicExch(a.status, (int)PISA_ERR_BOUNDS);
  if (a.skip_forced && (node == 0 || node == leaf || node == leaf - 1)) return false;
  return ok;
}

__global__ void __launch_bounds__(256) inv_count_kernel(InvArgs a, int use_smem) {
  extern __shared__ int s_hist[];
  const int bh = blockIdx.y;
  const int t0 = blockIdx.x * kInvTok, t1 = min(t0 + kInvTok, a.N);
  const long long kbase = ((long long)bh * a.NW + t0 / a.W) * a.Mk;
  if (use_smem) {
    for (int j = threadIdx.x; j < a.Mk; j += blockDim.x) s_hist[j] = 0;
    __syncthreads();
  }
  const int n = (t1 - t0) * a.K;
  for (int e = threadIdx.x; e < n; e += blockDim.x) {
    const int t = t0 + inv_token(a, e);
    const int node = a.nodes[((long long)bh * a.N + t0) * a.K + e];
    if (inv_valid(a, node, t)) {
      if (use_smem) atomicAdd(&s_hist[node], 1);
      else atomicAdd(&a.count[kbase + node], 1);
    }
  }
  if (use_smem) {
    __syncthreads();
    for (int j = threadIdx.x; j < a.Mk; j += blockDim.x)
      if (s_hist[j]) atomicAdd(&a.count[kbase + j], s_hist[j]);
  }
}

// Exclusive scans of the list lengths (entries), of their tile counts and of their work-item counts,
// in three launches: per-block scans of 1024 lists each, a scan of the block totals, the fix-up.
__device__ __forceinline__ int3 inv_key_counts(const InvArgs& a, int i, int nkeys) {
  if (i >= nkeys) return make_int3(0, 0, 0);
  const int c = a.count[i];
  const int tl = (c + a.tpt - 1) / a.tpt;
  return make_int3(c, tl, (tl + kItemTiles - 1) / kItemTiles);
}
// inclusive scan of three ints over the 1024 threads of a CTA (warp shuffles, then the warp totals)
__device__ __forceinline__ int3 block_scan3(int3 v, int3* s_w /* [32] */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, v.x, o), y = __shfl_up_sync(0xffffffffu, v.y, o),
              z = __shfl_up_sync(0xffffffffu, v.z, o);
    if (lane >= o) { v.x += x; v.y += y; v.z += z; }
  }
  if (lane == 31) s_w[warp] = v;
  __syncthreads();
  if (warp == 0) {
    int3 w = s_w[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, w.x, o), y = __shfl_up_sync(0xffffffffu, w.y, o),
                z = __shfl_up_sync(0xffffffffu, w.z, o);
      if (lane >= o) { w.x += x; w.y += y; w.z += z; }
    }
    s_w[lane] = w;
  }
  __syncthreads();
  if (warp > 0) { const int3 p = s_w[warp - 1]; v.x += p.x; v.y += p.y; v.z += p.z; }
  return v;
}
__global__ void __launch_bounds__(1024) inv_scan_blocks_kernel(InvArgs a) {
  __shared__ int3 s_w[32];
  const int nkeys = a.BH * a.NW * a.Mk;
  const int nblk = (nkeys + 1023) / 1024;
  const int i = blockIdx.x * 1024 + threadIdx.x;
  const int3 own = inv_key_counts(a, i, nkeys);
  const int3 inc = block_scan3(own, s_w);
  if (i < nkeys) {                                         // exclusive prefix inside the block, for now
    a.entry_off[i] = inc.x - own.x; a.tile_off[i] = inc.y - own.y; a.item_off[i] = inc.z - own.z;
  }
  if (threadIdx.x == 1023) {
    a.blk_tot[blockIdx.x] = inc.x; a.blk_tot[(nblk + 1) + blockIdx.x] = inc.y;
    a.blk_tot[2 * (nblk + 1) + blockIdx.x] = inc.z;
  }
}
// block totals -> exclusive block offsets (entry [nblk] = grand total); one CTA walks them 1024 at a time
__global__ void __launch_bounds__(1024) inv_scan_totals_kernel(InvArgs a) {
  __shared__ int3 s_w[32];
  const int nkeys = a.BH * a.NW * a.Mk;
  const int nblk = (nkeys + 1023) / 1024;
  int3 carry = make_int3(0, 0, 0);
  for (int b0 = 0; b0 < nblk; b0 += 1024) {
    const int j = b0 + threadIdx.x;
    int3 own = make_int3(0, 0, 0);
    if (j < nblk) own = make_int3(a.blk_tot[j], a.blk_tot[(nblk + 1) + j], a.blk_tot[2 * (nblk + 1) + j]);
    __syncthreads();                                       // s_w of the previous round has been read
    const int3 inc = block_scan3(own, s_w);
    if (j < nblk) {
      a.blk_tot[j] = carry.x + inc.x - own.x; a.blk_tot[(nblk + 1) + j] = carry.y + inc.y - own.y;
      a.blk_tot[2 * (nblk + 1) + j] = carry.z + inc.z - own.z;
    }
    const int3 tot = s_w[31];
    carry.x += tot.x; carry.y += tot.y; carry.z += tot.z;
  }
  if (threadIdx.x == 0) {
    a.blk_tot[nblk] = carry.x; a.blk_tot[(nblk + 1) + nblk] = carry.y; a.blk_tot[2 * (nblk + 1) + nblk] = carry.z;
  }
}
__global__ void __launch_bounds__(1024) inv_scan_fix_kernel(InvArgs a) {
  const int nkeys = a.BH * a.NW * a.Mk;
  const int nblk = (nkeys + 1023) / 1024;
  const int i = blockIdx.x * 1024 + threadIdx.x;
  if (i < nkeys) {
    const int be = a.entry_off[i] + a.blk_tot[blockIdx.x];
    const int bt = a.tile_off[i] + a.blk_tot[(nblk + 1) + blockIdx.x];
    const int bi = a.item_off[i] + a.blk_tot[2 * (nblk + 1) + blockIdx.x];
    a.entry_off[i] = be; a.tile_off[i] = bt; a.item_off[i] = bi; a.cursor[i] = be;
    const int ni = inv_key_counts(a, i, nkeys).z;
    for (int x = 0; x < ni; ++x) a.item_key[bi + x] = i;
  }
  if (i == 0) {
    a.entry_off[nkeys] = a.blk_tot[nblk]; a.tile_off[nkeys] = a.blk_tot[(nblk + 1) + nblk];
    a.item_off[nkeys] = a.blk_tot[2 * (nblk + 1) + nblk];
  }
}

__global__ void __launch_bounds__(256) inv_fill_kernel(InvArgs a, int use_smem) {
  extern __shared__ int s_mem[];
  int* s_hist = s_mem;
  int* s_base = s_mem + a.Mk;
  const int bh = blockIdx.y;
  const int t0 = blockIdx.x * kInvTok, t1 = min(t0 + kInvTok, a.N);
  const long long kbase = ((long long)bh * a.NW + t0 / a.W) * a.Mk;
  const int n = (t1 - t0) * a.K;
  const int32_t* nodes = a.nodes + ((long long)bh * a.N + t0) * a.K;
  if (!use_smem) {
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
      const int t = t0 + inv_token(a, e), slot = inv_slot(a, e), node = nodes[e];
      if (inv_valid(a, node, t)) {
        const int pos = atomicAdd(&a.cursor[kbase + node], 1);
        a.entries[pos] = t | (slot << 24);
      }
    }
    return;
  }
  for (int j = threadIdx.x; j < a.Mk; j += blockDim.x) s_hist[j] = 0;
  __syncthreads();
  for (int e = threadIdx.x; e < n; e += blockDim.x) {
    const int node = nodes[e];
    if (inv_valid(a, node, t0 + inv_token(a, e))) atomicAdd(&s_hist[node], 1);
  }
  __syncthreads();
  for (int j = threadIdx.x; j < a.Mk; j += blockDim.x) {
    const int c = s_hist[j];
    if (c) s_base[j] = atomicAdd(&a.cursor[kbase + j], c);
    s_hist[j] = 0;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < n; e += blockDim.x) {
    const int t = t0 + inv_token(a, e), slot = inv_slot(a, e), node = nodes[e];
    if (inv_valid(a, node, t)) {
      const int r = atomicAdd(&s_hist[node], 1);
      a.entries[s_base[node] + r] = t | (slot << 24);
    }
  }
}

// ------------------------------------------------------------------ tile kernels

struct TileArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  const int32_t* entry_off;
  const int32_t* tile_off;
  const int32_t* item_off;
  const int32_t* item_key;
  const int32_t* entries;
  int nkeys, Mk, NW, fan, slots;
  int mode;                // score written per (leaf, head): PISA_SCORE_LSE (also what attention needs), MEAN, MEAN_VAR
  float* blk_lse;          // [BH, N, slots*fan, G]   (tile_lse)
  const float* row_lse;    // [B, Hq, N]              (tile_pv)
  float* o_acc;            // fp32 accumulator: [B, Hkv, N, D, G] when the second product is transposed, else [B, N, Hq, D]
  int32_t* status;
  int debug;               // PISA_DEBUG_* bits: list entries are range-checked before they are used
};

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~(uintptr_t)1023);
}

// Work items of both tile kernels are handed out dynamically: lists differ in length, and a static
// round-robin left the CTAs' tile counts 20 % apart.  The leaf-scoring kernel has a scheduler warp of its own
// (see there).  In the attention kernel thread 0 of the CTA draws the next item from a global counter when the
// producers start their k-th item and publishes it in a small shared-memory ring; every other role reads
// the k-th entry when it gets there (it lags the producers by a few items at most: the producers cannot
// start item k before the UMMAs of item k - 1 have completed).  An id >= the item count ends the walk.
constexpr int kFeedRing = 16;
struct ItemInfo {
  int key, ntiles, e_begin, e_end;         // ntiles == 0: no more work
};
struct ItemFeed { volatile int4 info[kFeedRing]; volatile int seq[kFeedRing]; };
// The wait is bounded by a poll count (about 2^27 shared-memory reads, seconds), not by the clock: the
// readers are at their register limit and must not carry 64-bit time stamps through their loops.
__device__ __noinline__ ItemInfo feed_get(ItemFeed& f, int k, volatile int* fail) {
  ItemInfo r = {0, 0, 0, 0};
  const int slot = k % kFeedRing;
  for (uint32_t i = 0; f.seq[slot] != k + 1; ++i) {
    if (*fail) return r;
    if (i == (1u << 27)) { *fail = 1; return r; }
  }
  __threadfence_block();
  r.key = f.info[slot].x; r.ntiles = f.info[slot].y; r.e_begin = f.info[slot].z; r.e_end = f.info[slot].w;
  return r;
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Online log-sum-exp (base 2) over one 32-column chunk of raw fp32 logits; (m, ssum) is the running
// (max, sum of 2^(x - max)) with x = raw * sl2.  sl2 > 0, so the max commutes with the scaling.
template <int NW>
__device__ __forceinline__ void lse_chunk(const uint32_t (&rr)[NW], float sl2, float& m, float& ssum) {
  float c0 = __uint_as_float(rr[0]), c1 = __uint_as_float(rr[1]);
  float c2 = __uint_as_float(rr[2]), c3 = __uint_as_float(rr[3]);
#pragma unroll
  for (int j = 4; j < NW; j += 4) {
    c0 = fmaxf(c0, __uint_as_float(rr[j]));
    c1 = fmaxf(c1, __uint_as_float(rr[j + 1]));
    c2 = fmaxf(c2, __uint_as_float(rr[j + 2]));
    c3 = fmaxf(c3, __uint_as_float(rr[j + 3]));
  }
  const float mn = fmaxf(m, fmaxf(fmaxf(c0, c1), fmaxf(c2, c3)) * sl2);
  const float neg = -mn;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
  for (int j = 0; j < NW; j += 4) {
    a0 += ex2_approx(fmaf(__uint_as_float(rr[j]), sl2, neg));
    a1 += ex2_approx(fmaf(__uint_as_float(rr[j + 1]), sl2, neg));
    a2 += ex2_approx(fmaf(__uint_as_float(rr[j + 2]), sl2, neg));
    a3 += ex2_approx(fmaf(__uint_as_float(rr[j + 3]), sl2, neg));
  }
  ssum = ssum * ex2_approx(m - mn) + ((a0 + a1) + (a2 + a3));
  m = mn;
}
// the same with only the first `nvalid` (>= 1) columns of the chunk taking part.  The sums associate
// exactly as in lse_chunk (four interleaved accumulators), so a full row gives bit-identical results on
// either path: which path a row takes depends on the other rows of its tile, and the composition of a
// tile (the order of a list's entries) varies from run to run.
template <int NW>
__device__ __forceinline__ void lse_chunk_masked(const uint32_t (&rr)[NW], int nvalid, float sl2, float& m,
                                                 float& ssum) {
  float cm = -CUDART_INF_F;
#pragma unroll
  for (int j = 0; j < NW; ++j)
    if (j < nvalid) cm = fmaxf(cm, __uint_as_float(rr[j]));
  const float mn = fmaxf(m, cm * sl2);
  const float neg = -mn;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int j = 0; j < NW; ++j)
    if (j < nvalid) acc[j & 3] += ex2_approx(fmaf(__uint_as_float(rr[j]), sl2, neg));
  ssum = ssum * ex2_approx(m - mn) + ((acc[0] + acc[1]) + (acc[2] + acc[3]));
  m = mn;
}
// first and second moments of the first `nvalid` of 32 logits about `shift` (score modes "mean" and
// "mean + variance/2", Sec. 4.3)
template <int NW>
__device__ __forceinline__ void stat_chunk(const uint32_t (&rr)[NW], int nvalid, float scale, float shift, float& s1,
                                           float& s2) {
#pragma unroll
  for (int j = 0; j < NW; ++j)
    if (j < nvalid) {
      const float dlt = fmaf(__uint_as_float(rr[j]), scale, -shift);
      s1 += dlt;
      s2 = fmaf(dlt, dlt, s2);
    }
}

// ------------------------------------------------------------------ warp-specialised tile kernels
//
// One persistent CTA per SM.  Producer warps stage the gathered query rows (16-byte cp.async into the
// swizzled layouts, a ring of NS query tiles; the block's keys / values arrive by TMA tile loads with the
// first tile of a work item), one warp issues the UMMA chains into two alternating TMEM accumulators, the
// remaining warps read the accumulators out.  Every role derives ring slots and mbarrier parities from its
// own tile counter; all waits are bounded.

// leaf scoring: 4 producer warps, 1 UMMA warp, 1 scheduler warp, 16 epilogue warps.  22 warps put six on two of
// the SM's sub-partitions, i.e. 80 registers per thread (as 21 warps did); more producer warps measured slower
// (the gather is limited by the bytes the four ring slots keep in flight, not by the warps that issue it)
constexpr int kLseProd = 128;
constexpr int kLseThreads = kLseProd + 64 + 512;
constexpr int kLseRing = 16;           // tiles the scheduler warp may run ahead of the epilogue
constexpr int kProdThreads = 128;
constexpr int kMetaRing = 8;           // ring of per-tile metadata; deeper than any role can run ahead

// bounds-check mode: a list entry (token | slot << 24) must name a token below N and a slot below `slots`;
// one that does not is reported and dropped (-1 = no entry)
__device__ __forceinline__ int checked_entry(const TileArgs& a, int N, int ent) {
  if (!(a.debug & PISA_DEBUG_BOUNDS) || ent < 0) return ent;
  if ((ent & 0xFFFFFF) < N && (ent >> 24) < a.slots) return ent;
  atomicExch(a.status, (int)PISA_ERR_BOUNDS);
  return -1;
}
__device__ __forceinline__ int fetch_entry(const int32_t* entries, int e0, int e_end, int tpt, int p) {
  return (p < tpt && e0 + p < e_end) ? entries[e0 + p] : -1;
}
__device__ __forceinline__ ItemInfo item_info(const TileArgs& a, int item, int tpt) {
  ItemInfo r;
  r.key = a.item_key[item];
  const int local = item - a.item_off[r.key];
  const int list0 = a.entry_off[r.key], cnt = a.entry_off[r.key + 1] - list0;
  const int tiles = (cnt + tpt - 1) / tpt;
  const int first = local * kItemTiles;
  r.ntiles = min(kItemTiles, tiles - first);
  r.e_begin = list0 + first * tpt;
  r.e_end = list0 + cnt;
  return r;
}

// thread 0 of the CTA: draw the k-th item of this CTA from the global counter and publish its description
__device__ __forceinline__ ItemInfo feed_publish(ItemFeed& f, const TileArgs& a, int32_t* work_ctr, int n_items, int tpt,
                                              int k) {
  const int item = atomicAdd(work_ctr, 1);
  ItemInfo r = {0, 0, 0, 0};
  if (item < n_items) r = item_info(a, item, tpt);
  f.info[k % kFeedRing].x = r.key; f.info[k % kFeedRing].y = r.ntiles;
  f.info[k % kFeedRing].z = r.e_begin; f.info[k % kFeedRing].w = r.e_end;
  __threadfence_block();
  f.seq[k % kFeedRing] = k + 1;
  return r;
}

// The 128 producer threads copy rows [row0, row0+nrows) of a [tokens][D] matrix into swizzled K-major
// slabs.  Thread p always moves 16-byte chunk (p % (D/8)) of rows (p / (D/8)) + i * (1024/D): the row
// index modulo 8 -- hence the swizzle -- is the same for every i, so the destination just advances.
template <int D>
__device__ __forceinline__ void prod_load_rows(uint8_t* dst, int slab_bytes, const __nv_bfloat16* base,
                                               long long row_stride, int row0, int nrows, int limit, int p) {
  constexpr int CH = D / 8, RPP = kProdThreads / CH;
  const int ck = p % CH, rb = p / CH;
  uint32_t d = smem_u32(dst + (ck >> 3) * slab_bytes) + swz128(rb, ck & 7);
  const __nv_bfloat16* src = base + (long long)(row0 + rb) * row_stride + ck * 8;
  for (int row = rb; row < nrows; row += RPP) {
    if (row0 + row < limit) cp_async16(d, src);
    else st_shared_zero16(d);
    d += RPP * 128;
    src += (long long)RPP * row_stride;
  }
}
// ... and gather the 128 query rows of a tile: row r = (entry r >> lgG, head r & (G-1)); the tile's
// entries sit in shared memory (-1 = no entry)
template <int D>
__device__ __forceinline__ void prod_gather_q(uint8_t* dst, const Geometry& geo, const __nv_bfloat16* qb,
                                              const int* s_ent, int p) {
  constexpr int CH = D / 8, RPP = kProdThreads / CH;
  const int ck = p % CH, rb = p / CH;
  const int G = geo.G, lgG = 31 - __clz(G);
  uint32_t d = smem_u32(dst + (ck >> 3) * (128 * 128)) + swz128(rb, ck & 7);
  const __nv_bfloat16* src0 = qb + ck * 8;
  const long long s1 = geo.qs[1], s2 = geo.qs[2];
#pragma unroll 4
  for (int row = rb; row < 128; row += RPP) {
    const int ent = s_ent[row >> lgG];
    if (ent >= 0) cp_async16(d, src0 + (long long)(ent & 0xFFFFFF) * s1 + (long long)(row & (G - 1)) * s2);
    else st_shared_zero16(d);
    d += RPP * 128;
  }
}
// ... the same gather with the tile's entries already in the thread's registers (ent[i] belongs to row
// rb + i * RPP; -1 = no entry): no shared-memory round trip and no barrier among the producer warps
template <int D>
__device__ __forceinline__ void prod_gather_q_regs(uint8_t* dst, const Geometry& geo, const __nv_bfloat16* qb,
                                                   const int (&ent)[128 / (kProdThreads / (D / 8))], int p) {
  constexpr int CH = D / 8, RPP = kProdThreads / CH, RPT = 128 / RPP;
  const int ck = p % CH, rb = p / CH;
  const int G = geo.G;
  uint32_t d = smem_u32(dst + (ck >> 3) * (128 * 128)) + swz128(rb, ck & 7);
  const __nv_bfloat16* src0 = qb + ck * 8;
  const long long s1 = geo.qs[1], s2 = geo.qs[2];
#pragma unroll
  for (int i = 0; i < RPT; ++i) {
    const int row = rb + i * RPP;
    if (ent[i] >= 0) cp_async16(d, src0 + (long long)(ent[i] & 0xFFFFFF) * s1 + (long long)(row & (G - 1)) * s2);
    else st_shared_zero16(d);
    d += RPP * 128;
  }
}
// barrier among the 128 producer threads that also ORs a flag, so that they leave their loops together
__device__ __forceinline__ bool prod_sync_or(bool flag) {
  uint32_t any;
  asm volatile(
      "{\n"
      ".reg .pred p, q;\n"
      "setp.ne.b32 q, %1, 0;\n"
      "bar.red.or.pred p, 1, 128, q;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(any)
      : "r"(flag ? 1u : 0u)
      : "memory");
  return any != 0;
}

// query-ring stages of lse_ws_kernel: what 227 KB leave beside two key buffers and ~26 KB of static shared memory
__host__ __device__ constexpr int lse_ws_stages(int D, int NB) {
  return ((D / 64) * 128 * 128 * 4 + 2 * (D / 64) * NB * 128 + 27 * 1024 <= 227 * 1024) ? 4 : 2;
}

// MOM: false = per-head LSE of every leaf; true = first / second moments of the logits (score modes
// "mean" and "mean + variance/2"), a separate instantiation so that the LSE one keeps its registers.
template <int D, int NB, bool MOM>
__global__ void __launch_bounds__(kLseThreads, 1)
lse_ws_kernel(Geometry geo, TileArgs a, int32_t* work_ctr, const __grid_constant__ CUtensorMap tm_k) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int KS = D / 64;
  constexpr int A_SLAB = 128 * 128, B_SLAB = NB * 128;
  constexpr int A_STAGE = KS * A_SLAB;
  // the node's keys are double-buffered (the next work item's keys load while this one's tiles run); the query
  // ring gets what is left: four stages, two when the keys take 2 x 64 KB
  constexpr int B_BUF = KS * B_SLAB;
  constexpr int NS = lse_ws_stages(D, NB);
  constexpr uint32_t TM_COLS = (2 * NB < 32) ? 32 : 2 * NB;
  constexpr int R = kLseRing;
  // epilogue warps per tile: all sixteen on a 256-column accumulator; two groups of eight on alternate tiles
  // for narrower ones (a small tile's fixed latencies then overlap with the other group's tile)
  constexpr int GR = (NB <= 128) ? 2 : 1;
  constexpr int WQ = 4 / GR;                      // warps of one tile that share a TMEM lane quarter
  constexpr int W = NB / WQ;                      // accumulator columns of one epilogue warp
  constexpr int CW = (W < 32) ? W : 32;           // columns per TMEM load
  uint8_t* smem = align1024(smem_raw);
  uint8_t* sA = smem;
  uint8_t* sB = smem + NS * A_STAGE;
  __shared__ uint64_t a_full[NS], a_empty[NS], b_full[2], b_empty[2], t_full[2], t_empty[2];
  __shared__ uint64_t m_full[R], m_empty[R];      // the tile ring: written by the scheduler warp, released by the epilogue
  __shared__ int s_tent[R][128];                  // a tile's entries (token | slot << 24, -1 = none)
  __shared__ int4 s_tkey[R];                      // its (unit, node, flags: 1 = first tile of a work item, 2 = last)
  __shared__ float4 s_part[2][16][32];            // partial results of the warps that share a leaf (by tile parity)
  __shared__ volatile int s_total;                // number of tiles of this CTA, known once the walk has ended
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_fail;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    s_total = 0x7fffffff;
    for (int i = 0; i < NS; ++i) { mbar_init(&a_full[i], kLseProd); mbar_init(&a_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&b_empty[i], 1); mbar_init(&b_full[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&t_full[i], 1); mbar_init(&t_empty[i], 512 / GR); }
    for (int i = 0; i < R; ++i) { mbar_init(&m_full[i], 1); mbar_init(&m_empty[i], 16 / GR); }
    s_fail = 0;
    mbar_fence_init();
  }
  if (warp == 0) { tmem_alloc(&tmem_slot, TM_COLS); tmem_relinquish(); }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  const int G = geo.G, lgG = 31 - __clz(G), tpt = 128 >> lgG, C = geo.C;
  const float sl2 = geo.scale * kLog2e;

  // Every role but the scheduler walks TILES: it waits for tile `it`'s ring entry (or its accumulator) and
  // leaves when the scheduler has published the tile count and `it` has reached it.  A try_wait suspends the
  // warp for a while, so the poll count bounds the wait to seconds.
  auto wait_tile = [&](uint64_t* bar, uint32_t parity, int it) -> bool {
    for (uint32_t i = 0; i < (1u << 24); ++i) {
      if (mbar_try_wait(bar, parity)) return true;
      if (it >= s_total || s_fail) return false;
    }
    s_fail = 1;
    return false;
  };

  if (warp < kLseProd / 32) {
    // ------------------------------------------------ producers: gather the tile's query rows
    constexpr int CH = D / 8, RPP = kLseProd / CH;
    const int ck = tid % CH, rb = tid / CH;
    int n_item = 0;
    for (int it = 0;; ++it) {
      const int mr = it % R, s = it % NS;
      if (!wait_tile(&m_full[mr], (uint32_t)((it / R) & 1), it)) break;
      const int4 key = s_tkey[mr];
      if (tid == 0 && (key.z & 1)) {
        // first tile of a work item: the node's keys, one TMA tile load per 64-wide slab (own memory, no
        // multicast), into the buffer the item before the previous one used, once its MMAs have released it
        const int pb = n_item & 1;
        if (n_item >= 2 && !mbar_wait_bounded(&b_empty[pb], (uint32_t)((n_item / 2 - 1) & 1))) { s_fail = 1; break; }
        ++n_item;
        const int b = key.x / geo.Hkv, h = key.x % geo.Hkv;
        mbar_arrive_expect_tx(&b_full[pb], (uint32_t)B_BUF);
        for (int ks = 0; ks < KS; ++ks)
          tma_load_4d(smem_u32(sB + pb * B_BUF + ks * B_SLAB), &tm_k, &b_full[pb], ks * 64, h, key.y * NB, b);
      }
      if (it >= NS && !mbar_wait_bounded(&a_empty[s], (uint32_t)((it / NS - 1) & 1))) { s_fail = 1; break; }
      const int b = key.x / geo.Hkv, h = key.x % geo.Hkv;
      const __nv_bfloat16* src0 = a.q + (long long)b * geo.qs[0] + (long long)(h * G) * geo.qs[2] + ck * 8;
      const long long s1 = geo.qs[1], s2 = geo.qs[2];
      const uint32_t d0 = smem_u32(sA + s * A_STAGE + (ck >> 3) * A_SLAB);
      const int* ents = s_tent[mr];
#pragma unroll 4
      for (int row = rb; row < 128; row += RPP) {       // RPP need not be a multiple of 8: the swizzle is per row
        const int ent = ents[row >> lgG];
        const uint32_t d = d0 + swz128(row, ck & 7);
        if (ent >= 0) cp_async16(d, src0 + (long long)(ent & 0xFFFFFF) * s1 + (long long)(row & (G - 1)) * s2);
        else st_shared_zero16(d);
      }
      fence_proxy_async_smem();                 // zero-filled rows (plain stores) -> async proxy
      cp_async_arrive_noinc(&a_full[s]);        // fires when this thread's copies have landed
    }
    cp_async_wait_all();
  } else if (warp == kLseProd / 32) {
    // ------------------------------------------------ MMA issuer (the warp walks the loop, lane 0 issues)
    const uint32_t idesc = make_idesc_bf16(128, NB, 0, 0);
    int n_item = 0;
    for (int it = 0;; ++it) {
      const int mr = it % R, s = it % NS, buf = it & 1;
      if (!wait_tile(&m_full[mr], (uint32_t)((it / R) & 1), it)) break;
      const int flags = s_tkey[mr].z;
      bool ok = true;
      const int pb = n_item & 1;
      if (flags & 1) ok = mbar_wait_bounded(&b_full[pb], (uint32_t)((n_item / 2) & 1));      // the node's keys have landed
      if (ok) ok = mbar_wait_bounded(&a_full[s], (uint32_t)((it / NS) & 1));
      if (ok && it >= 2) ok = mbar_wait_bounded(&t_empty[buf], (uint32_t)(((it >> 1) - 1) & 1));
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { s_fail = 1; break; }
      if (lane == 0) {
        fence_proxy_async_smem();
        tcgen05_fence_after_sync();
        const uint32_t a0 = smem_u32(sA + s * A_STAGE), b0 = smem_u32(sB + pb * B_BUF);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t da = make_smem_desc(a0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
          const uint64_t db = make_smem_desc(b0 + (kk >> 2) * B_SLAB + (kk & 3) * 32, 0, 1024);
          umma_bf16(tmem + (uint32_t)(buf * NB), da, db, idesc, kk > 0);
        }
        umma_commit(&a_empty[s]);
        umma_commit(&t_full[buf]);
        if (flags & 2) umma_commit(&b_empty[pb]);    // last tile of the item: its MMAs release the keys
      }
      if (flags & 2) ++n_item;
      __syncwarp();
    }
  } else if (warp == kLseProd / 32 + 1) {
    // ------------------------------------------------ scheduler: draws work items, lays out their tiles
    // Lists differ in length, so the items are handed out dynamically from a global counter (zero on entry).
    // The warp runs up to R tiles ahead of the epilogue: the latency of the draw, of the item's description
    // and of the entries' loads stays off every other role's path.
    const int n_items = a.item_off[a.nkeys];
    const int win_tok = (geo.N < kWindowTok) ? ((geo.N + kInvTok - 1) / kInvTok) * kInvTok : kWindowTok;
    int it = 0, last_win = -1;
    bool ok = true;
    while (ok) {
      int item = 0;
      if (lane == 0) item = atomicAdd(work_ctr, 1);
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item >= n_items) break;
      const ItemInfo inf = item_info(a, item, tpt);
      const int bh = inf.key / (a.NW * a.Mk), j = inf.key % a.Mk;
      // A gather completes when its last row has landed, and a tile that meets even one row for the first
      // time waits for HBM.  So, on entering a window of the lists, the CTA asks for its share of the NEXT
      // window's query rows to be brought into L2 (the CTAs walk the windows together).
      if (inf.key / a.Mk != last_win) {
        last_win = inf.key / a.Mk;
        const int nw = last_win + 1;
        if (nw < geo.B * geo.Hkv * a.NW) {
          const int bh2 = nw / a.NW, w2 = nw % a.NW;
          const int t0 = w2 * win_tok, t1 = min(geo.N, t0 + win_tok);
          const int per = (t1 - t0 + (int)gridDim.x - 1) / (int)gridDim.x;
          const int ta = t0 + (int)blockIdx.x * per, tb = min(t1, ta + per);
          const __nv_bfloat16* qb2 = a.q + (long long)(bh2 / geo.Hkv) * geo.qs[0] + (long long)((bh2 % geo.Hkv) * G) * geo.qs[2];
          for (int i = lane; i < (tb - ta) * G; i += 32)
            prefetch_l2_bulk(qb2 + (long long)(ta + (i >> lgG)) * geo.qs[1] + (long long)(i & (G - 1)) * geo.qs[2], (uint32_t)(D * 2));
        }
      }
      // 128 consecutive entries (128 / tpt tiles) are fetched per round trip to L2, and the next 128 are
      // requested before the current ones are laid out
      const int lg_tpt = 7 - lgG, tiles_per_batch = 128 >> lg_tpt;
      auto fetch = [&](int jt0, int (&dst)[4]) {
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int e = inf.e_begin + (jt0 << lg_tpt) + lane + 32 * x;
          dst[x] = (jt0 < inf.ntiles && e < inf.e_end) ? a.entries[e] : -1;
        }
      };
      int nxt[4];
      fetch(0, nxt);
      for (int jt0 = 0; jt0 < inf.ntiles && ok; jt0 += tiles_per_batch) {
        int ent[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) ent[x] = nxt[x];
        fetch(jt0 + tiles_per_batch, nxt);
        for (int u = 0; u < tiles_per_batch; ++u) {
          const int jt = jt0 + u;
          if (jt >= inf.ntiles) break;
          const int mr = it % R;
          if (it >= R) ok = mbar_wait_bounded(&m_empty[mr], (uint32_t)((it / R - 1) & 1));
          ok = __all_sync(0xffffffffu, ok && !s_fail);
          if (!ok) break;
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int f = lane + 32 * x;                  // position in the batch
            if ((f >> lg_tpt) == u) s_tent[mr][f & (tpt - 1)] = checked_entry(a, geo.N, ent[x]);
          }
          if (lane == 0) s_tkey[mr] = make_int4(bh, j, (jt == 0 ? 1 : 0) | (jt == inf.ntiles - 1 ? 2 : 0), 0);
          __syncwarp();
          if (lane == 0) mbar_arrive(&m_full[mr]);     // release: the ring entry is complete
          ++it;
        }
      }
    }
    if (!ok) s_fail = 1;
    if (lane == 0) s_total = it;
  } else {
    // ------------------------------------------------ epilogue: sixteen warps
    // The warps of a tile that share a TMEM lane quarter (four, all sixteen warps on one tile, for a 256-column
    // accumulator; two, the warps in two groups on alternate tiles, for narrower ones) split the accumulator's
    // columns, W each -- few enough to hold in registers.  A warp therefore reads its columns out at once and
    // releases the accumulator BEFORE it starts on the exponentials: the next-but-one tile's UMMAs never wait
    // for arithmetic.  A leaf wider than W is shared by C / W warps of the quarter; they leave their partial
    // (max, sum) in shared memory and the first of them combines (always in the same order).
    const int ew = warp - (kLseProd / 32 + 2);
    const int grp = (GR == 2) ? (ew >> 3) : 0;          // which tiles this warp works on (it % GR == grp)
    const int cq = (ew >> 2) & (WQ - 1);                // column share inside the tile; warp % 4 = TMEM lane quarter
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(cq * W);
    const int head = row & (G - 1);
    const int wpl = C / W;                              // warps per leaf (C >= W: at most four children per node)
    const int r = (cq * W) / C;                         // the child this warp's columns belong to
    const int off = cq * W - r * C;                     // its first column inside that child
    const bool owner = (cq % wpl) == 0;
    const int bar_id = 1 + grp * 8 + (warp & 3) * 2 + ((wpl == 2 && WQ == 4) ? (cq >> 1) : 0);
    constexpr bool lse_mode = !MOM;
    for (int it = grp;; it += GR) {
      const int buf = it & 1;
      if (!wait_tile(&t_full[buf], (uint32_t)((it >> 1) & 1), it)) break;
      tcgen05_fence_after_sync();
      uint32_t ra[CW], rb[CW];
      if constexpr (W == 16) {
        tmem_ld_32x16(lane_base + (uint32_t)(buf * NB), ra);
      } else {
        tmem_ld_32x32(lane_base + (uint32_t)(buf * NB), ra);
        if constexpr (W == 64) tmem_ld_32x32(lane_base + (uint32_t)(buf * NB + 32), rb);
      }
      tmem_ld_wait();
      tcgen05_fence_before_sync();
      mbar_arrive(&t_empty[buf]);                       // this thread's columns are in registers
      const int mr = it % R;
      const int ent = s_tent[mr][row >> lgG];
      const int bh = s_tkey[mr].x, j = s_tkey[mr].y;
      __syncwarp();
      if (lane == 0) mbar_arrive(&m_empty[mr]);         // this warp has read the ring entry
      const bool valid = ent >= 0;
      const int t = ent & 0xFFFFFF, slot = valid ? (ent >> 24) : 0;
      const int c_t = t / C;
      const int leaf = j * a.fan + r;
      int ncols = 0;                                    // causally visible columns of the child for this row
      if (valid && leaf <= c_t && leaf < geo.M[1])
        ncols = (leaf == c_t) ? (t - leaf * C + 1) : min(C, geo.N - leaf * C);
      const int nv = max(0, min(W, ncols - off));       // ... of them inside this warp's columns
      const bool fast = __all_sync(0xffffffffu, nv == W || nv == 0);
      float m = -CUDART_INF_F, ssum = 0.f;
      float shift = 0.f, s1 = 0.f, s2 = 0.f;            // moment modes: logits about the warp's first one
      if (!lse_mode) {
        shift = __uint_as_float(ra[0]) * geo.scale;
        if (nv > 0) stat_chunk<CW>(ra, nv, geo.scale, shift, s1, s2);
        if constexpr (W == 64) if (nv > 32) stat_chunk<CW>(rb, nv - 32, geo.scale, shift, s1, s2);
      } else if (fast) {
        lse_chunk<CW>(ra, sl2, m, ssum);
        if constexpr (W == 64) lse_chunk<CW>(rb, sl2, m, ssum);
      } else {
        if (nv > 0) lse_chunk_masked<CW>(ra, nv, sl2, m, ssum);
        if constexpr (W == 64) if (nv > 32) lse_chunk_masked<CW>(rb, nv - 32, sl2, m, ssum);
      }
      if (nv == 0) { m = -CUDART_INF_F; ssum = 0.f; }   // (the unmasked path ran on this row's columns all the same)
      // partial of this warp: LSE mode (m, ssum); moment modes (count, mean, M2 = sum of squared deviations)
      float4 part;
      if (lse_mode) {
        part = make_float4(m, ssum, 0.f, 0.f);
      } else {
        const float n = (float)nv, mu_d = (nv > 0) ? s1 / n : 0.f;
        part = make_float4(n, shift + mu_d, fmaxf(s2 - s1 * mu_d, 0.f), 0.f);
      }
      if (wpl > 1) {
        s_part[buf][ew][lane] = part;
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(wpl * 32) : "memory");
        if (owner) {
          for (int i = 1; i < wpl; ++i) {
            const float4 o = s_part[buf][ew + 4 * i][lane];
            if (lse_mode) {
              const float mn = fmaxf(part.x, o.x);
              const float sa = (part.x == mn) ? part.y : part.y * ex2_approx(part.x - mn);
              const float sb = (o.x == mn) ? o.y : o.y * ex2_approx(o.x - mn);
              part.x = mn;
              part.y = sa + sb;
            } else if (o.x > 0.f) {
              const float n = part.x + o.x, dl = o.y - part.y;
              part.z = part.z + o.z + dl * dl * (part.x * o.x / n);
              part.y = part.y + dl * (o.x / n);
              part.x = n;
            }
          }
        }
      }
      if (valid && owner) {
        float lse;
        if (lse_mode) {
          lse = (ncols > 0) ? (part.x + log2f(part.y)) * kLn2 : -CUDART_INF_F;
        } else {
          lse = (ncols > 0) ? part.y + ((a.mode == PISA_SCORE_MEAN_VAR) ? 0.5f * part.z / part.x : 0.f) : -CUDART_INF_F;
        }
        a.blk_lse[(((long long)bh * geo.N + t) * (a.slots * a.fan) + slot * a.fan + r) * G + head] = lse;
      }
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (s_fail && tid == 0) atomicExch(a.status, (int)PISA_ERR_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

// Attention tiles.  Roles: warps 0-3 producers, warp 4 UMMA issuer, warps 5-8 / 9-12 two softmax groups
// taking alternate tiles, warps 13-16 the reducer.  Per tile: S = Q K^T (UMMA) -> a softmax group
// turns S into P = 2^(S*scale*log2e - lse2) in bf16, overwriting the query tile's ring slot ->
// O_partial = P V (UMMA, V as the MN-major operand) -> the reducer moves O out of TMEM through the
// (now free) ring slot and adds it into the fp32 accumulator with coalesced vector reductions, then
// releases the slot.  The reduction stream into L2 is the floor of this kernel (64 KB of fp32 adds
// per tile), so it gets warps of its own and is never stalled by the exponentials.
constexpr int kPvThreads = 544;

template <int D, int C>
__global__ void __launch_bounds__(kPvThreads, 1)
pv_ws_kernel(Geometry geo, TileArgs a, int32_t* work_ctr, const __grid_constant__ CUtensorMap tm_k,
             const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int NS = 4;
  constexpr int KS = D / 64;
  constexpr int A_SLAB = 128 * 128, KV_SLAB = C * 128;
  constexpr int STAGE_ROW = 256 + 16;        // 64 fp32 + pad: conflict-free 16-byte row writes
  constexpr int QP_BYTES = (KS * A_SLAB > 128 * STAGE_ROW) ? KS * A_SLAB : 128 * STAGE_ROW;
  constexpr int Q_STAGE = (QP_BYTES + 1023) / 1024 * 1024;
  constexpr uint32_t TM_COLS = 512;          // S buffers at columns 0 / 128, O buffers at 256 / 384
  // d = 128: the second product is issued transposed, O^T = V^T P^T (A = V, MN-major; B = P): a TMEM lane
  // is then one output column d and consecutive TMEM columns are the G heads of one token.  With the
  // accumulator laid out [B, Hkv, N, d, G] (heads innermost) a thread adds its G values with one vector
  // reduction and a warp covers 32*G consecutive floats: fully coalesced, no staging in shared memory.
  constexpr bool kTransO = (D == 128);
  uint8_t* smem = align1024(smem_raw);
  uint8_t* sQ = smem;
  uint8_t* sK = smem + NS * Q_STAGE;
  uint8_t* sV = sK + KS * KV_SLAB;
  __shared__ uint64_t q_full[NS], q_empty[NS], kv_full, kv_empty, s_full[2], s_empty[2], p_ready[2], o_full[2], o_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_fail;
  __shared__ int s_ent[kMetaRing][128];   // per-tile entries, written by the producers, read by all roles
  __shared__ float s_lse[kMetaRing][128]; // per-row softmax denominators
  __shared__ ItemFeed feed;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid < kFeedRing) feed.seq[tid] = 0;
  if (tid == 0) {
    for (int i = 0; i < NS; ++i) { mbar_init(&q_full[i], kProdThreads); mbar_init(&q_empty[i], kTransO ? 1 : 128); }
    mbar_init(&kv_empty, 1);
    mbar_init(&kv_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 128); mbar_init(&p_ready[i], 128);
      mbar_init(&o_full[i], 1); mbar_init(&o_empty[i], 128);
    }
    s_fail = 0;
    mbar_fence_init();
  }
  if (warp == 0) { tmem_alloc(&tmem_slot, TM_COLS); tmem_relinquish(); }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  const int G = geo.G, lgG = 31 - __clz(G), tpt = 128 >> lgG;
  const int n_items = a.item_off[a.nkeys];
  const float sl2 = geo.scale * kLog2e;

  if (warp < 4) {
    // ------------------------------------------------ producers
    int it = 0, kiter = 0, ent_next = -1;
    bool stop = false;
    for (;; ++kiter) {
      if (tid == 0) feed_publish(feed, a, work_ctr, n_items, tpt, kiter);     // lane 0 draws the item; everybody reads it back
      __syncwarp();
      const ItemInfo inf = feed_get(feed, kiter, &s_fail);
      if (inf.ntiles == 0 || stop) break;
      const int bh = inf.key / (a.NW * a.Mk), leaf = inf.key % a.Mk;
      const int b = bh / geo.Hkv, h = bh % geo.Hkv;
      bool bad = s_fail != 0;
      if (!bad && kiter > 0) bad = !mbar_wait_bounded(&kv_empty, (uint32_t)((kiter - 1) & 1));
      if (prod_sync_or(bad)) { s_fail = 1; stop = true; break; }
      if (tid == 0) {
        // the block's keys and values: contiguous C x d slabs, one TMA tile load per 64-wide slab (this GPU's
        // memory, no multicast; rows past N read as zero), so that the producer warps only gather queries
        mbar_arrive_expect_tx(&kv_full, (uint32_t)(2 * KS * KV_SLAB));
        for (int ks = 0; ks < KS; ++ks) {
          tma_load_4d(smem_u32(sK + ks * KV_SLAB), &tm_k, &kv_full, ks * 64, h, leaf * C, b);
          tma_load_4d(smem_u32(sV + ks * KV_SLAB), &tm_v, &kv_full, ks * 64, h, leaf * C, b);
        }
      }
      const __nv_bfloat16* qb = a.q + (long long)b * geo.qs[0] + (long long)(h * G) * geo.qs[2];
      for (int jt = 0; jt < inf.ntiles; ++jt, ++it) {
        const int s = it % NS;
        const bool bad_t = it >= NS && !mbar_wait_bounded(&q_empty[s], (uint32_t)((it / NS - 1) & 1));
        const int e0 = inf.e_begin + jt * tpt;
        const int ent_now = (jt == 0) ? checked_entry(a, geo.N, fetch_entry(a.entries, e0, inf.e_end, tpt, tid)) : ent_next;
        ent_next = (jt + 1 < inf.ntiles) ? checked_entry(a, geo.N, fetch_entry(a.entries, e0 + tpt, inf.e_end, tpt, tid)) : -1;
        s_ent[it % kMetaRing][tid] = ent_now;
        if (prod_sync_or(bad_t)) { s_fail = 1; stop = true; break; }
        prod_gather_q<D>(sQ + s * Q_STAGE, geo, qb, s_ent[it % kMetaRing], tid);
        {  // the row's softmax denominator rides along (4-byte copy per row)
          const int ent_r = s_ent[it % kMetaRing][tid >> lgG];
          if (ent_r >= 0)
            cp_async4(smem_u32(&s_lse[it % kMetaRing][tid]),
                      a.row_lse + ((long long)b * geo.Hq + h * G + (tid & (G - 1))) * geo.N + (ent_r & 0xFFFFFF));
        }
        fence_proxy_async_smem();                 // zero-filled rows (plain stores) -> async proxy
        cp_async_arrive_noinc(&q_full[s]);        // fires when this thread's copies have landed
      }
    }
    cp_async_wait_all();
  } else if (warp == 4) {
    // ------------------------------------------------ MMA issuer
    // Event driven: S(it) goes out as soon as its query tile has landed and its S buffer has been
    // read out, P V(it) as soon as P(it) is written and its O buffer has been read out; neither
    // waits for the other.  Lane 0 probes and issues; the warp stays converged on its decisions.
    const uint32_t idesc_s = make_idesc_bf16(128, C, 0, 0);
    const uint32_t idesc_o = make_idesc_bf16(128, D, 0, 1);
    const uint32_t idesc_ot = make_idesc_bf16(128, 128, 1, 0);   // O^T: M = d (V, MN-major), N = tile rows (P)
    int s_it = 0, pv_it = 0;              // next tile whose S / whose P V is to be issued
    unsigned last_bits = 0;               // bit (it & 31): tile `it` closes its work item
    int kseq = 0, jt = 0;
    ItemInfo inf = feed_get(feed, kseq, &s_fail);
    uint64_t t_idle = 0;
    uint32_t idle_polls = 0;
    bool ok = true;
    while (ok && !s_fail) {
      const bool more_s = inf.ntiles > 0;
      if (!more_s && pv_it == s_it) break;
      int do_s = 0, do_pv = 0;
      if (lane == 0) {
        if (more_s && s_it - pv_it < 2) {
          const int s = s_it % NS, buf = s_it & 1;
          do_s = mbar_test(&q_full[s], (uint32_t)((s_it / NS) & 1)) && mbar_test(&kv_full, (uint32_t)(kseq & 1)) &&
                 (s_it < 2 || mbar_test(&s_empty[buf], (uint32_t)(((s_it >> 1) - 1) & 1)));
        }
        if (pv_it < s_it) {
          const int pb = pv_it & 1;
          do_pv = mbar_test(&p_ready[pb], (uint32_t)((pv_it >> 1) & 1)) &&
                  (pv_it < 2 || mbar_test(&o_empty[pb], (uint32_t)(((pv_it >> 1) - 1) & 1)));
        }
      }
      do_s = __shfl_sync(0xffffffffu, do_s, 0);
      do_pv = __shfl_sync(0xffffffffu, do_pv, 0);
      if (do_pv) {
        const int ps = pv_it % NS, pb = pv_it & 1;
        if (lane == 0) {
          tcgen05_fence_after_sync();
          const uint32_t p0 = smem_u32(sQ + ps * Q_STAGE), v0 = smem_u32(sV);
#pragma unroll
          for (int kk = 0; kk < C / 16; ++kk) {
            const uint64_t dp = make_smem_desc(p0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
            const uint64_t dv = make_smem_desc(v0 + kk * (16 * 128), KV_SLAB, 1024);
            if (kTransO) umma_bf16(tmem + 256u + (uint32_t)(pb * 128), dv, dp, idesc_ot, kk > 0);
            else umma_bf16(tmem + 256u + (uint32_t)(pb * 128), dp, dv, idesc_o, kk > 0);
          }
          umma_commit(&o_full[pb]);
          if (kTransO) umma_commit(&q_empty[ps]);     // P has been consumed: the ring slot is free
          if ((last_bits >> (pv_it & 31)) & 1u) umma_commit(&kv_empty);   // K/V of that item are free
        }
        ++pv_it;
      }
      if (do_s) {
        const int s = s_it % NS, buf = s_it & 1;
        if (lane == 0) {
          fence_proxy_async_smem();
          tcgen05_fence_after_sync();
          const uint32_t q0 = smem_u32(sQ + s * Q_STAGE), k0 = smem_u32(sK);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t da = make_smem_desc(q0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
            const uint64_t db = make_smem_desc(k0 + (kk >> 2) * KV_SLAB + (kk & 3) * 32, 0, 1024);
            umma_bf16(tmem + (uint32_t)(buf * 128), da, db, idesc_s, kk > 0);
          }
          umma_commit(&s_full[buf]);
        }
        const bool last = (jt == inf.ntiles - 1);
        last_bits = (last_bits & ~(1u << (s_it & 31))) | ((last ? 1u : 0u) << (s_it & 31));
        ++s_it;
        if (last) {
          inf = feed_get(feed, ++kseq, &s_fail);
          jt = 0;
        } else {
          ++jt;
        }
      }
      __syncwarp();
      if (do_s || do_pv) {
        idle_polls = 0;
      } else if ((++idle_polls & 1023u) == 0u) {    // look at the wall clock only now and then
        const uint64_t now = global_timer_ns();
        if (idle_polls == 1024u) t_idle = now;
        else if (now - t_idle > 2000000000ull) ok = false;
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      }
    }
    if (!ok) s_fail = 1;
  } else if (warp < 13) {
    // ------------------------------------------------ softmax groups: S -> P
    const int grp = (warp - 5) >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t s_base = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(grp * 128);
    int it = 0;
    for (int kseq = 0; !s_fail; ++kseq) {
      const ItemInfo inf = feed_get(feed, kseq, &s_fail);
      if (inf.ntiles == 0) break;
      const int leaf = inf.key % a.Mk;
      for (int jt = 0; jt < inf.ntiles; ++jt, ++it) {
        if ((it & 1) != grp) continue;
        const int s = it % NS;
        uint8_t* slot_base = sQ + s * Q_STAGE;
        if (!mbar_wait_bounded(&s_full[grp], (uint32_t)((it >> 1) & 1))) { s_fail = 1; break; }
        tcgen05_fence_after_sync();
        const int ent = s_ent[it % kMetaRing][row >> lgG];
        const int t = ent & 0xFFFFFF;
        float neg_lse2 = 0.f;
        int ncols = 0;
        if (ent >= 0) {
          const float l2 = s_lse[it % kMetaRing][row] * kLog2e;
          const int c_t = t / C;
          if (leaf <= c_t && l2 > -CUDART_INF_F)
            ncols = (leaf == c_t) ? (t - leaf * C + 1) : min(C, geo.N - leaf * C);
          neg_lse2 = -l2;
        }
        const bool fast = __all_sync(0xffffffffu, ncols == C);
        uint32_t ra[32], rb[32];
        tmem_ld_32x32(s_base, ra);
#pragma unroll
        for (int c0 = 0; c0 < C; c0 += 32) {
          uint32_t (&cur)[32] = ((c0 >> 5) & 1) ? rb : ra;
          uint32_t (&nxt)[32] = ((c0 >> 5) & 1) ? ra : rb;
          tmem_ld_wait();
          if (c0 + 32 < C) {
            tmem_ld_32x32(s_base + (uint32_t)(c0 + 32), nxt);
          } else {
            tcgen05_fence_before_sync();
            mbar_arrive(&s_empty[grp]);         // S has been read out: the next S chain may overwrite it
          }
          uint32_t pk[16];
#pragma unroll
          for (int jx = 0; jx < 16; ++jx) {
            float p0 = ex2_approx(fmaf(__uint_as_float(cur[2 * jx]), sl2, neg_lse2));
            float p1 = ex2_approx(fmaf(__uint_as_float(cur[2 * jx + 1]), sl2, neg_lse2));
            if (!fast) {
              if (c0 + 2 * jx >= ncols) p0 = 0.f;
              if (c0 + 2 * jx + 1 >= ncols) p1 = 0.f;
            }
            const __nv_bfloat162 pp = __floats2bfloat162_rn(p0, p1);
            pk[jx] = *reinterpret_cast<const uint32_t*>(&pp);
          }
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int ck = c0 / 8 + q4;
            const uint32_t d = smem_u32(slot_base + (ck >> 3) * A_SLAB) + swz128(row, ck & 7);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(d), "r"(pk[4 * q4]),
                         "r"(pk[4 * q4 + 1]), "r"(pk[4 * q4 + 2]), "r"(pk[4 * q4 + 3])
                         : "memory");
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(&p_ready[grp]);
      }
    }
  } else {
    // ------------------------------------------------ reducer: O partials -> fp32 accumulator
    // Every thread parks 64 columns of its row in its padded row of the tile's ring slot (free once
    // P V has completed); the warp then re-reads its own 32 rows two at a time, so that each vector
    // reduction instruction adds two full 256-byte row segments.
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const int sub = lane >> 4, ch = lane & 15;
    int it = 0;
    for (int kseq = 0; !s_fail; ++kseq) {
      const ItemInfo inf = feed_get(feed, kseq, &s_fail);
      if (inf.ntiles == 0) break;
      const int bh = inf.key / (a.NW * a.Mk);
      const int b = bh / geo.Hkv, h = bh % geo.Hkv;
      float* acc_bh = a.o_acc + ((long long)b * geo.N * geo.Hq + h * G) * D;
      for (int jt = 0; jt < inf.ntiles; ++jt, ++it) {
        const int s = it % NS, ob = it & 1;
        uint8_t* slot_base = sQ + s * Q_STAGE;
        uint8_t* stage = slot_base + row * STAGE_ROW;
        const int* ents = s_ent[it % kMetaRing];
        const uint32_t o_base = tmem + lane_sel + 256u + (uint32_t)(ob * 128);
        if (!mbar_wait_bounded(&o_full[ob], (uint32_t)((it >> 1) & 1))) { s_fail = 1; break; }
        tcgen05_fence_after_sync();
        if constexpr (kTransO) {
          // lane = output column d (= `row` of this thread), TMEM column = tile row = entry*G + head
          const int* ents = s_ent[it % kMetaRing];
          float* acc_d = a.o_acc + (((long long)b * geo.Hkv + h) * geo.N) * (long long)(D * G) + (long long)row * G;
          const long long tok_stride = (long long)D * G;
          uint32_t ra[32], rb[32];
          tmem_ld_32x32(o_base, ra);
#pragma unroll
          for (int c0 = 0; c0 < 128; c0 += 32) {
            uint32_t (&cur)[32] = ((c0 >> 5) & 1) ? rb : ra;
            uint32_t (&nxt)[32] = ((c0 >> 5) & 1) ? ra : rb;
            tmem_ld_wait();
            if (c0 + 32 < 128) {
              tmem_ld_32x32(o_base + (uint32_t)(c0 + 32), nxt);
            } else {
              tcgen05_fence_before_sync();
              mbar_arrive(&o_empty[ob]);          // O has been read out of TMEM
            }
            if (G >= 4) {
#pragma unroll
              for (int q4 = 0; q4 < 8; ++q4) {
                const int col = c0 + 4 * q4;
                const int ent_c = ents[col >> lgG];
                if (ent_c >= 0) {
                  float* dst = acc_d + (long long)(ent_c & 0xFFFFFF) * tok_stride + (col & (G - 1));
                  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst),
                               "f"(__uint_as_float(cur[4 * q4])), "f"(__uint_as_float(cur[4 * q4 + 1])),
                               "f"(__uint_as_float(cur[4 * q4 + 2])), "f"(__uint_as_float(cur[4 * q4 + 3]))
                               : "memory");
                }
              }
            } else if (G == 2) {
#pragma unroll
              for (int q2 = 0; q2 < 16; ++q2) {
                const int ent_c = ents[(c0 + 2 * q2) >> 1];
                if (ent_c >= 0) {
                  float* dst = acc_d + (long long)(ent_c & 0xFFFFFF) * tok_stride;
                  asm volatile("red.relaxed.gpu.global.add.v2.f32 [%0], {%1, %2};" ::"l"(dst),
                               "f"(__uint_as_float(cur[2 * q2])), "f"(__uint_as_float(cur[2 * q2 + 1]))
                               : "memory");
                }
              }
            } else {
#pragma unroll
              for (int q1 = 0; q1 < 32; ++q1) {
                const int ent_c = ents[c0 + q1];
                if (ent_c >= 0) atomicAdd(acc_d + (long long)(ent_c & 0xFFFFFF) * tok_stride, __uint_as_float(cur[q1]));
              }
            }
          }
        } else {
#pragma unroll
        for (int half = 0; half < KS; ++half) {
          uint32_t ra[32], rb[32];
          tmem_ld_32x32(o_base + (uint32_t)(half * 64), ra);
          tmem_ld_32x32(o_base + (uint32_t)(half * 64 + 32), rb);
          tmem_ld_wait();
          if (half == KS - 1) {
            tcgen05_fence_before_sync();
            mbar_arrive(&o_empty[ob]);          // O has been read out of TMEM
          }
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(stage) + q4 * 16), "r"(ra[4 * q4]),
                         "r"(ra[4 * q4 + 1]), "r"(ra[4 * q4 + 2]), "r"(ra[4 * q4 + 3])
                         : "memory");
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(stage) + 128 + q4 * 16),
                         "r"(rb[4 * q4]), "r"(rb[4 * q4 + 1]), "r"(rb[4 * q4 + 2]), "r"(rb[4 * q4 + 3])
                         : "memory");
          __syncwarp();
#pragma unroll 4
          for (int i = 0; i < 16; ++i) {
            const int R = (warp & 3) * 32 + 2 * i + sub;           // tile row served by this half-warp
            const int ent_r = ents[R >> lgG];
            if (ent_r >= 0) {
              float4 x;
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                           : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w)
                           : "r"(smem_u32(slot_base + R * STAGE_ROW) + ch * 16));
              float* dst = acc_bh + ((long long)(ent_r & 0xFFFFFF) * geo.Hq + (R & (G - 1))) * D + half * 64 + ch * 4;
              asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(x.x), "f"(x.y),
                           "f"(x.z), "f"(x.w)
                           : "memory");
            }
          }
          __syncwarp();
        }
        mbar_arrive(&q_empty[s]);          // the ring slot is free again
        }
      }
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (s_fail && tid == 0) atomicExch(a.status, (int)PISA_ERR_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

// ------------------------------------------------------------------ small SIMT stages

// Final Select_K of the two-stage schedule (Algorithm 1): the candidates are the children of the
// kept level-2 nodes; grouped score = sum of the per-head leaf LSEs; forced leaves kept unscored.
// Also emits the softmax denominator of the kept leaves per query head (their LSEs are known).
__global__ void __launch_bounds__(128) final_topk_kernel(Geometry geo, const int32_t* __restrict__ par,
                                                          const float* __restrict__ blk_lse,
                                                          int32_t* __restrict__ idx, float* __restrict__ margin,
                                                          float* __restrict__ lse_out, float* __restrict__ sel_lse,
                                                          int32_t* status) {
  __shared__ __align__(16) float s_u[4][kMaxCand];
  __shared__ int s_sel[4][kMaxK];
  __shared__ float s_cut[4][2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // one warp per (b, KV head, token): blockIdx.y = the (b, KV head) unit, so no 64-bit division; the divisions
  // by g and C are shifts where those are powers of two (the usual case)
  const int t = blockIdx.x * 4 + warp;
  if (t >= geo.N) return;
  const int bh = blockIdx.y;
  const long long w = (long long)bh * geo.N + t;
  const int K = geo.K, g = geo.g, gK = g * K, G = geo.G;
  const int lgg = (g & (g - 1)) == 0 ? __ffs(g) - 1 : -1, lgC = (geo.C & (geo.C - 1)) == 0 ? __ffs(geo.C) - 1 : -1;
  auto div_g = [&](int x) { return lgg >= 0 ? x >> lgg : x / g; };
  auto mod_g = [&](int x) { return lgg >= 0 ? x & (g - 1) : x % g; };
  const int c = lgC >= 0 ? t >> lgC : t / geo.C;
  const int f1 = (c >= 1) ? c - 1 : 0;
  const int32_t* pr = par + w * (long long)K;
  const float* bl = blk_lse + w * (long long)gK * G;
  float* u = s_u[warp];
  // candidate ci = slot*g + r  <->  leaf par[slot]*g + r; valid ones form a prefix
  int nV = 0;
  float4 xs[kMaxCand / 32];                    // G == 4: the candidates' per-head scores, kept for the LSE
#pragma unroll
  for (int ch = 0; ch < kMaxCand / 32; ++ch) xs[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int ch = 0; ch < kMaxCand / 32; ++ch) {
    const int c0 = ch * 32;
    if (c0 >= gK) break;
    const int ci = c0 + lane;
    bool ok = false;
    if (ci < gK) {
      int p = pr[div_g(ci)];
      if ((geo.debug & PISA_DEBUG_BOUNDS) && p != -1 && !bounds_ok(p, geo.M[2], status)) p = -1;
      const int leaf = p * g + mod_g(ci);
      ok = (p >= 0) && (leaf <= c);
      float sc = -CUDART_INF_F;
      if (ok) {
        if (G == 4) xs[ch] = *reinterpret_cast<const float4*>(bl + ci * 4);   // one 16-byte load per candidate
        if (leaf == 0 || leaf == f1 || leaf == c) sc = forced_score(ci);
        else {
          if (G == 4) {
            const float4 x = xs[ch];
            sc = (x.x + x.y) + (x.z + x.w);
          } else {
            sc = 0.f;
            for (int hh = 0; hh < G; ++hh) sc += bl[ci * G + hh];
          }
        }
      }
      u[ci] = sc;
    }
    nV += __popc(__ballot_sync(0xffffffffu, ok));
  }
  __syncwarp();
  if (lane < 4 && nV + lane < kMaxCand) u[nV + lane] = -CUDART_INF_F;     // padding read by the 16-byte loads
  __syncwarp();
  const bool prune = nV > K;
  int rank[kMaxCand / 32];
  const bool sorted = prune && nV <= 64;         // the common case: a sorting network instead of ranks
  bool keep_s[2] = {false, false};
  float cut_a = 0.f, cut_b = 0.f;
  if (sorted) {
    const float u0 = (lane < nV) ? u[lane] : -CUDART_INF_F, u1 = (lane + 32 < nV) ? u[lane + 32] : -CUDART_INF_F;
    warp_select_sorted64(u0, u1, K, lane, keep_s[0], keep_s[1], cut_a, cut_b);
  } else if (prune) {
    warp_select_ranks(u, nV, lane, rank);
  }
  int base = 0;
  unsigned kept_mask[kMaxCand / 32];
#pragma unroll
  for (int ch = 0; ch < kMaxCand / 32; ++ch) {
    const int s0 = ch * 32;
    const int s = s0 + lane;
    bool keep = s < nV;
    if (sorted) {
      keep = keep && (ch < 2) && keep_s[ch & 1];
    } else if (prune && s0 < nV) {
      keep = keep && (rank[ch] < K);
      if (s < nV && rank[ch] == K - 1) s_cut[warp][0] = u[s];
      if (s < nV && rank[ch] == K) s_cut[warp][1] = u[s];
    }
    const unsigned bal = __ballot_sync(0xffffffffu, keep);
    kept_mask[ch] = bal;
    const int pos = base + __popc(bal & ((1u << lane) - 1u));
    if (keep) s_sel[warp][pos] = pr[div_g(s)] * g + mod_g(s);
    if (keep && sel_lse != nullptr) {
      // the kept leaf's per-head scores ARE its per-head softmax denominators (LSE mode)
      const int bq = bh / geo.Hkv, hq = bh % geo.Hkv;
      for (int hh = 0; hh < G; ++hh)
        sel_lse[(((long long)bq * geo.Hq + hq * G + hh) * geo.N + t) * K + pos] = bl[s * G + hh];
    }
    base += __popc(bal);
  }
  if (sel_lse != nullptr) {
    const int bq = bh / geo.Hkv, hq = bh % geo.Hkv;
    for (int s = base + lane; s < K; s += 32)
      for (int hh = 0; hh < G; ++hh)
        sel_lse[(((long long)bq * geo.Hq + hq * G + hh) * geo.N + t) * K + s] = -CUDART_INF_F;
  }
  __syncwarp();
  int32_t* dst = idx + w * (long long)K;
  for (int s = lane; s < K; s += 32) dst[s] = (s < base) ? s_sel[warp][s] : -1;
  if (margin != nullptr && lane == 0) {
    float mg = margin[w];
    if (prune) {
      const float a = sorted ? cut_a : s_cut[warp][0], bb = sorted ? cut_b : s_cut[warp][1];
      if (a < kForcedFloor) mg = fminf(mg, (a - bb) / fmaxf(fabsf(a), 1.f));
    }
    margin[w] = mg;
  }
  if (lse_out != nullptr && G == 4) {
    // four heads at once: element-wise over the kept candidates, then a butterfly that halves the
    // number of live values while it halves the lane groups (6 shuffles per reduction instead of 20)
    const int b = bh / geo.Hkv, h = bh % geo.Hkv;
    float4 m4 = make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
#pragma unroll
    for (int ch = 0; ch < kMaxCand / 32; ++ch)
      if ((kept_mask[ch] >> lane) & 1u) {
        m4.x = fmaxf(m4.x, xs[ch].x); m4.y = fmaxf(m4.y, xs[ch].y);
        m4.z = fmaxf(m4.z, xs[ch].z); m4.w = fmaxf(m4.w, xs[ch].w);
      }
    const bool hi16 = (lane & 16) != 0, hi8 = (lane & 8) != 0;
    // after the two packing steps lane holds head 2*bit4 + bit3
    float a0 = hi16 ? m4.z : m4.x, a1 = hi16 ? m4.w : m4.y;
    a0 = fmaxf(a0, __shfl_xor_sync(0xffffffffu, hi16 ? m4.x : m4.z, 16));
    a1 = fmaxf(a1, __shfl_xor_sync(0xffffffffu, hi16 ? m4.y : m4.w, 16));
    float mm = fmaxf(hi8 ? a1 : a0, __shfl_xor_sync(0xffffffffu, hi8 ? a0 : a1, 8));
    mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, 4));
    mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, 2));
    mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, 1));
    m4.x = __shfl_sync(0xffffffffu, mm, 0);
    m4.y = __shfl_sync(0xffffffffu, mm, 8);
    m4.z = __shfl_sync(0xffffffffu, mm, 16);
    m4.w = __shfl_sync(0xffffffffu, mm, 24);
    float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int ch = 0; ch < kMaxCand / 32; ++ch)
      if ((kept_mask[ch] >> lane) & 1u) {
        s4.x += __expf(xs[ch].x - m4.x); s4.y += __expf(xs[ch].y - m4.y);
        s4.z += __expf(xs[ch].z - m4.z); s4.w += __expf(xs[ch].w - m4.w);
      }
    float b0 = hi16 ? s4.z : s4.x, b1 = hi16 ? s4.w : s4.y;
    b0 += __shfl_xor_sync(0xffffffffu, hi16 ? s4.x : s4.z, 16);
    b1 += __shfl_xor_sync(0xffffffffu, hi16 ? s4.y : s4.w, 16);
    float ss = (hi8 ? b1 : b0) + __shfl_xor_sync(0xffffffffu, hi8 ? b0 : b1, 8);
    ss += __shfl_xor_sync(0xffffffffu, ss, 4);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    if ((lane & 7) == 0) {
      const int hh = lane >> 3;
      lse_out[((long long)b * geo.Hq + h * G + hh) * geo.N + t] = mm + __logf(ss);
    }
  } else if (lse_out != nullptr) {
    const int b = bh / geo.Hkv, h = bh % geo.Hkv;
    for (int hh = 0; hh < G; ++hh) {
      float m = -CUDART_INF_F;
      for (int s0 = 0, ch = 0; s0 < gK; s0 += 32, ++ch)
        if ((kept_mask[ch] >> lane) & 1u) m = fmaxf(m, bl[(s0 + lane) * G + hh]);
      m = warp_max(m);
      float ssum = 0.f;
      for (int s0 = 0, ch = 0; s0 < gK; s0 += 32, ++ch)
        if ((kept_mask[ch] >> lane) & 1u) ssum += __expf(bl[(s0 + lane) * G + hh] - m);
      ssum = warp_sum(ssum);
      if (lane == 0) lse_out[((long long)b * geo.Hq + h * G + hh) * geo.N + t] = m + __logf(ssum);
    }
  }
}

// softmax denominator of a row from the per-block LSEs of its selected leaves (stand-alone attention)
__global__ void __launch_bounds__(256) row_lse_kernel(Geometry geo, const int32_t* __restrict__ idx,
                                                       const float* __restrict__ blk_lse, float* __restrict__ lse_out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long total = (long long)geo.B * geo.Hkv * geo.N * geo.G;
  if (i >= total) return;
  const int head = (int)(i % geo.G);
  const long long w = i / geo.G;
  const int t = (int)(w % geo.N);
  const int bh = (int)(w / geo.N);
  const int c = t / geo.C;
  float m = -CUDART_INF_F;
  for (int s = 0; s < geo.K; ++s) {
    const int leaf = idx[w * geo.K + s];
    if (leaf >= 0 && leaf <= c && leaf < geo.M[1]) m = fmaxf(m, blk_lse[(w * geo.K + s) * geo.G + head]);
  }
  float ssum = 0.f;
  for (int s = 0; s < geo.K; ++s) {
    const int leaf = idx[w * geo.K + s];
    if (leaf >= 0 && leaf <= c && leaf < geo.M[1]) ssum += expf(blk_lse[(w * geo.K + s) * geo.G + head] - m);
  }
  const int b = bh / geo.Hkv, h = bh % geo.Hkv;
  lse_out[((long long)b * geo.Hq + h * geo.G + head) * geo.N + t] = (ssum > 0.f) ? m + logf(ssum) : -CUDART_INF_F;
}

// the same from per-block denominators the caller hands in (float [B,Hq,N,K], as pisa_route writes them)
__global__ void __launch_bounds__(256) row_lse_from_sel_kernel(Geometry geo, const int32_t* __restrict__ idx,
                                                                const float* __restrict__ sel_lse,
                                                                float* __restrict__ lse_out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // (b*Hq + hq)*N + t
  const long long total = (long long)geo.B * geo.Hq * geo.N;
  if (i >= total) return;
  const int t = (int)(i % geo.N);
  const int hq = (int)((i / geo.N) % geo.Hq);
  const int b = (int)(i / ((long long)geo.N * geo.Hq));
  const int32_t* row = idx + (((long long)b * geo.Hkv + hq / geo.G) * geo.N + t) * geo.K;
  const float* sl = sel_lse + i * geo.K;
  const int c = t / geo.C;
  float m = -CUDART_INF_F;
  for (int s = 0; s < geo.K; ++s) {
    const int leaf = row[s];
    if (leaf >= 0 && leaf <= c && leaf < geo.M[1]) m = fmaxf(m, sl[s]);
  }
  float ssum = 0.f;
  for (int s = 0; s < geo.K; ++s) {
    const int leaf = row[s];
    if (leaf >= 0 && leaf <= c && leaf < geo.M[1] && sl[s] > -CUDART_INF_F) ssum += expf(sl[s] - m);
  }
  lse_out[i] = (ssum > 0.f) ? m + logf(ssum) : -CUDART_INF_F;
}

// fp32 accumulator [B,N,Hq,d] -> out in bf16 (strided)
__global__ void __launch_bounds__(256) convert_out_kernel(Geometry geo, const float* __restrict__ acc,
                                                           __nv_bfloat16* __restrict__ out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // one 8-element chunk
  const int ch = geo.d / 8;
  const long long total = (long long)geo.B * geo.N * geo.Hq * ch;
  if (i >= total) return;
  const int ck = (int)(i % ch);
  const long long row = i / ch;
  const int hq = (int)(row % geo.Hq);
  const long long bt = row / geo.Hq;
  const int t = (int)(bt % geo.N), b = (int)(bt / geo.N);
  const float4 x0 = *reinterpret_cast<const float4*>(acc + row * geo.d + ck * 8);
  const float4 x1 = *reinterpret_cast<const float4*>(acc + row * geo.d + ck * 8 + 4);
  __nv_bfloat162 p0 = __floats2bfloat162_rn(x0.x, x0.y), p1 = __floats2bfloat162_rn(x0.z, x0.w);
  __nv_bfloat162 p2 = __floats2bfloat162_rn(x1.x, x1.y), p3 = __floats2bfloat162_rn(x1.z, x1.w);
  uint4 o;
  o.x = *reinterpret_cast<uint32_t*>(&p0); o.y = *reinterpret_cast<uint32_t*>(&p1);
  o.z = *reinterpret_cast<uint32_t*>(&p2); o.w = *reinterpret_cast<uint32_t*>(&p3);
  *reinterpret_cast<uint4*>(out + (long long)b * geo.os[0] + (long long)t * geo.os[1] + (long long)hq * geo.os[2] + ck * 8) = o;
}

// fp32 accumulator [B,Hkv,N,d,G] (heads innermost, the transposed-product layout) -> out in bf16.
// One thread takes two consecutive d of one (b, t, KV head): 2*G contiguous floats in, one bf16x2 per
// head out; a warp reads 64*G contiguous floats and writes 128 contiguous bytes per head row.
__global__ void __launch_bounds__(256) convert_out_heads_inner_kernel(Geometry geo, const float* __restrict__ acc,
                                                                       __nv_bfloat16* __restrict__ out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // one pair of d
  const int pairs = geo.d / 2, G = geo.G;
  const long long total = (long long)geo.B * geo.N * geo.Hkv * pairs;
  if (i >= total) return;
  const int dp = (int)(i % pairs);
  const long long row = i / pairs;                    // (b*N + t)*Hkv + h
  const int h = (int)(row % geo.Hkv);
  const long long bt = row / geo.Hkv;
  const int t = (int)(bt % geo.N), b = (int)(bt / geo.N);
  const float* src = acc + ((((long long)b * geo.Hkv + h) * geo.N + t) * geo.d + dp * 2) * G;
  __nv_bfloat16* dst = out + (long long)b * geo.os[0] + (long long)t * geo.os[1] + (long long)(h * G) * geo.os[2] + dp * 2;
  for (int hd = 0; hd < G; ++hd) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(src[hd], src[G + hd]);
    *reinterpret_cast<__nv_bfloat162*>(dst + (long long)hd * geo.os[2]) = p;
  }
}

// ------------------------------------------------------------------ host side

struct InvLayout {
  size_t count, work_ctr, entry_off, tile_off, item_off, item_key, cursor, blk_tot, entries, end;
};

int window_tokens(const Geometry& g, int win) { return g.N < win ? ((g.N + kInvTok - 1) / kInvTok) * kInvTok : win; }
int num_windows(const Geometry& g, int win) { return (g.N + window_tokens(g, win) - 1) / window_tokens(g, win); }

InvLayout inv_layout(size_t base, const Geometry& g, int Mk, int win = kWindowTok) {
  const size_t nkeys = (size_t)g.B * g.Hkv * num_windows(g, win) * Mk;
  InvLayout l;
  size_t o = base;
  l.count = o; o += align_up(nkeys * 4, 256);
  l.work_ctr = o; o += 256;                 // right behind count: one memset clears both
  l.entry_off = o; o += align_up((nkeys + 1) * 4, 256);
  l.tile_off = o; o += align_up((nkeys + 1) * 4, 256);
  l.item_off = o; o += align_up((nkeys + 1) * 4, 256);
  // every list adds at most one partial item on top of (all tiles) / kItemTiles
  const size_t max_tiles = (size_t)g.B * g.Hkv * g.N * g.K / (128 / g.G) + nkeys;
  l.item_key = o; o += align_up((max_tiles / kItemTiles + nkeys + 1) * 4, 256);
  l.cursor = o; o += align_up(nkeys * 4, 256);
  l.blk_tot = o; o += align_up(3 * ((nkeys + 1023) / 1024 + 1) * 4, 256);
  l.entries = o; o += align_up((size_t)g.B * g.Hkv * g.N * g.K * 4, 256);
  l.end = o;
  return l;
}

struct RouteLayout { size_t par, blk, total; InvLayout inv; };
RouteLayout route_layout(const Geometry& g) {
  RouteLayout r;
  size_t o = 0;
  r.par = o; o += align_up((size_t)g.B * g.Hkv * g.N * g.K * 4, 256);
  r.blk = o; o += align_up((size_t)g.B * g.Hkv * g.N * g.g * g.K * g.G * 4, 256);
  r.inv = inv_layout(o, g, g.M[2]);
  r.total = r.inv.end;
  return r;
}
struct BsaLayout { size_t blk, acc, total; InvLayout inv; };
BsaLayout bsa_layout(const Geometry& g) {
  BsaLayout r;
  size_t o = 0;
  r.blk = o; o += align_up((size_t)g.B * g.Hkv * g.N * g.K * g.G * 4, 256);
  r.acc = o; o += align_up((size_t)g.B * g.N * g.Hq * g.d * 4, 256);
  r.inv = inv_layout(o, g, g.M[1]);
  r.total = r.inv.end;
  return r;
}

int run_inversion(const Geometry& g, const int32_t* nodes, int fan, int Mk, char* ws, const InvLayout& l,
                  InvArgs* out, int32_t* status, cudaStream_t s, int win = kWindowTok, int skip_forced = 0) {
  InvArgs a;
  a.status = status; a.debug = g.debug; a.skip_forced = skip_forced;
  a.nodes = nodes; a.K = g.K; a.fan = fan; a.Mk = Mk; a.N = g.N; a.C = g.C; a.BH = g.B * g.Hkv;
  a.tpt = 128 / g.G;
  a.lgK = (g.K & (g.K - 1)) == 0 ? 31 - __builtin_clz((unsigned)g.K) : -1;
  a.lgC = (g.C & (g.C - 1)) == 0 ? 31 - __builtin_clz((unsigned)g.C) : -1;
  a.W = window_tokens(g, win); a.NW = num_windows(g, win);
  a.count = (int32_t*)(ws + l.count); a.entry_off = (int32_t*)(ws + l.entry_off);
  a.tile_off = (int32_t*)(ws + l.tile_off); a.item_off = (int32_t*)(ws + l.item_off);
  a.item_key = (int32_t*)(ws + l.item_key);
  a.cursor = (int32_t*)(ws + l.cursor);
  a.blk_tot = (int32_t*)(ws + l.blk_tot);
  a.entries = (int32_t*)(ws + l.entries);
  a.work_ctr = (int32_t*)(ws + l.work_ctr);
  const size_t nkeys = (size_t)a.BH * a.NW * Mk;
  cudaError_t e = cudaMemsetAsync(a.count, 0, l.work_ctr + 256 - l.count, s);
  if (e != cudaSuccess) { record_cuda_error("inversion memset", e); return PISA_ERR_CUDA; }
  const int use_smem = (2 * (size_t)Mk * 4 <= 96 * 1024) ? 1 : 0;
  const size_t sm_count = use_smem ? (size_t)Mk * 4 : 0, sm_fill = use_smem ? 2 * (size_t)Mk * 4 : 0;
  dim3 grid((g.N + kInvTok - 1) / kInvTok, a.BH);
  if (sm_fill > 48 * 1024) {
    cudaFuncSetAttribute(inv_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_count);
    cudaFuncSetAttribute(inv_fill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_fill);
  }
  inv_count_kernel<<<grid, 256, sm_count, s>>>(a, use_smem);
  int st = check_launch("inv_count");
  if (st != PISA_OK) return st;
  const unsigned nblk = (unsigned)((nkeys + 1023) / 1024);
  inv_scan_blocks_kernel<<<nblk, 1024, 0, s>>>(a);
  st = check_launch("inv_scan_blocks");
  if (st != PISA_OK) return st;
  inv_scan_totals_kernel<<<1, 1024, 0, s>>>(a);
  st = check_launch("inv_scan_totals");
  if (st != PISA_OK) return st;
  inv_scan_fix_kernel<<<nblk, 1024, 0, s>>>(a);
  st = check_launch("inv_scan_fix");
  if (st != PISA_OK) return st;
  inv_fill_kernel<<<grid, 256, sm_fill, s>>>(a, use_smem);
  st = check_launch("inv_fill");
  *out = a;
  return st;
}

template <int D, int NB, bool MOM>
int launch_tile_lse_m(const Geometry& g, const TileArgs& a, int32_t* work_ctr, cudaStream_t s) {
  CUtensorMap tm_k;
  {
    const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.Hkv, (uint64_t)g.N, (uint64_t)g.B};
    const uint32_t box[4] = {64u, 1u, (uint32_t)NB, 1u};
    const uint64_t sk[4] = {2, (uint64_t)g.ks[2] * 2, (uint64_t)g.ks[1] * 2, (uint64_t)g.ks[0] * 2};
    if (!tma::make_map(&tm_k, 2, 4, a.k, dims, sk, box, true)) {
      record_cuda_error("lse_ws tensor map", cudaErrorInvalidValue);
      return PISA_ERR_CUDA;
    }
  }
  const size_t smem = (size_t)(D / 64) * (lse_ws_stages(D, NB) * 128 * 128 + 2 * NB * 128) + 1024;
  cudaError_t e = cudaFuncSetAttribute(lse_ws_kernel<D, NB, MOM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { record_cuda_error("lse_ws attr", e); return PISA_ERR_CUDA; }
  lse_ws_kernel<D, NB, MOM><<<num_sms(), kLseThreads, smem, s>>>(g, a, work_ctr, tm_k);
  return check_launch("lse_ws");
}
template <int D, int NB>
int launch_tile_lse(const Geometry& g, const TileArgs& a, int32_t* work_ctr, cudaStream_t s) {
  return (a.mode == PISA_SCORE_LSE) ? launch_tile_lse_m<D, NB, false>(g, a, work_ctr, s)
                                    : launch_tile_lse_m<D, NB, true>(g, a, work_ctr, s);
}

int dispatch_tile_lse(const Geometry& g, int nb, const TileArgs& a, int32_t* work_ctr, cudaStream_t s) {
  if (g.d == 128) {
    if (nb == 64) return launch_tile_lse<128, 64>(g, a, work_ctr, s);
    if (nb == 128) return launch_tile_lse<128, 128>(g, a, work_ctr, s);
    if (nb == 256) return launch_tile_lse<128, 256>(g, a, work_ctr, s);
  } else if (g.d == 64) {
    if (nb == 64) return launch_tile_lse<64, 64>(g, a, work_ctr, s);
    if (nb == 128) return launch_tile_lse<64, 128>(g, a, work_ctr, s);
    if (nb == 256) return launch_tile_lse<64, 256>(g, a, work_ctr, s);
  }
  return PISA_ERR_UNSUPPORTED;
}

// work_ctr: the launch's next-work-item counter (zero on entry)
template <int D, int C>
int launch_tile_pv(const Geometry& g, const TileArgs& a, int32_t* work_ctr, cudaStream_t s) {
  constexpr int KS = D / 64;
  CUtensorMap tm_k, tm_v;
  {
    const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.Hkv, (uint64_t)g.N, (uint64_t)g.B};
    const uint32_t box[4] = {64u, 1u, (uint32_t)C, 1u};
    const uint64_t sk[4] = {2, (uint64_t)g.ks[2] * 2, (uint64_t)g.ks[1] * 2, (uint64_t)g.ks[0] * 2};
    const uint64_t sv[4] = {2, (uint64_t)g.vs[2] * 2, (uint64_t)g.vs[1] * 2, (uint64_t)g.vs[0] * 2};
    if (!tma::make_map(&tm_k, 2, 4, a.k, dims, sk, box, true) || !tma::make_map(&tm_v, 2, 4, a.v, dims, sv, box, true)) {
      record_cuda_error("pv_ws tensor maps", cudaErrorInvalidValue);
      return PISA_ERR_CUDA;
    }
  }
  constexpr int QP = (KS * 128 * 128 > 128 * 272) ? KS * 128 * 128 : 128 * 272;
  const size_t smem = 4 * (size_t)((QP + 1023) / 1024 * 1024) + 2 * (size_t)KS * C * 128 + 1024;
  cudaError_t e = cudaFuncSetAttribute(pv_ws_kernel<D, C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { record_cuda_error("pv_ws attr", e); return PISA_ERR_CUDA; }
  pv_ws_kernel<D, C><<<num_sms(), kPvThreads, smem, s>>>(g, a, work_ctr, tm_k, tm_v);
  return check_launch("pv_ws");
}

int dispatch_tile_pv(const Geometry& g, const TileArgs& a, int32_t* work_ctr, cudaStream_t s) {
  if (g.d == 128 && g.C == 128) return launch_tile_pv<128, 128>(g, a, work_ctr, s);
  if (g.d == 128 && g.C == 64) return launch_tile_pv<128, 64>(g, a, work_ctr, s);
  if (g.d == 64 && g.C == 128) return launch_tile_pv<64, 128>(g, a, work_ctr, s);
  if (g.d == 64 && g.C == 64) return launch_tile_pv<64, 64>(g, a, work_ctr, s);
  return PISA_ERR_UNSUPPORTED;
}

#include "bsa_bwd_kernel.cuh"

struct BwdLayout { size_t delta, dq, dk, dv, total; InvLayout inv; };
BwdLayout bwd_layout(const Geometry& g) {
  BwdLayout r;
  size_t o = 0;
  r.delta = o; o += align_up((size_t)g.B * g.Hq * g.N * 4, 256);
  r.dq = o; o += align_up((size_t)g.B * g.N * g.Hq * g.d * 4, 256);
  r.dk = o; o += align_up((size_t)g.B * g.N * g.Hkv * g.d * 4, 256);
  r.dv = o; o += align_up((size_t)g.B * g.N * g.Hkv * g.d * 4, 256);
  r.inv = inv_layout(o, g, g.M[1], kBwdWindowTok);
  r.total = r.inv.end;
  return r;
}

template <int C, int DIN>
int launch_bwd(const Geometry& g, const BwdArgs& a, cudaStream_t s) {
  // Q, dO (two pairs when C = 64), P, dS, K, V
  const size_t smem = (C == 64 ? 8 : 4) * (size_t)(128 * 128) + 2 * (size_t)(C / 64) * (128 * 128) +
                      4 * (size_t)(C * 128) + 1024;
  cudaError_t e = cudaFuncSetAttribute(bsa_bwd_kernel<C, DIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { record_cuda_error("bsa_bwd attr", e); return PISA_ERR_CUDA; }
  bsa_bwd_kernel<C, DIN><<<num_sms(), kBwdThreads, smem, s>>>(g, a);
  return check_launch("bsa_bwd");
}

}  // namespace

bool tensor_path_supported(const Geometry& g, int dtype) {
  if (dtype != PISA_BF16) return false;
  if (g.d != 64 && g.d != 128) return false;
  if (g.C != 64 && g.C != 128) return false;
  const int nb = g.g * g.C;
  if (nb != 128 && nb != 256) return false;
  if (g.L < 2 || g.N >= (1 << 24)) return false;
  if ((long long)g.B * g.Hkv * g.N * g.K >= (1LL << 31)) return false;   // entry offsets are int32
  if ((long long)g.B * g.Hkv > 65535) return false;                      // the (b, KV head) unit is a grid's y index
  return true;
}

size_t tensor_route_workspace_bytes(const Geometry& g) { return route_layout(g).total; }
size_t tensor_bsa_workspace_bytes(const Geometry& g) { return bsa_layout(g).total; }

int tensor_route(const Geometry& g, int dtype, const void* q, const void* k, const void* pyramid, int32_t* idx,
                 float* sel_lse, float* margin, float* lse_out, void* ws_, int32_t* status, cudaStream_t s) {
  char* ws = (char*)ws_;
  const RouteLayout L = route_layout(g);
  int32_t* par = (int32_t*)(ws + L.par);
  float* blk = (float*)(ws + L.blk);
  kernel_mark("route_stage1", s);
  int st = route_stage1_mma_supported(g, dtype) ? launch_route_stage1_mma(g, q, pyramid, par, margin, s)
                                                : launch_route_stage1_simt(g, dtype, q, pyramid, par, margin, s);
  if (st != PISA_OK) return st;
  kernel_mark("invert_by_parent", s);
  InvArgs inv;
  st = run_inversion(g, par, g.g, g.M[2], ws, L.inv, &inv, status, s);
  if (st != PISA_OK) return st;
  TileArgs a = {};
  a.q = (const __nv_bfloat16*)q; a.k = (const __nv_bfloat16*)k; a.v = nullptr;
  a.entry_off = inv.entry_off; a.tile_off = inv.tile_off; a.item_off = inv.item_off; a.item_key = inv.item_key; a.entries = inv.entries;
  a.nkeys = g.B * g.Hkv * inv.NW * g.M[2]; a.Mk = g.M[2]; a.NW = inv.NW; a.fan = g.g; a.slots = g.K;
  a.blk_lse = blk; a.status = status; a.mode = g.score_mode; a.debug = g.debug;
  kernel_mark("leaf_lse_tiles", s);
  st = dispatch_tile_lse(g, g.g * g.C, a, inv.work_ctr, s);
  if (st != PISA_OK) return st;
  kernel_mark("final_topk", s);
  // only the LSE scores are also the per-leaf softmax denominators the attention stage can reuse
  const bool lse_scores = g.score_mode == PISA_SCORE_LSE;
  final_topk_kernel<<<dim3((unsigned)((g.N + 3) / 4), (unsigned)(g.B * g.Hkv)), 128, 0, s>>>(
      g, par, blk, idx, margin, lse_scores ? lse_out : nullptr, lse_scores ? sel_lse : nullptr, status);
  st = check_launch("final_topk");
  if (st != PISA_OK || sel_lse == nullptr || lse_scores) return st;
  // the other score modes rank by moments of the logits: the denominators take a pass of their own
  kernel_mark("sel_lse", s);
  return launch_sel_lse_simt(g, dtype, q, k, idx, sel_lse, status, s);
}

int tensor_bsa(const Geometry& g, int dtype, const void* q, const void* k, const void* v, const int32_t* idx,
               const float* sel_lse, void* out, float* lse, bool lse_ready, bool forced_present, void* ws_,
               int32_t* status, cudaStream_t s) {
  (void)dtype;
  char* ws = (char*)ws_;
  const BsaLayout L = bsa_layout(g);
  float* blk = (float*)(ws + L.blk);
  float* acc = (float*)(ws + L.acc);
  kernel_mark("invert_by_leaf", s);
  InvArgs inv;
  // idx that came out of the routing holds every row's forced leaves: those go to the query-major
  // local-window kernel, which also initialises the accumulator (it needs the rows' denominators, so only
  // when the routing handed them over: the block-LSE pass below walks the very lists they are left out of)
  const bool local = forced_present && lse_ready && local_window_supported(g, dtype);
  int st = run_inversion(g, idx, 1, g.M[1], ws, L.inv, &inv, status, s, kWindowTok, local ? 1 : 0);
  if (st != PISA_OK) return st;
  TileArgs a = {};
  a.q = (const __nv_bfloat16*)q; a.k = (const __nv_bfloat16*)k; a.v = (const __nv_bfloat16*)v;
  a.entry_off = inv.entry_off; a.tile_off = inv.tile_off; a.item_off = inv.item_off; a.item_key = inv.item_key; a.entries = inv.entries;
  a.nkeys = g.B * g.Hkv * inv.NW * g.M[1]; a.Mk = g.M[1]; a.NW = inv.NW; a.fan = 1; a.slots = g.K;
  a.blk_lse = blk; a.row_lse = lse; a.o_acc = acc; a.status = status; a.debug = g.debug;
  if (!lse_ready && sel_lse != nullptr) {
    kernel_mark("row_lse", s);
    const long long rows = (long long)g.B * g.Hq * g.N;
    row_lse_from_sel_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, s>>>(g, idx, sel_lse, lse);
    st = check_launch("row_lse_from_sel");
    if (st != PISA_OK) return st;
  } else if (!lse_ready) {
    kernel_mark("block_lse_tiles", s);
    st = dispatch_tile_lse(g, g.C, a, inv.work_ctr, s);
    if (st != PISA_OK) return st;
    const long long rows = (long long)g.B * g.Hkv * g.N * g.G;
    row_lse_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, s>>>(g, idx, blk, lse);
    st = check_launch("row_lse");
    if (st != PISA_OK) return st;
  }
  if (local) {
    kernel_mark("local_window", s);
    st = launch_local_window(g, q, k, v, lse, acc, status, s);
    if (st != PISA_OK) return st;
  } else {
    kernel_mark("accumulator_memset", s);
    cudaError_t e = cudaMemsetAsync(acc, 0, (size_t)g.B * g.N * g.Hq * g.d * 4, s);
    if (e != cudaSuccess) { record_cuda_error("accumulator memset", e); return PISA_ERR_CUDA; }
  }
  kernel_mark("attention_tiles", s);
  st = dispatch_tile_pv(g, a, inv.work_ctr + 1, s);            // the block-LSE pass above, if it ran, used the first counter
  if (st != PISA_OK) return st;
  kernel_mark("convert_out", s);
  if (g.d == 128) {
    const long long n = (long long)g.B * g.N * g.Hkv * (g.d / 2);
    convert_out_heads_inner_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(g, acc, (__nv_bfloat16*)out);
  } else {
    const long long n = (long long)g.B * g.N * g.Hq * (g.d / 8);
    convert_out_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(g, acc, (__nv_bfloat16*)out);
  }
  return check_launch("convert_out");
}

// the backward reads only leaf-level lists: the routing's conditions on g*C and on the depth do not apply
bool tensor_bwd_supported(const Geometry& g, int dtype) {
  if (dtype != PISA_BF16) return false;
  if (g.d != 64 && g.d != 128) return false;
  if (g.C != 64 && g.C != 128) return false;
  if (g.N >= (1 << 24)) return false;
  if ((long long)g.B * g.Hkv * g.N * g.K >= (1LL << 31)) return false;   // entry offsets are int32
  if ((long long)g.B * g.Hkv > 65535) return false;                      // the (b, KV head) unit is a grid's y index
  return true;
}
size_t tensor_bwd_workspace_bytes(const Geometry& g) { return bwd_layout(g).total; }

int tensor_bsa_bwd(const Geometry& g, const void* q, const void* k, const void* v, const int32_t* idx,
                   const void* out, const float* lse, const void* dout, void* dq, void* dk, void* dv,
                   const long long* dq_strides, long long dkv_pitch, void* ws_, int32_t* status, cudaStream_t s) {
  char* ws = (char*)ws_;
  const BwdLayout L = bwd_layout(g);
  kernel_mark("invert_by_leaf", s);
  InvArgs inv;
  int st = run_inversion(g, idx, 1, g.M[1], ws, L.inv, &inv, status, s, kBwdWindowTok);
  if (st != PISA_OK) return st;
  BwdArgs a = {};
  a.q = (const __nv_bfloat16*)q; a.k = (const __nv_bfloat16*)k; a.v = (const __nv_bfloat16*)v;
  a.dout = (const __nv_bfloat16*)dout; a.lse = lse;
  float* delta = (float*)(ws + L.delta);
  a.delta = delta;
  a.entry_off = inv.entry_off; a.item_off = inv.item_off; a.item_key = inv.item_key; a.entries = inv.entries;
  a.nkeys = g.B * g.Hkv * inv.NW * g.M[1]; a.Mk = g.M[1]; a.NW = inv.NW;
  a.dq_acc = (float*)(ws + L.dq); a.dk_acc = (float*)(ws + L.dk); a.dv_acc = (float*)(ws + L.dv);
  a.status = status;
  kernel_mark("gradient_memset", s);
  cudaError_t e = cudaMemsetAsync(ws + L.dq, 0, L.inv.count - L.dq, s);     // dq, dk, dv accumulators are adjacent
  if (e != cudaSuccess) { record_cuda_error("gradient memset", e); return PISA_ERR_CUDA; }
  kernel_mark("delta", s);
  {
    const long long rows = (long long)g.B * g.N * g.Hq;
    bwd_delta_kernel<<<(unsigned)((rows * 32 + 255) / 256), 256, 0, s>>>(g, (const __nv_bfloat16*)out,
                                                                        (const __nv_bfloat16*)dout, delta);
    st = check_launch("bwd_delta");
    if (st != PISA_OK) return st;
  }
  kernel_mark("backward_tiles", s);
  if (g.d == 128) st = (g.C == 128) ? launch_bwd<128, 128>(g, a, s) : launch_bwd<64, 128>(g, a, s);
  else st = (g.C == 128) ? launch_bwd<128, 64>(g, a, s) : launch_bwd<64, 64>(g, a, s);
  if (st != PISA_OK) return st;
  kernel_mark("convert_gradients", s);
  {
    Geometry gd = g;                                   // dq: the caller's dense [B, N, Hq, d] (this chunk's heads of it)
    gd.os[0] = dq_strides[0]; gd.os[1] = dq_strides[1]; gd.os[2] = dq_strides[2];
    const long long n = (long long)g.B * g.N * g.Hkv * (g.d / 2);
    convert_out_heads_inner_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(gd, a.dq_acc, (__nv_bfloat16*)dq);
    st = check_launch("convert_dq");
    if (st != PISA_OK) return st;
    const long long n2 = (long long)g.B * g.N * g.Hkv * g.d / 2;
    const int row2 = g.Hkv * g.d / 2;                 // one token's pairs in the accumulator; dkv_pitch in the output
    bwd_convert_kernel<<<(unsigned)((n2 + 255) / 256), 256, 0, s>>>(a.dk_acc, (__nv_bfloat16*)dk, n2, row2, dkv_pitch / 2);
    bwd_convert_kernel<<<(unsigned)((n2 + 255) / 256), 256, 0, s>>>(a.dv_acc, (__nv_bfloat16*)dv, n2, row2, dkv_pitch / 2);
    st = check_launch("convert_dkv");
  }
  return st;
}

}  // namespace pisa
