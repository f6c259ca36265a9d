// Attention over the forced leaves, query-major (App. B "Causal masking": the first, the previous and the
// current leaf are kept for every query).
//
// These three blocks are the one part of a row's selection that its neighbours share: all tokens of leaf
// c attend to leaves {0, c-1, c}.  Their queries are contiguous in q, so instead of going through the
// inverted lists (one gathered query row and one fp32 reduction row per (token, block) pair) they are
// served as dense tiles:
//   work item = (b, KV head, leaf c, tile of 128 / G tokens of that leaf) = one 128-row A tile
//               (row = token * G + head), loaded with one 4-D TMA tile load per 64-wide K slab;
//   per forced block: K and V slabs by TMA tile loads (this GPU's memory, no multicast),
//               S = Q K^T (tcgen05, TMEM) -> P = 2^(S * scale * log2e - lse_row) in bf16 (the row's
//               denominator is known from the routing, so P is final: no running maximum), causal
//               mask only inside the current leaf -> O^T += V^T P^T (d = 128; O += P V with d = 64: a 64-row
//               accumulator has another TMEM layout) accumulated in TMEM over the blocks;
//   result    = the fp32 accumulator rows of these tokens are STORED (not added): this kernel initialises
//               the accumulator the list-driven attention kernel then adds the routed blocks into, so
//               no memset is needed and the routed kernel never sees a masked block.
// Roles: warp 0 TMA producer, warps 1 and 2 UMMA issuers (first / second products), warps 4-7 and 8-11 two
// softmax / read-out groups taking alternate blocks.  Every wait is bounded.
#include <math_constants.h>

#include "pisa_common.cuh"
#include "tc_utils.cuh"
#include "tma_map.cuh"

namespace pisa {

using namespace tc;

namespace {

constexpr int kLocalThreads = 384;        // TMA warp, two UMMA issuers, (one idle), two softmax / read-out groups of four warps
constexpr float kLog2eL = 1.4426950408889634f;

struct LocalArgs {
  const float* row_lse;    // [B, Hq, N] natural log
  float* o_acc;            // fp32: [B, Hkv, N, 128, G] for d = 128, [B, N, Hq, 64] for d = 64 (the layouts of pv_ws)
  int32_t* status;
  int tiles_per_leaf;      // C / (128 / G)
  int n_items;             // B * Hkv * M1 * tiles_per_leaf
};

__device__ __forceinline__ float ex2l(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct LocalItem { int b, h, c, tile, nb, blk[3]; };
__device__ __forceinline__ LocalItem local_item(const Geometry& geo, const LocalArgs& a, int item) {
  LocalItem r;
  r.tile = item % a.tiles_per_leaf;
  int x = item / a.tiles_per_leaf;
  r.c = x % geo.M[1];
  x /= geo.M[1];
  r.h = x % geo.Hkv;
  r.b = x / geo.Hkv;
  r.nb = 0;
  r.blk[r.nb++] = 0;
  if (r.c >= 2) r.blk[r.nb++] = r.c - 1;
  if (r.c >= 1) r.blk[r.nb++] = r.c;
  return r;
}

}  // namespace

// C: leaf size (64 or 128); D: head dimension (64 or 128).
template <int C, int D>
__global__ void __launch_bounds__(kLocalThreads, 1)
local_window_kernel(Geometry geo, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, LocalArgs a) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int KS = D / 64;
  constexpr bool kTransO = (D == 128);
  constexpr int A_SLAB = 128 * 128, KV_SLAB = C * 128;
  constexpr int Q_BYTES = KS * A_SLAB, KV_BYTES = KS * KV_SLAB, P_BYTES = (C / 64) * A_SLAB;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // One query tile (it is free once the item's last S has been computed, well before the item ends, so the next
  // one loads under the remaining products) and TWO P tiles: the softmax of block j + 1 runs while P(j) V(j) does.
  uint8_t* sQ = smem;                      // [Q_BYTES]
  uint8_t* sK = sQ + Q_BYTES;              // [2][KV_BYTES]
  uint8_t* sV = sK + 2 * KV_BYTES;         // [2][KV_BYTES]
  uint8_t* sP = sV + 2 * KV_BYTES;         // [2][P_BYTES]
  __shared__ uint64_t q_full, q_empty, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], s_empty[2],
      p_full[2], p_empty[2], o_full, o_empty;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_fail;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
      mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 4);
      mbar_init(&p_full[i], 4); mbar_init(&p_empty[i], 1);
    }
    mbar_init(&q_full, 1); mbar_init(&q_empty, 1);
    mbar_init(&o_full, 1); mbar_init(&o_empty, 8);
    s_fail = 0;
    mbar_fence_init();
  }
  if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem = tmem_slot;         // S buffers at columns 0 / 128, O^T at 256
  const int G = geo.G, lgG = 31 - __clz(G), tpt = 128 >> lgG;

  if (warp == 0) {
    // ------------------------------------------------ TMA producer (one thread)
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v);
      int it = 0, kv = 0;                  // items and (item, block) steps of this CTA
      for (int item = blockIdx.x; item < a.n_items && !s_fail; item += gridDim.x, ++it) {
        const LocalItem w = local_item(geo, a, item);
        if (it >= 1 && !mbar_wait_bounded(&q_empty, (uint32_t)((it - 1) & 1))) { s_fail = 1; break; }
        mbar_arrive_expect_tx(&q_full, (uint32_t)Q_BYTES);
        for (int ks = 0; ks < KS; ++ks)
          tma_load_4d(smem_u32(sQ + ks * A_SLAB), &tm_q, &q_full, ks * 64, w.h * G, w.c * C + w.tile * tpt, w.b);
        for (int j = 0; j < w.nb; ++j, ++kv) {
          const int s = kv & 1;
          if (kv >= 2 && !mbar_wait_bounded(&k_empty[s], (uint32_t)(((kv >> 1) - 1) & 1))) { s_fail = 1; break; }
          mbar_arrive_expect_tx(&k_full[s], (uint32_t)KV_BYTES);
          for (int ks = 0; ks < KS; ++ks)
            tma_load_4d(smem_u32(sK + s * KV_BYTES + ks * KV_SLAB), &tm_k, &k_full[s], ks * 64, w.h, w.blk[j] * C, w.b);
          if (kv >= 2 && !mbar_wait_bounded(&v_empty[s], (uint32_t)(((kv >> 1) - 1) & 1))) { s_fail = 1; break; }
          mbar_arrive_expect_tx(&v_full[s], (uint32_t)KV_BYTES);
          for (int ks = 0; ks < KS; ++ks)
            tma_load_4d(smem_u32(sV + s * KV_BYTES + ks * KV_SLAB), &tm_v, &v_full[s], ks * 64, w.h, w.blk[j] * C, w.b);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ UMMA issuer of the first products, S = Q K^T
    // (its own warp: an issue blocks while the tensor pipe works its queue off, and the two kinds of product
    // wait for different things -- S for keys and a free S buffer, P V for the softmax)
    const uint32_t idesc_s = make_idesc_bf16(128, C, 0, 0);
    int it = 0, kv = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < a.n_items && ok && !s_fail; item += gridDim.x, ++it) {
      const LocalItem w = local_item(geo, a, item);
      ok = mbar_wait_bounded(&q_full, (uint32_t)(it & 1));
      for (int j = 0; j < w.nb && ok; ++j) {
        const int kvj = kv + j, s = kvj & 1;
        ok = mbar_wait_bounded(&k_full[s], (uint32_t)((kvj >> 1) & 1));
        if (ok && kvj >= 2) ok = mbar_wait_bounded(&s_empty[s], (uint32_t)(((kvj >> 1) - 1) & 1));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) {
          tcgen05_fence_after_sync();
          const uint32_t q0 = smem_u32(sQ), k0 = smem_u32(sK + s * KV_BYTES);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t da = make_smem_desc(q0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
            const uint64_t db = make_smem_desc(k0 + (kk >> 2) * KV_SLAB + (kk & 3) * 32, 0, 1024);
            umma_bf16(tmem + (uint32_t)(s * 128), da, db, idesc_s, kk > 0);
          }
          umma_commit(&s_full[s]);
          umma_commit(&k_empty[s]);
          if (j == w.nb - 1) umma_commit(&q_empty);          // every S of this item has been issued
        }
        __syncwarp();
      }
      kv += w.nb;
    }
    if (!ok) s_fail = 1;
  } else if (warp == 2) {
    // ------------------------------------------------ UMMA issuer of the second products, O^T += V^T P^T
    const uint32_t idesc_ot = make_idesc_bf16(128, 128, 1, 0);     // O^T: M = d (V, MN-major), N = tile rows (P)
    const uint32_t idesc_o = make_idesc_bf16(128, D, 0, 1);        // O: M = tile rows (P), N = d (V, MN-major)
    int it = 0, kv = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < a.n_items && ok && !s_fail; item += gridDim.x, ++it) {
      const LocalItem w = local_item(geo, a, item);
      for (int j = 0; j < w.nb && ok; ++j) {
        const int kvj = kv + j, s = kvj & 1;
        ok = mbar_wait_bounded(&p_full[s], (uint32_t)((kvj >> 1) & 1));
        if (ok) ok = mbar_wait_bounded(&v_full[s], (uint32_t)((kvj >> 1) & 1));
        if (ok && j == 0 && it >= 1) ok = mbar_wait_bounded(&o_empty, (uint32_t)((it - 1) & 1));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) {
          tcgen05_fence_after_sync();
          const uint32_t p0 = smem_u32(sP + s * P_BYTES), v0 = smem_u32(sV + s * KV_BYTES);
#pragma unroll
          for (int kk = 0; kk < C / 16; ++kk) {
            const uint64_t dp = make_smem_desc(p0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
            const uint64_t dv = make_smem_desc(v0 + kk * (16 * 128), KV_SLAB, 1024);
            if (kTransO) umma_bf16(tmem + 256u, dv, dp, idesc_ot, (j > 0 || kk > 0) ? 1u : 0u);
            else umma_bf16(tmem + 256u, dp, dv, idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(&p_empty[s]);
          umma_commit(&v_empty[s]);
          if (j == w.nb - 1) umma_commit(&o_full);
        }
        __syncwarp();
      }
      kv += w.nb;
    }
    if (!ok) s_fail = 1;
  } else if (warp >= 4) {
    // ------------------------------------------------ softmax and read-out warps (TMEM lane quarter = warp % 4)
    // Two groups of four: a group takes every other (item, block) step -- S buffer, P buffer and barriers of
    // its parity -- so that two warps per SM sub-partition overlap their exponentials and TMEM waits; both
    // read the item's accumulator out, half of its columns each.
    const int grp = (warp - 4) >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;             // S: tile row = token * G + head;  O^T: output column d
    const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
    const float sl2 = geo.scale * kLog2eL;
    int it = 0, kv = 0;
    bool ok = true;
    // the row's softmax denominator is fetched one item ahead (the load would otherwise open every item)
    auto row_lse_of = [&](int item) -> float {
      if (item >= a.n_items) return 0.f;
      const LocalItem x = local_item(geo, a, item);
      const int tx = x.c * C + x.tile * tpt + (row >> lgG);
      return (tx < geo.N) ? a.row_lse[((long long)x.b * geo.Hq + x.h * G + (row & (G - 1))) * geo.N + tx] : 0.f;
    };
    float lse_next = row_lse_of((int)blockIdx.x);
    for (int item = blockIdx.x; item < a.n_items && ok && !s_fail; item += gridDim.x, ++it) {
      const LocalItem w = local_item(geo, a, item);
      const int t0 = w.c * C + w.tile * tpt;         // first token of the tile
      const int t = t0 + (row >> lgG);
      const bool live = t < geo.N;
      const float neg_lse2 = -lse_next * kLog2eL;
      lse_next = row_lse_of(item + (int)gridDim.x);
      for (int j = 0; j < w.nb && ok; ++j, ++kv) {
        const int s = kv & 1;
        if (s != grp) continue;
        // visible keys of this block for this row: all of an earlier leaf, keys <= t of the row's own leaf
        const int ncols = !live ? 0 : ((w.blk[j] == w.c) ? (t - w.c * C + 1) : C);
        ok = mbar_wait_bounded(&s_full[s], (uint32_t)((kv >> 1) & 1));
        if (ok && kv >= 2) ok = mbar_wait_bounded(&p_empty[s], (uint32_t)(((kv >> 1) - 1) & 1));
        if (!ok) break;
        tcgen05_fence_after_sync();
        const uint32_t s_base = tmem + lane_sel + (uint32_t)(s * 128);
        const bool fast = __all_sync(0xffffffffu, ncols == C);     // no masked column in this warp's rows
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
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_empty[s]);     // S has been read out
          }
          uint32_t pk[16];
#pragma unroll
          for (int jx = 0; jx < 16; ++jx) {
            float p0 = ex2l(fmaf(__uint_as_float(cur[2 * jx]), sl2, neg_lse2));
            float p1 = ex2l(fmaf(__uint_as_float(cur[2 * jx + 1]), sl2, neg_lse2));
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
            const uint32_t dst = smem_u32(sP + s * P_BYTES + (ck >> 3) * A_SLAB) + swz128(row, ck & 7);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * q4]), "r"(pk[4 * q4 + 1]),
                         "r"(pk[4 * q4 + 2]), "r"(pk[4 * q4 + 3])
                         : "memory");
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[s]);
      }
      if (!ok) break;
      // read-out: lane = output column d, TMEM column = tile row; the G heads of a token are G consecutive columns
      ok = mbar_wait_bounded(&o_full, (uint32_t)(it & 1));
      if (!ok) break;
      tcgen05_fence_after_sync();
      const uint32_t o_base = tmem + lane_sel + 256u;
      if constexpr (kTransO) {
        // lane = output column d, TMEM column = tile row; the G heads of a token are G consecutive columns of
        // the heads-innermost accumulator [B, Hkv, N, d, G]; each group reads half of the columns
        float* acc_d = a.o_acc + (((long long)w.b * geo.Hkv + w.h) * geo.N) * (long long)(D * G) + (long long)row * G;
        const long long tok_stride = (long long)D * G;
        uint32_t ra[32], rb[32];
        const int cbeg = grp * 64;
        tmem_ld_32x32(o_base + (uint32_t)cbeg, ra);
#pragma unroll
        for (int cc = 0; cc < 64; cc += 32) {
          const int c0 = cbeg + cc;
          uint32_t (&cur)[32] = ((cc >> 5) & 1) ? rb : ra;
          uint32_t (&nxt)[32] = ((cc >> 5) & 1) ? ra : rb;
          tmem_ld_wait();
          if (cc + 32 < 64) {
            tmem_ld_32x32(o_base + (uint32_t)(c0 + 32), nxt);
          } else {
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_empty);          // O has been read out of TMEM
          }
          if (G >= 4) {
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) {
              const int col = c0 + 4 * q4;
              const int tt = t0 + (col >> lgG);
              if (tt < geo.N)
                *reinterpret_cast<float4*>(acc_d + (long long)tt * tok_stride + (col & (G - 1))) =
                    make_float4(__uint_as_float(cur[4 * q4]), __uint_as_float(cur[4 * q4 + 1]),
                                __uint_as_float(cur[4 * q4 + 2]), __uint_as_float(cur[4 * q4 + 3]));
            }
          } else {
#pragma unroll
            for (int q1 = 0; q1 < 32; ++q1) {
              const int col = c0 + q1;
              const int tt = t0 + (col >> lgG);
              if (tt < geo.N) acc_d[(long long)tt * tok_stride + (col & (G - 1))] = __uint_as_float(cur[q1]);
            }
          }
        }
      } else {
        // lane = tile row (token, head), TMEM column = output column d; the token-major accumulator
        // [B, N, Hq, d]; each group stores half of the row's columns (D / 2 = 32)
        static_assert(D == 64, "the direct read-out is written for d = 64");
        uint32_t ra[32];
        tmem_ld_32x32(o_base + (uint32_t)(grp * 32), ra);
        tmem_ld_wait();
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&o_empty);              // O has been read out of TMEM
        if (live) {
          float* dst = a.o_acc + (((long long)w.b * geo.N + t) * geo.Hq + w.h * G + (row & (G - 1))) * D + grp * 32;
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            *reinterpret_cast<float4*>(dst + 4 * q4) =
                make_float4(__uint_as_float(ra[4 * q4]), __uint_as_float(ra[4 * q4 + 1]), __uint_as_float(ra[4 * q4 + 2]),
                            __uint_as_float(ra[4 * q4 + 3]));
        }
      }
    }
    if (!ok) s_fail = 1;
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (s_fail && tid == 0) atomicExch(a.status, (int)PISA_ERR_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, 512);
}

bool local_window_supported(const Geometry& g, int dtype) {
  if (dtype != PISA_BF16 || (g.d != 128 && g.d != 64)) return false;
  if (g.C != 64 && g.C != 128) return false;
  const int tpt = 128 / g.G;
  if (g.G > 16 || g.C % tpt != 0) return false;
  for (int i = 0; i < 3; ++i)
    if ((g.qs[i] * 2) % 16 || (g.ks[i] * 2) % 16 || (g.vs[i] * 2) % 16) return false;
  return tma::encoder() != nullptr;
}

template <int C, int D>
static int launch_local_c(const Geometry& g, const void* q, const void* k, const void* v, const float* row_lse,
                          float* o_acc, int32_t* status, cudaStream_t s) {
  const int tpt = 128 / g.G;
  LocalArgs a;
  a.row_lse = row_lse; a.o_acc = o_acc; a.status = status;
  a.tiles_per_leaf = g.C / tpt;
  const long long items = (long long)g.B * g.Hkv * g.M[1] * a.tiles_per_leaf;
  if (items > 0x7fffffffLL) return PISA_ERR_UNSUPPORTED;
  a.n_items = (int)items;
  CUtensorMap tm_q, tm_k, tm_v;
  {
    const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.Hq, (uint64_t)g.N, (uint64_t)g.B};
    const uint64_t str[4] = {2, (uint64_t)g.qs[2] * 2, (uint64_t)g.qs[1] * 2, (uint64_t)g.qs[0] * 2};
    const uint32_t box[4] = {64u, (uint32_t)g.G, (uint32_t)tpt, 1u};
    if (!tma::make_map(&tm_q, 2, 4, q, dims, str, box, true)) return PISA_ERR_UNSUPPORTED;
  }
  {
    const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.Hkv, (uint64_t)g.N, (uint64_t)g.B};
    const uint32_t box[4] = {64u, 1u, (uint32_t)C, 1u};
    const uint64_t sk[4] = {2, (uint64_t)g.ks[2] * 2, (uint64_t)g.ks[1] * 2, (uint64_t)g.ks[0] * 2};
    const uint64_t sv[4] = {2, (uint64_t)g.vs[2] * 2, (uint64_t)g.vs[1] * 2, (uint64_t)g.vs[0] * 2};
    if (!tma::make_map(&tm_k, 2, 4, k, dims, sk, box, true)) return PISA_ERR_UNSUPPORTED;
    if (!tma::make_map(&tm_v, 2, 4, v, dims, sv, box, true)) return PISA_ERR_UNSUPPORTED;
  }
  const size_t smem = (size_t)(D / 64) * ((size_t)(128 * 128) + 4 * (size_t)(C * 128)) + 2 * (size_t)(C / 64) * 128 * 128 + 1024;
  cudaError_t e = cudaFuncSetAttribute(local_window_kernel<C, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { record_cuda_error("local_window attr", e); return PISA_ERR_CUDA; }
  const int grid = a.n_items < num_sms() ? a.n_items : num_sms();
  local_window_kernel<C, D><<<grid, kLocalThreads, smem, s>>>(g, tm_q, tm_k, tm_v, a);
  return check_launch("local_window");
}

int launch_local_window(const Geometry& g, const void* q, const void* k, const void* v, const float* row_lse,
                        float* o_acc, int32_t* status, cudaStream_t s) {
  if (g.d == 128) {
    if (g.C == 128) return launch_local_c<128, 128>(g, q, k, v, row_lse, o_acc, status, s);
    return launch_local_c<64, 128>(g, q, k, v, row_lse, o_acc, status, s);
  }
  if (g.C == 128) return launch_local_c<128, 64>(g, q, k, v, row_lse, o_acc, status, s);
  return launch_local_c<64, 64>(g, q, k, v, row_lse, o_acc, status, s);
}

}  // namespace pisa
