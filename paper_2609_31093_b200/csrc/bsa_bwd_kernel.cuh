// Backward of the block-sparse attention with the selected indices held fixed (App. B), d = 128 or 64.
// Included by tensor_path.cu inside its unnamed namespace: it works on the same inverted
// (key block -> tokens) lists, work items and operand layouts as the forward attention kernel.
//
// One CTA per SM, eight warps, no role specialisation: the five products of a tile depend on one
// another through the element-wise step, so a tile is walked in order
//   gather Q, dO rows (cp.async)  ->  S = Q K^T,  dP = dO V^T           (two UMMA chains)
//   P = 2^(S*scale*log2e - lse2),  dS = P o (dP - delta) * scale        (TMEM -> registers -> bf16 in smem)
//   dV^T += dO^T P,  dK^T += Q^T dS,  dQ^T = K^T dS^T                   (three UMMA chains)
//   dQ^T -> fp32 accumulator (vector reductions, heads innermost)
// with dV^T and dK^T ([d lanes] x [C columns] each) staying in TMEM over all the tiles of a work
// item and added to the fp32 key/value gradient accumulators once per item.  All three gradient
// products are issued transposed (M = d = 128) so that C = 64 needs no 64-row UMMA shape and every
// read-out has d along the TMEM lanes: a warp's reduction covers 32 consecutive floats.
// TMEM: S / dQ^T at columns 0..127 (dQ^T reuses S once P and dS are in shared memory), dP at
// 128.., dV^T at 256.., dK^T at 384...  delta = rowsum(dO o O) comes from a small kernel of its own.
// d = 64 runs on the same M = 128 shapes: rows are staged as 128 columns with the upper 64 zero, and only
// the first 64 TMEM lanes of the gradients are read out (half of the tensor work is padding; the kernel is
// bound by its gathers and reductions, not by the tensor pipe).
#pragma once

constexpr int kBwdThreads = 256;

struct BwdArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  const __nv_bfloat16* dout;      // [B, N, Hq, D], strides of `out`
  const float* lse;               // [B, Hq, N] natural log
  const float* delta;             // [B, Hq, N]
  const int32_t* entry_off;
  const int32_t* item_off;
  const int32_t* item_key;
  const int32_t* entries;
  int nkeys, Mk, NW;
  float* dq_acc;                  // [B, Hkv, N, D, G] fp32
  float* dk_acc;                  // [B, N, Hkv, D] fp32
  float* dv_acc;
  int32_t* status;
};

// delta[b, hq, t] = sum_d dO[b,t,hq,d] * O[b,t,hq,d]; one warp per row
__global__ void __launch_bounds__(256) bwd_delta_kernel(Geometry geo, const __nv_bfloat16* __restrict__ out,
                                                        const __nv_bfloat16* __restrict__ dout,
                                                        float* __restrict__ delta) {
  const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const long long rows = (long long)geo.B * geo.N * geo.Hq;
  if (w >= rows) return;
  const int hq = (int)(w % geo.Hq);
  const long long bt = w / geo.Hq;
  const int t = (int)(bt % geo.N), b = (int)(bt / geo.N);
  const long long off = (long long)b * geo.os[0] + (long long)t * geo.os[1] + (long long)hq * geo.os[2];
  float s = 0.f;
  for (int dd = lane; dd < geo.d; dd += 32) s += __bfloat162float(out[off + dd]) * __bfloat162float(dout[off + dd]);
  s = warp_sum(s);
  if (lane == 0) delta[((long long)b * geo.Hq + hq) * geo.N + t] = s;
}

// fp32 -> bf16, contiguous
// fp32 accumulator rows of `row2` element pairs, dense -> bf16 rows `dst_pitch2` pairs apart (a chunk of
// KV heads writes its columns of the caller's [B, N, Hkv, d] tensor)
__global__ void __launch_bounds__(256) bwd_convert_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                          long long n2, int row2, long long dst_pitch2) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n2) return;
  const float2 x = reinterpret_cast<const float2*>(src)[i];
  const long long row = i / row2;
  reinterpret_cast<__nv_bfloat162*>(dst)[row * dst_pitch2 + (i - row * row2)] = __floats2bfloat162_rn(x.x, x.y);
}

// 256 threads copy `nrows` rows of 256 bytes ([row][128 bf16]) into two swizzled K-major slabs of
// `slab_bytes` each; src_of(row) returns the row's address or nullptr (zero fill).
template <int CHV, typename F>                              // CHV: 16-byte chunks a source row really has (d / 8)
__device__ __forceinline__ void bwd_load_rows(uint8_t* dst, int slab_bytes, int nrows, int p, F src_of) {
  const int ck = p & 15, rb = p >> 4;                       // 16-byte chunk of the row, first row
  uint32_t d = smem_u32(dst + (ck >> 3) * slab_bytes) + swz128(rb, ck & 7);
  for (int row = rb; row < nrows; row += 16) {              // row % 8 is the same for all of a thread's rows
    const __nv_bfloat16* src = (ck < CHV) ? src_of(row) : nullptr;
    if (src != nullptr) cp_async16(d, src + ck * 8);
    else st_shared_zero16(d);
    d += 16 * 128;
  }
}

__device__ __forceinline__ ItemInfo item_info_keys(const int32_t* item_key, const int32_t* item_off,
                                                   const int32_t* entry_off, int item, int tpt) {
  ItemInfo r;
  r.key = item_key[item];
  const int local = item - item_off[r.key];
  const int list0 = entry_off[r.key], cnt = entry_off[r.key + 1] - list0;
  const int tiles = (cnt + tpt - 1) / tpt;
  const int first = local * kItemTiles;
  r.ntiles = min(kItemTiles, tiles - first);
  r.e_begin = list0 + first * tpt;
  r.e_end = list0 + cnt;
  return r;
}

template <int C, int DIN>
__global__ void __launch_bounds__(kBwdThreads, 1) bsa_bwd_kernel(Geometry geo, BwdArgs a) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int D = 128;                                    // staged (padded) head dimension
  constexpr int CHV = DIN / 8;
  constexpr int A_SLAB = 128 * 128;                         // one 64-column slab of a 128-row tile
  constexpr int KV_SLAB = C * 128;
  constexpr int P_BYTES = (C / 64) * A_SLAB;
  uint8_t* smem = align1024(smem_raw);
  uint8_t* sQ = smem;
  uint8_t* sdO = sQ + 2 * A_SLAB;
  uint8_t* sP = sdO + 2 * A_SLAB;
  uint8_t* sdS = sP + P_BYTES;
  uint8_t* sK = sdS + P_BYTES;
  uint8_t* sV = sK + 2 * KV_SLAB;
  // C = 64 leaves room for a second pair of Q / dO tiles: the next tile is then gathered under the whole
  // of the current one instead of only under its dQ^T reduction
  constexpr bool DB = (C == 64);
  constexpr int NM = DB ? 3 : 2;                            // metadata buffers: tiles jt, jt+1 (and jt+2)
  uint8_t* sQ1 = sV + 2 * KV_SLAB;
  uint8_t* sdO1 = sQ1 + 2 * A_SLAB;
  __shared__ uint64_t bar_mma;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_fail;
  __shared__ int s_ent2[NM][128];                           // per-tile metadata
  __shared__ float s_nlse22[NM][128], s_delta2[NM][128];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    mbar_init(&bar_mma, 1);
    s_fail = 0;
    mbar_fence_init();
  }
  if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  const int G = geo.G, lgG = 31 - __clz(G), tpt = 128 >> lgG;
  const float sl2 = geo.scale * kLog2e;
  const int n_items = a.item_off[a.nkeys];
  // descriptors: S/dP chains contract over d (K-major operands); the gradient chains contract over the
  // tile rows or the keys with both "row-of-memory = contraction index" operands MN-major
  const uint32_t idesc_s = make_idesc_bf16(128, C, 0, 0);
  const uint32_t idesc_g = make_idesc_bf16(128, C, 1, 1);     // dV^T = dO^T P, dK^T = Q^T dS
  const uint32_t idesc_q = make_idesc_bf16(128, 128, 1, 0);   // dQ^T = K^T dS^T
  uint32_t phase = 0;                                          // completed phases of bar_mma

  const int q4r = warp & 3;                                    // TMEM lane quarter of this warp
  const int row = q4r * 32 + lane;                             // tile row (S, dP) or output column d (gradients)
  const int chalf = warp >> 2;                                 // which half of the columns this warp takes
  const uint32_t lane_sel = (uint32_t)(q4r * 32) << 16;

  bool dead = false;
  for (int item = blockIdx.x; item < n_items && !dead; item += gridDim.x) {
    const ItemInfo inf = item_info_keys(a.item_key, a.item_off, a.entry_off, item, tpt);
    const int bh = inf.key / (a.NW * a.Mk), leaf = inf.key % a.Mk;
    const int b = bh / geo.Hkv, h = bh % geo.Hkv;
    const __nv_bfloat16* kb = a.k + (long long)b * geo.ks[0] + (long long)h * geo.ks[2];
    const __nv_bfloat16* vb = a.v + (long long)b * geo.vs[0] + (long long)h * geo.vs[2];
    bwd_load_rows<CHV>(sK, KV_SLAB, C, tid, [&](int r) {
      const int t = leaf * C + r;
      return (t < geo.N) ? kb + (long long)t * geo.ks[1] : (const __nv_bfloat16*)nullptr;
    });
    bwd_load_rows<CHV>(sV, KV_SLAB, C, tid, [&](int r) {
      const int t = leaf * C + r;
      return (t < geo.N) ? vb + (long long)t * geo.vs[1] : (const __nv_bfloat16*)nullptr;
    });
    const __nv_bfloat16* qb = a.q + (long long)b * geo.qs[0] + (long long)(h * G) * geo.qs[2];
    const __nv_bfloat16* dob = a.dout + (long long)b * geo.os[0] + (long long)(h * G) * geo.os[2];
    // rows of a tile: entry, -lse*log2e and delta per row (threads 0..127, one row each)
    auto load_meta = [&](int jt_, int& ent, float& nl, float& dl) {
      const int e = inf.e_begin + jt_ * tpt + (tid >> lgG);
      ent = (jt_ < inf.ntiles && e < inf.e_end) ? a.entries[e] : -1;
      nl = 0.f; dl = 0.f;
      if (ent >= 0) {
        const long long li = ((long long)b * geo.Hq + h * G + (tid & (G - 1))) * geo.N + (ent & 0xFFFFFF);
        nl = -a.lse[li] * kLog2e;
        dl = a.delta[li];
      }
    };
    auto gather_tile = [&](const int* ents, int buf) {
      bwd_load_rows<CHV>((DB && buf) ? sQ1 : sQ, A_SLAB, 128, tid, [&](int r) {
        const int ent = ents[r];
        return (ent >= 0) ? qb + (long long)(ent & 0xFFFFFF) * geo.qs[1] + (long long)(r & (G - 1)) * geo.qs[2]
                          : (const __nv_bfloat16*)nullptr;
      });
      bwd_load_rows<CHV>((DB && buf) ? sdO1 : sdO, A_SLAB, 128, tid, [&](int r) {
        const int ent = ents[r];
        return (ent >= 0) ? dob + (long long)(ent & 0xFFFFFF) * geo.os[1] + (long long)(r & (G - 1)) * geo.os[2]
                          : (const __nv_bfloat16*)nullptr;
      });
    };
    // first tile of the item: metadata and gathers up front; later tiles are fetched while the previous
    // tile's dQ^T is being reduced
    if (tid < 128) {
      int ent; float nl, dl;
      load_meta(0, ent, nl, dl);
      s_ent2[0][tid] = ent; s_nlse22[0][tid] = nl; s_delta2[0][tid] = dl;
      if (DB) {
        load_meta(1, ent, nl, dl);
        s_ent2[1][tid] = ent; s_nlse22[1][tid] = nl; s_delta2[1][tid] = dl;
      }
    }
    __syncthreads();
    gather_tile(s_ent2[0], 0);
    for (int jt = 0; jt < inf.ntiles && !dead; ++jt) {
      const int cb = jt % NM;                                // this tile's metadata buffer
      const int nb = (jt + NM - 1) % NM;                     // where the metadata fetched during this tile goes
      const int qb_i = DB ? (jt & 1) : 0;                    // this tile's Q / dO pair
      const int* s_ent = s_ent2[cb];
      const float* s_nlse2 = s_nlse22[cb];
      const float* s_delta = s_delta2[cb];
      // metadata of the tile after the one already known: loads issued now, stored once this tile's
      // products are under way
      int n_ent = -1; float n_nl = 0.f, n_dl = 0.f;
      if (tid < 128) load_meta(jt + NM - 1, n_ent, n_nl, n_dl);
      cp_async_wait_all();
      fence_proxy_async_smem();
      __syncthreads();
      // the other Q / dO pair was last read by the previous tile's products, which have completed
      if (DB && jt + 1 < inf.ntiles) gather_tile(s_ent2[(jt + 1) % NM], qb_i ^ 1);
      // ---- S = Q K^T, dP = dO V^T
      if (tid == 0) {
        tcgen05_fence_after_sync();
        const uint32_t q0 = smem_u32(qb_i ? sQ1 : sQ), o0 = smem_u32(qb_i ? sdO1 : sdO), k0 = smem_u32(sK),
                       v0 = smem_u32(sV);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t da = make_smem_desc(q0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
          const uint64_t db = make_smem_desc(k0 + (kk >> 2) * KV_SLAB + (kk & 3) * 32, 0, 1024);
          umma_bf16(tmem, da, db, idesc_s, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t da = make_smem_desc(o0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
          const uint64_t db = make_smem_desc(v0 + (kk >> 2) * KV_SLAB + (kk & 3) * 32, 0, 1024);
          umma_bf16(tmem + 128u, da, db, idesc_s, kk > 0);
        }
        umma_commit(&bar_mma);
      }
      {
        const bool ok = mbar_wait_bounded(&bar_mma, phase & 1u);
        ++phase;
        if (__syncthreads_or(!ok)) { s_fail = 1; dead = true; break; }
      }
      tcgen05_fence_after_sync();
      // ---- P and dS: this warp's 32 rows x C/2 columns, bf16 into the swizzled [row][key] tiles
      {
        const int ent = s_ent[row];
        int ncols = 0;                                        // visible keys of the block for this row
        if (ent >= 0) {
          const int t = ent & 0xFFFFFF, c_t = t / C;
          if (leaf < c_t) ncols = min(C, geo.N - leaf * C);
          else if (leaf == c_t) ncols = t - leaf * C + 1;
        }
        const float nl2 = (ent >= 0) ? s_nlse2[row] : 0.f;
        const float dl = (ent >= 0) ? s_delta[row] : 0.f;
#pragma unroll
        for (int cc = 0; cc < C / 2; cc += 32) {
          const int c0 = chalf * (C / 2) + cc;
          uint32_t rs[32], rp[32];
          tmem_ld_32x32(tmem + lane_sel + (uint32_t)c0, rs);
          tmem_ld_32x32(tmem + lane_sel + 128u + (uint32_t)c0, rp);
          tmem_ld_wait();
          uint32_t pk[16], dk[16];
#pragma unroll
          for (int jx = 0; jx < 16; ++jx) {
            float p0 = (c0 + 2 * jx < ncols) ? ex2_approx(fmaf(__uint_as_float(rs[2 * jx]), sl2, nl2)) : 0.f;
            float p1 = (c0 + 2 * jx + 1 < ncols) ? ex2_approx(fmaf(__uint_as_float(rs[2 * jx + 1]), sl2, nl2)) : 0.f;
            const float d0 = p0 * (__uint_as_float(rp[2 * jx]) - dl) * geo.scale;
            const float d1 = p1 * (__uint_as_float(rp[2 * jx + 1]) - dl) * geo.scale;
            const __nv_bfloat162 pp = __floats2bfloat162_rn(p0, p1);
            const __nv_bfloat162 dd = __floats2bfloat162_rn(d0, d1);
            pk[jx] = *reinterpret_cast<const uint32_t*>(&pp);
            dk[jx] = *reinterpret_cast<const uint32_t*>(&dd);
          }
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int ck = c0 / 8 + q4;
            const uint32_t off = (uint32_t)((ck >> 3) * A_SLAB) + swz128(row, ck & 7);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(sP) + off), "r"(pk[4 * q4]),
                         "r"(pk[4 * q4 + 1]), "r"(pk[4 * q4 + 2]), "r"(pk[4 * q4 + 3])
                         : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(sdS) + off), "r"(dk[4 * q4]),
                         "r"(dk[4 * q4 + 1]), "r"(dk[4 * q4 + 2]), "r"(dk[4 * q4 + 3])
                         : "memory");
          }
        }
      }
      fence_proxy_async_smem();
      tcgen05_fence_before_sync();
      __syncthreads();
      // ---- dV^T += dO^T P,  dK^T += Q^T dS,  dQ^T = K^T dS^T
      if (tid == 0) {
        tcgen05_fence_after_sync();
        const uint32_t q0 = smem_u32(qb_i ? sQ1 : sQ), o0 = smem_u32(qb_i ? sdO1 : sdO), k0 = smem_u32(sK);
        const uint32_t p0 = smem_u32(sP), s0 = smem_u32(sdS);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {                       // contraction over the 128 tile rows
          const uint64_t da = make_smem_desc(o0 + kk * 2048, A_SLAB, 1024);
          const uint64_t db = make_smem_desc(p0 + kk * 2048, A_SLAB, 1024);
          umma_bf16(tmem + 256u, da, db, idesc_g, (jt > 0) || (kk > 0));
        }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t da = make_smem_desc(q0 + kk * 2048, A_SLAB, 1024);
          const uint64_t db = make_smem_desc(s0 + kk * 2048, A_SLAB, 1024);
          umma_bf16(tmem + 384u, da, db, idesc_g, (jt > 0) || (kk > 0));
        }
#pragma unroll
        for (int kk = 0; kk < C / 16; ++kk) {                  // contraction over the block's keys
          const uint64_t da = make_smem_desc(k0 + kk * 2048, KV_SLAB, 1024);
          const uint64_t db = make_smem_desc(s0 + (kk >> 2) * A_SLAB + (kk & 3) * 32, 0, 1024);
          umma_bf16(tmem, da, db, idesc_q, kk > 0);
        }
        umma_commit(&bar_mma);
      }
      {
        const bool ok = mbar_wait_bounded(&bar_mma, phase & 1u);
        ++phase;
        if (__syncthreads_or(!ok)) { s_fail = 1; dead = true; break; }
      }
      tcgen05_fence_after_sync();
      // Q, dO, P, dS tiles are free: (single pair) bring in the next tile while this one's dQ^T is reduced
      if (tid < 128) { s_ent2[nb][tid] = n_ent; s_nlse22[nb][tid] = n_nl; s_delta2[nb][tid] = n_dl; }
      __syncthreads();
      if (!DB && jt + 1 < inf.ntiles) gather_tile(s_ent2[nb], 0);
      // ---- dQ^T out of TMEM: lane = column d, TMEM column = tile row (entry*G + head); this warp's 64 rows
      {
        float* acc_d = a.dq_acc + (((long long)b * geo.Hkv + h) * geo.N) * (long long)(DIN * G) + (long long)row * G;
        const long long tok_stride = (long long)DIN * G;
        const bool live = row < DIN;                          // lanes beyond d hold padding
#pragma unroll
        for (int cc = 0; cc < 64; cc += 32) {
          const int c0 = chalf * 64 + cc;
          uint32_t r[32];
          tmem_ld_32x32(tmem + lane_sel + (uint32_t)c0, r);
          tmem_ld_wait();
          if (G >= 4) {
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) {
              const int col = c0 + 4 * q4;
              const int ent_c = s_ent[col];
              if (ent_c >= 0 && live) {
                float* dst = acc_d + (long long)(ent_c & 0xFFFFFF) * tok_stride + (col & (G - 1));
                asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst),
                             "f"(__uint_as_float(r[4 * q4])), "f"(__uint_as_float(r[4 * q4 + 1])),
                             "f"(__uint_as_float(r[4 * q4 + 2])), "f"(__uint_as_float(r[4 * q4 + 3]))
                             : "memory");
              }
            }
          } else {
#pragma unroll
            for (int q1 = 0; q1 < 32; ++q1) {
              const int col = c0 + q1;
              const int ent_c = s_ent[col];
              if (ent_c >= 0 && live)
                atomicAdd(acc_d + (long long)(ent_c & 0xFFFFFF) * tok_stride + (col & (G - 1)), __uint_as_float(r[q1]));
            }
          }
        }
      }
      tcgen05_fence_before_sync();
      __syncthreads();                                       // tiles and the S / dQ^T columns are free again
    }
    if (dead) break;
    // ---- the item's dV^T and dK^T: lane = column d, TMEM column = key of the block
    {
      tcgen05_fence_after_sync();
#pragma unroll
      for (int cc = 0; cc < C / 2; cc += 32) {
        const int c0 = chalf * (C / 2) + cc;
        uint32_t rv[32], rk[32];
        tmem_ld_32x32(tmem + lane_sel + 256u + (uint32_t)c0, rv);
        tmem_ld_32x32(tmem + lane_sel + 384u + (uint32_t)c0, rk);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int t = leaf * C + c0 + j;
          if (t < geo.N && row < DIN) {
            const long long o = (((long long)b * geo.N + t) * geo.Hkv + h) * DIN + row;
            atomicAdd(a.dv_acc + o, __uint_as_float(rv[j]));
            atomicAdd(a.dk_acc + o, __uint_as_float(rk[j]));
          }
        }
      }
      tcgen05_fence_before_sync();
      __syncthreads();                                       // K, V tiles and the accumulators are free again
    }
  }
  cp_async_wait_all();                                      // nothing of this CTA's copies may outlive it
  tcgen05_fence_before_sync();
  __syncthreads();
  if (s_fail && tid == 0) atomicExch(a.status, (int)PISA_ERR_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, 512);
}
