// Warp-level m16n8k16 building blocks shared by the per-token routing kernels (prefill stage 1 and
// the decoding step): the group's query heads as the B operand held in registers, rows of a
// [rows][D] bf16 matrix (child summaries or raw keys) as the A operand loaded straight from
// global memory into fragment registers.
//
// Both operands permute the contraction index identically so that a lane's fragment pieces are
// contiguous 16-byte chunks in memory: lane (gid = lane/4, tig = lane%4) loads, for every group c4 of
// 32 elements, chunk (c4*4 + tig) of its row; the two MMAs per group pair the chunk's halves.
#pragma once

#include <math_constants.h>

#include "pisa_common.cuh"

namespace pisa {
namespace frag {

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg128(const void* p) { return *reinterpret_cast<const uint4*>(p); }

// 32 bytes per lane in one load (sm_100): four lanes then cover a whole 128-byte line of a row, half the
// L1 wavefronts per byte of the 16-byte form.  `p` must be 32-byte aligned.
struct U32x8 { uint32_t r[8]; };
__device__ __forceinline__ U32x8 ldg256(const void* p) {
  U32x8 v;
  asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3]), "=r"(v.r[4]), "=r"(v.r[5]), "=r"(v.r[6]),
                 "=r"(v.r[7])
               : "l"(p));
  return v;
}

// running (max, sum exp) of a stream of logits
__device__ __forceinline__ void lse_add(float& m, float& s, float z) {
  const float mn = fmaxf(m, z);
  s = s * __expf(m - mn) + __expf(z - mn);
  m = mn;
}
// merge of two running (max, sum exp) pairs; an empty stream is (-inf, 0)
__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  if (mn > -CUDART_INF_F) s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
  m = mn;
}

// B fragments of the group's query heads: column n = gid of head tile nt is head nt*8 + gid
// (zero beyond G).  `row0` points at head 0 of the group, heads `head_stride` elements apart.
template <int D, int NT>
struct QFrag {
  uint32_t r[NT][D / 32][4];
  __device__ __forceinline__ void load(const __nv_bfloat16* row0, long long head_stride, int G, int lane) {
    const int gid = lane >> 2, tig = lane & 3;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int head = nt * 8 + gid;
#pragma unroll
      for (int c4 = 0; c4 < D / 32; ++c4) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (head < G) v = ldg128(row0 + (long long)head * head_stride + (c4 * 4 + tig) * 8);
        r[nt][c4][0] = v.x; r[nt][c4][1] = v.y; r[nt][c4][2] = v.z; r[nt][c4][3] = v.w;
      }
    }
  }
};

// Dot products of two rows with the group's heads.  Fragment row gid is `lo`, row gid + 8 is `hi`
// (null = absent: zeros).  z[nt][0..1] = lo . heads nt*8 + 2*tig + {0,1}; z[nt][2..3] = hi . same heads.
template <int D, int NT>
__device__ __forceinline__ void rows2_dot(const QFrag<D, NT>& q, const __nv_bfloat16* lo, const __nv_bfloat16* hi,
                                          int lane, float (&z)[NT][4]) {
  const int tig = lane & 3;
  uint4 a[D / 32], b[D / 32];
#pragma unroll
  for (int c4 = 0; c4 < D / 32; ++c4) {
    a[c4] = lo ? ldg128(lo + (c4 * 4 + tig) * 8) : make_uint4(0u, 0u, 0u, 0u);
    b[c4] = hi ? ldg128(hi + (c4 * 4 + tig) * 8) : make_uint4(0u, 0u, 0u, 0u);
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    z[nt][0] = z[nt][1] = z[nt][2] = z[nt][3] = 0.f;
#pragma unroll
    for (int c4 = 0; c4 < D / 32; ++c4) {
      mma_bf16_16816(z[nt], a[c4].x, b[c4].x, a[c4].y, b[c4].y, q.r[nt][c4][0], q.r[nt][c4][1]);
      mma_bf16_16816(z[nt], a[c4].z, b[c4].z, a[c4].w, b[c4].w, q.r[nt][c4][2], q.r[nt][c4][3]);
    }
  }
}

// The same dot products with the loads split from the arithmetic, so that a caller can put the loads
// of several row pairs in flight before the first MMA waits on any of them.
template <int D>
struct RowPair {
  uint4 a[D / 32], b[D / 32];
  __device__ __forceinline__ void load(const __nv_bfloat16* lo, const __nv_bfloat16* hi, int lane) {
    const int tig = lane & 3;
#pragma unroll
    for (int c4 = 0; c4 < D / 32; ++c4) {
      a[c4] = lo ? ldg128(lo + (c4 * 4 + tig) * 8) : make_uint4(0u, 0u, 0u, 0u);
      b[c4] = hi ? ldg128(hi + (c4 * 4 + tig) * 8) : make_uint4(0u, 0u, 0u, 0u);
    }
  }
};
template <int D, int NT>
__device__ __forceinline__ void rows2_dot(const QFrag<D, NT>& q, const RowPair<D>& r, float (&z)[NT][4]) {
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    z[nt][0] = z[nt][1] = z[nt][2] = z[nt][3] = 0.f;
#pragma unroll
    for (int c4 = 0; c4 < D / 32; ++c4) {
      mma_bf16_16816(z[nt], r.a[c4].x, r.b[c4].x, r.a[c4].y, r.b[c4].y, q.r[nt][c4][0], q.r[nt][c4][1]);
      mma_bf16_16816(z[nt], r.a[c4].z, r.b[c4].z, r.a[c4].w, r.b[c4].w, q.r[nt][c4][2], q.r[nt][c4][3]);
    }
  }
}

}  // namespace frag
}  // namespace pisa
