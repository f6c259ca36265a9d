// Internal declarations shared by the libpisa translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pisa.h"

namespace pisa {

constexpr int kMaxLevels = 34;     // ceil(log2(2^31)) + slack
constexpr int kMaxK = 32;          // block budget (one kept node per lane)
constexpr int kMaxCand = 128;      // g*K, candidates per level
constexpr int kWarp = 32;

// Resolved problem description handed to the kernels (by value).
struct Geometry {
  int B, N, Hq, Hkv, G, d, C, g, K, L;
  int score_mode;
  int debug;                       // PISA_DEBUG_* bits
  float scale;
  int M[kMaxLevels];               // M[0] = N, M[l] = blocks at level l
  long long span[kMaxLevels];      // span[l] = g^(l-1): leaves under one level-l node
  long long level_off[kMaxLevels]; // element offset of level l in the pyramid buffer
  long long qs[3], ks[3], vs[3], os[3];  // element strides (b, n, h)
};

// Status word at the start of every workspace (device int32[4]; [0] = pisa_status).
constexpr size_t kStatusBytes = 256;

// Index check of the PISA_DEBUG_BOUNDS mode: true if 0 <= v < n; otherwise records PISA_ERR_BOUNDS in
// the status word (the caller then skips the access).
__device__ __forceinline__ bool bounds_ok(long long v, long long n, int32_t* status) {
  if (v >= 0 && v < n) return true;
  atomicExch(status, (int)PISA_ERR_BOUNDS);
  return false;
}

int resolve(const pisa_params_t* p, Geometry* g);                // validates; returns pisa_status
size_t align_up(size_t x, size_t a);

// launchers (each returns a pisa_status; errors come from cudaGetLastError after the launch)
// status (nullable): the status word a bounded wait reports into
int launch_pyramid(const Geometry& g, int dtype, const void* k, void* pyramid, int32_t* status, cudaStream_t s);
int launch_route_simt(const Geometry& g, int dtype, const void* q, const void* k, const void* pyramid,
                      int32_t* idx, float* margin, cudaStream_t s);
// stage 1 of the two-stage schedule (needs L >= 2): kept level-2 nodes [B,Hkv,N,K] (ascending,
// -1 padded) and the cut margin of the intermediate levels
int launch_route_stage1_simt(const Geometry& g, int dtype, const void* q, const void* pyramid,
                             int32_t* cand_out, float* margin, cudaStream_t s);
// the same stage on warp-level tensor-core MMAs (bf16, LSE score)
bool route_stage1_mma_supported(const Geometry& g, int dtype);
int launch_route_stage1_mma(const Geometry& g, const void* q, const void* pyramid, int32_t* par, float* margin,
                            cudaStream_t s);
int launch_bsa_simt(const Geometry& g, int dtype, const void* q, const void* k, const void* v,
                    const int32_t* idx, void* out, float* lse, cudaStream_t s);
int launch_flat_simt(const Geometry& g, int dtype, const void* q, const void* pyramid, int32_t* idx,
                     cudaStream_t s);
// the same selection on tcgen05 (bf16, d in {64, 128}); status: the workspace's status word
bool flat_tc_supported(const Geometry& g, int dtype);
int launch_flat_tc(const Geometry& g, const void* q, const void* pyramid, int32_t* idx, int32_t* status,
                   cudaStream_t s);
// per-head softmax denominators of the selected leaves, float [B,Hq,N,K] (exact fp32, any shape)
int launch_sel_lse_simt(const Geometry& g, int dtype, const void* q, const void* k, const int32_t* idx,
                        float* sel_lse, int32_t* status, cudaStream_t s);
// one CTA waiting, with a time limit, on a barrier nobody arrives at (self-test of the bounded waits)
int launch_wait_timeout(int32_t* status, unsigned long long limit_ns, cudaStream_t s);
int num_sms();                        // SM count of the current device

// packed variable-length batches run as padded batches: the copies between the two layouts.
// A table names up to kPackSeqs sequences (first token in the packed tensors, length); sequence i of the
// table is batch element b_first + i of the padded tensors [B', g.N, H, d] (g.N = padded length).
constexpr int kPackSeqs = 384;
struct PackTable { int n; int off[kPackSeqs]; int len[kPackSeqs]; };
int launch_pack_gather(const Geometry& g, int elem_bytes, const void* q, const void* k, const void* v, void* q_pad,
                       void* k_pad, void* v_pad, const PackTable& tab, int b_first, cudaStream_t s);
int launch_pack_scatter(const Geometry& g, int elem_bytes, const void* out_pad, const float* lse_pad,
                        const int32_t* idx_pad, void* out, float* lse, int32_t* idx, const PackTable& tab, int b_first,
                        cudaStream_t s);
int launch_pack_gather_bwd(const Geometry& g, int elem_bytes, const void* out, const void* dout, const int32_t* idx,
                           const float* lse, void* out_pad, void* dout_pad, int32_t* idx_pad, float* lse_pad,
                           const PackTable& tab, int b_first, cudaStream_t s);
int launch_pack_scatter_grads(const Geometry& g, int elem_bytes, const void* dq_pad, const void* dk_pad,
                              const void* dv_pad, void* dq, void* dk, void* dv, const PackTable& tab, int b_first,
                              cudaStream_t s);

// decoding step (one token per sequence); ws points past the status word
bool decode_supported(const Geometry& g, int dtype);
size_t decode_workspace_bytes(const Geometry& g);
int launch_decode_step(const Geometry& g, int pos, const void* q, const void* k, const void* v, void* pyramid,
                       int32_t* idx, void* out, float* lse, void* ws, cudaStream_t s);

// with stage timing on, records an event on `s` named after the kernel(s) that follow it
void kernel_mark(const char* name, cudaStream_t s);
int check_launch(const char* what);   // cudaGetLastError -> pisa_status, records the text
void record_cuda_error(const char* what, cudaError_t e);

// ---------------------------------------------------------------- device helpers

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kVec = 4;                       // elements per 16-byte chunk
  __device__ static inline void load_chunk(const float* p, float (&x)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
  __device__ static inline float to_float(float v) { return v; }
  __device__ static inline float from_float(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static inline void load_chunk(const __nv_bfloat16* p, float (&x)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static inline float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
  __device__ static inline __nv_bfloat16 from_float(float v) { return __float2bfloat16_rn(v); }
};

__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------- Select_K ranks (Algorithm 1)
//
// Forced candidates are never scored: they take distinct scores above every real one, ordered by
// position, so that they rank first.  A real score never comes near kForcedFloor.
constexpr float kForcedFloor = 1.0e38f;
__device__ __forceinline__ float forced_score(int pos) { return 3.0e38f - (float)pos * 1.0e34f; }

// Rank of each candidate under (score descending, position ascending), for the candidates
// s = lane + 32*k this lane owns.  `u` is the warp's score array in shared memory, 16-byte aligned,
// n <= kMaxCand scores followed by -inf up to the next multiple of four.  The common case, all
// scores distinct, only counts the strictly larger ones (four per 16-byte load); whether a tie
// exists shows in the sum of the counts (every unordered pair of distinct scores is counted exactly
// once), and only then the exact order with positions is evaluated.
__device__ __forceinline__ void warp_select_ranks(const float* u, int n, int lane, int (&rank)[kMaxCand / 32]) {
  constexpr int SLOTS = kMaxCand / 32;
  float ui[SLOTS];
#pragma unroll
  for (int k = 0; k < SLOTS; ++k) {
    const int s = lane + 32 * k;
    ui[k] = (s < n) ? u[s] : 0.f;
    rank[k] = 0;
  }
  const float4* u4 = reinterpret_cast<const float4*>(u);
  const int n4 = (n + 3) >> 2;
  for (int j4 = 0; j4 < n4; ++j4) {
    const float4 v = u4[j4];
#pragma unroll
    for (int k = 0; k < SLOTS; ++k)
      if (32 * k < n) rank[k] += (int)(v.x > ui[k]) + (int)(v.y > ui[k]) + (int)(v.z > ui[k]) + (int)(v.w > ui[k]);
  }
  int tot = 0;
#pragma unroll
  for (int k = 0; k < SLOTS; ++k)
    if (lane + 32 * k < n) tot += rank[k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
  if (tot != n * (n - 1) / 2) {
#pragma unroll
    for (int k = 0; k < SLOTS; ++k) {
      const int s = lane + 32 * k;
      if (s < n) {
        int r = 0;
        for (int j = 0; j < n; ++j) {
          const float uj = u[j];
          r += (uj > ui[k]) || (uj == ui[k] && j < s);
        }
        rank[k] = r;
      }
    }
  }
}

// Select_K for at most 64 candidates (two per lane: s = lane and lane + 32) without ranks: a bitonic
// network sorts the 64 scores across the warp (padding = -inf), the K-th largest is the threshold, and
// a candidate is kept if its score is larger, or equal with few enough equal ones before it (ties go to
// the smaller position, as the ranks do).  u0 / u1: the scores of this lane's candidates (-inf beyond n).
// Needs n > K.  cut_k / cut_k1: the K-th and (K+1)-th largest scores (the cut margin is their gap).
__device__ __forceinline__ void warp_select_sorted64(float u0, float u1, int K, int lane, bool& keep0, bool& keep1,
                                                     float& cut_k, float& cut_k1) {
  float v0 = u0, v1 = u1;                      // element e = lane + 32 * k; sorted ascending by e
#pragma unroll
  for (int size = 2; size <= 64; size <<= 1) {
#pragma unroll
    for (int j = size >> 1; j > 0; j >>= 1) {
      if (j == 32) {                           // partner = the lane's other element; the last merge is ascending
        const float lo = fminf(v0, v1), hi = fmaxf(v0, v1);
        v0 = lo; v1 = hi;
      } else {
        const float o0 = __shfl_xor_sync(0xffffffffu, v0, j), o1 = __shfl_xor_sync(0xffffffffu, v1, j);
        const bool lower = (lane & j) == 0;
        // ascending block when bit `size` of e is clear: a lane bit below 32, the element bit at 32, none at 64
        const bool asc0 = (size < 32) ? ((lane & size) == 0) : true;
        const bool asc1 = (size < 32) ? ((lane & size) == 0) : (size == 64);
        v0 = (lower == asc0) ? fminf(v0, o0) : fmaxf(v0, o0);
        v1 = (lower == asc1) ? fminf(v1, o1) : fmaxf(v1, o1);
      }
    }
  }
  // position p of the sorted order sits in lane p & 31, element p >> 5; K-th largest = position 64 - K
  const int pk = 64 - K, pk1 = pk - 1;
  const float a0 = __shfl_sync(0xffffffffu, v0, pk & 31), a1 = __shfl_sync(0xffffffffu, v1, pk & 31);
  const float b0 = __shfl_sync(0xffffffffu, v0, pk1 & 31), b1 = __shfl_sync(0xffffffffu, v1, pk1 & 31);
  cut_k = (pk >> 5) ? a1 : a0;
  cut_k1 = (pk1 >> 5) ? b1 : b0;
  const float T = cut_k;
  const unsigned gt0 = __ballot_sync(0xffffffffu, u0 > T), gt1 = __ballot_sync(0xffffffffu, u1 > T);
  const unsigned eq0 = __ballot_sync(0xffffffffu, u0 == T), eq1 = __ballot_sync(0xffffffffu, u1 == T);
  const int room = K - __popc(gt0) - __popc(gt1);                       // equal ones still to keep (>= 1)
  const unsigned lt = (1u << lane) - 1u;
  keep0 = (u0 > T) || ((u0 == T) && __popc(eq0 & lt) < room);
  keep1 = (u1 > T) || ((u1 == T) && __popc(eq0) + __popc(eq1 & lt) < room);
}

}  // namespace pisa
