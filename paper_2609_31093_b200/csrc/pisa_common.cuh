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
  float scale;
  int M[kMaxLevels];               // M[0] = N, M[l] = blocks at level l
  long long span[kMaxLevels];      // span[l] = g^(l-1): leaves under one level-l node
  long long level_off[kMaxLevels]; // element offset of level l in the pyramid buffer
  long long qs[3], ks[3], vs[3], os[3];  // element strides (b, n, h)
};

// Status word at the start of every workspace (device int32[4]; [0] = pisa_status).
constexpr size_t kStatusBytes = 256;

int resolve(const pisa_params_t* p, Geometry* g);                // validates; returns pisa_status
size_t align_up(size_t x, size_t a);

// launchers (each returns a pisa_status; errors come from cudaGetLastError after the launch)
int launch_pyramid(const Geometry& g, int dtype, const void* k, void* pyramid, cudaStream_t s);
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

}  // namespace pisa
