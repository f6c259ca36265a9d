// Tensor-core (tcgen05 / TMEM) path: key-block-major leaf scoring and block-sparse attention.
#pragma once

#include "pisa_common.cuh"

namespace pisa {

bool tensor_path_supported(const Geometry& g, int dtype);
size_t tensor_route_workspace_bytes(const Geometry& g);
size_t tensor_bsa_workspace_bytes(const Geometry& g);
// ws points past the status word; status is the workspace's status word
// lse_out (nullable): softmax denominators of the kept leaves, float [B,Hq,N]
// sel_lse (nullable): per-head denominators of the kept leaves, float [B,Hq,N,K]
int tensor_route(const Geometry& g, int dtype, const void* q, const void* k, const void* pyramid, int32_t* idx,
                 float* sel_lse, float* margin, float* lse_out, void* ws, int32_t* status, cudaStream_t s);
// lse_ready: `lse` already holds the denominators of exactly these idx (as tensor_route writes them)
// sel_lse (nullable): per-block denominators of exactly these idx (as tensor_route writes them); used when
// lse_ready is false to skip the block-LSE pass
// forced_present: idx comes from the routing, i.e. every row holds its forced leaves (0, c-1, c): they are then
// served by the query-major local-window kernel instead of the lists
int tensor_bsa(const Geometry& g, int dtype, const void* q, const void* k, const void* v, const int32_t* idx,
               const float* sel_lse, void* out, float* lse, bool lse_ready, bool forced_present, void* ws,
               int32_t* status, cudaStream_t s);

// attention over the forced leaves, query-major (local_window.cu); stores the fp32 accumulator [B,Hkv,N,128,G]
bool local_window_supported(const Geometry& g, int dtype);
int launch_local_window(const Geometry& g, const void* q, const void* k, const void* v, const float* row_lse,
                        float* o_acc, int32_t* status, cudaStream_t s);

// backward of the block-sparse attention with frozen indices; dq [B,N,Hq,d], dk, dv [B,N,Hkv,d] dense
bool tensor_bwd_supported(const Geometry& g, int dtype);
size_t tensor_bwd_workspace_bytes(const Geometry& g);
// dq_strides: element strides (b, n, h) of dq; dkv_pitch: elements between consecutive tokens of dk / dv
// (both describe the caller's dense tensors, of which a chunk of units writes its part)
int tensor_bsa_bwd(const Geometry& g, const void* q, const void* k, const void* v, const int32_t* idx,
                   const void* out, const float* lse, const void* dout, void* dq, void* dk, void* dv,
                   const long long* dq_strides, long long dkv_pitch, void* ws, int32_t* status, cudaStream_t s);

}  // namespace pisa
