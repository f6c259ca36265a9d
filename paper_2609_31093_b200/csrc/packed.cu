// Packed variable-length batches as padded batches.
//
// The method is causal: what a token selects and attends to depends on the tokens before it and on
// nothing after it (every scored node lies wholly in its past; the partial nodes on its own path are
// forced, never scored).  A short sequence therefore gives the same rows whether it is run alone or as
// the first `len` tokens of a longer, zero-filled batch element.  pisa_forward_packed uses that to run
// many short sequences through ONE set of launches: sequences of similar length are copied into a
// padded batch [B', N', H, d] (k and v zero past the end: a masked key must not be NaN), the ordinary
// batched forward runs on it, and the valid rows are copied back to the packed outputs.
#include "pisa_common.cuh"

namespace pisa {

namespace {

// packed <-> padded rows of up to five tensors in one launch (blockIdx.z picks the tensor); 16-byte vectors
struct PackSrc {
  const uint4* src[5];
  uint4* dst[5];
  int row_vec[5];                 // 16-byte vectors per token row (H * d * elem / 16)
};

__global__ void __launch_bounds__(256) pack_gather_kernel(PackSrc a, PackTable tab, int b_first, int Np) {
  const int z = blockIdx.z, bl = blockIdx.y;
  const int off = tab.off[bl], len = tab.len[bl];
  const int rv = a.row_vec[z];
  const long long n = (long long)Np * rv;
  const uint4* src = a.src[z] + (long long)off * rv;
  uint4* dst = a.dst[z] + (long long)(b_first + bl) * n;
  const long long n_valid = (long long)len * rv;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    dst[i] = (i < n_valid) ? src[i] : make_uint4(0u, 0u, 0u, 0u);
}

// padded -> packed: out rows [total, Hq, d], lse sequence-major [Hq, len], idx sequence-major [Hkv, len, K]
struct UnpackArgs {
  const uint4* out_pad;
  uint4* out;
  int out_row_vec;
  const float* lse_pad;
  float* lse;
  const int32_t* idx_pad;
  int32_t* idx;
  int Hq, Hkv, K;
};

__global__ void __launch_bounds__(256) pack_scatter_kernel(UnpackArgs a, PackTable tab, int b_first, int Np) {
  const int z = blockIdx.z, bl = blockIdx.y;
  const long long off = tab.off[bl];
  const int len = tab.len[bl];
  const long long b = b_first + bl;
  const long long tid0 = (long long)blockIdx.x * blockDim.x + threadIdx.x, step = (long long)gridDim.x * blockDim.x;
  if (z == 0) {
    const long long n = (long long)len * a.out_row_vec;
    const uint4* src = a.out_pad + b * Np * a.out_row_vec;
    uint4* dst = a.out + off * a.out_row_vec;
    for (long long i = tid0; i < n; i += step) dst[i] = src[i];
  } else if (z == 1) {
    const long long n = (long long)a.Hq * len;
    const float* src = a.lse_pad + b * a.Hq * Np;
    float* dst = a.lse + off * a.Hq;
    for (long long i = tid0; i < n; i += step) {
      const long long h = i / len, t = i - h * len;
      dst[i] = src[h * Np + t];
    }
  } else {
    const long long row = (long long)len * a.K, n = (long long)a.Hkv * row;
    const int32_t* src = a.idx_pad + b * a.Hkv * Np * a.K;
    int32_t* dst = a.idx + off * a.Hkv * a.K;
    for (long long i = tid0; i < n; i += step) {
      const long long h = i / row, r = i - h * row;
      dst[i] = src[h * (long long)Np * a.K + r];
    }
  }
}

// padded -> packed: the valid rows only (the gradients of a padded batch)
__global__ void __launch_bounds__(256) pack_scatter_rows_kernel(PackSrc a, PackTable tab, int b_first, int Np) {
  const int z = blockIdx.z, bl = blockIdx.y;
  const int rv = a.row_vec[z];
  const long long n_valid = (long long)tab.len[bl] * rv;
  const uint4* src = a.src[z] + (long long)(b_first + bl) * Np * rv;
  uint4* dst = a.dst[z] + (long long)tab.off[bl] * rv;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_valid; i += (long long)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

// packed -> padded for what the backward reads beside the rows: idx sequence-major [Hkv, len, K] -> [B', Hkv, Np, K]
// with -1 past the end (a padded query row then has no blocks and adds nothing to any key's gradient), lse
// sequence-major [Hq, len] -> [B', Hq, Np] with 0 past the end
struct PackMeta {
  const int32_t* idx;
  int32_t* idx_pad;
  const float* lse;
  float* lse_pad;
  int Hq, Hkv, K;
};
__global__ void __launch_bounds__(256) pack_gather_meta_kernel(PackMeta a, PackTable tab, int b_first, int Np) {
  const int z = blockIdx.z, bl = blockIdx.y;
  const long long off = tab.off[bl];
  const int len = tab.len[bl];
  const long long b = b_first + bl;
  const long long tid0 = (long long)blockIdx.x * blockDim.x + threadIdx.x, step = (long long)gridDim.x * blockDim.x;
  if (z == 0) {
    const long long row = (long long)Np * a.K, n = (long long)a.Hkv * row;
    const int32_t* src = a.idx + off * a.Hkv * a.K;
    int32_t* dst = a.idx_pad + b * n;
    for (long long i = tid0; i < n; i += step) {
      const long long h = i / row, r = i - h * row;                 // r = t * K + slot
      dst[i] = (r < (long long)len * a.K) ? src[h * (long long)len * a.K + r] : -1;
    }
  } else {
    const long long n = (long long)a.Hq * Np;
    const float* src = a.lse + off * a.Hq;
    float* dst = a.lse_pad + b * n;
    for (long long i = tid0; i < n; i += step) {
      const long long h = i / Np, t = i - h * Np;
      dst[i] = (t < len) ? src[h * len + t] : 0.f;
    }
  }
}

int grid_x(long long work) {
  long long gx = (work + 255) / 256;
  const long long cap = 8LL * num_sms();
  if (gx > cap) gx = cap;
  return gx < 1 ? 1 : (int)gx;
}

}  // namespace

int launch_pack_gather(const Geometry& g, int elem_bytes, const void* q, const void* k, const void* v, void* q_pad,
                       void* k_pad, void* v_pad, const PackTable& tab, int b_first, cudaStream_t s) {
  PackSrc a = {};
  a.src[0] = (const uint4*)q; a.src[1] = (const uint4*)k; a.src[2] = (const uint4*)v;
  a.dst[0] = (uint4*)q_pad; a.dst[1] = (uint4*)k_pad; a.dst[2] = (uint4*)v_pad;
  a.row_vec[0] = g.Hq * g.d * elem_bytes / 16;
  a.row_vec[1] = a.row_vec[2] = g.Hkv * g.d * elem_bytes / 16;
  dim3 grid(grid_x((long long)g.N * a.row_vec[0]), tab.n, 3);
  pack_gather_kernel<<<grid, 256, 0, s>>>(a, tab, b_first, g.N);
  return check_launch("pack_gather");
}

int launch_pack_scatter(const Geometry& g, int elem_bytes, const void* out_pad, const float* lse_pad,
                        const int32_t* idx_pad, void* out, float* lse, int32_t* idx, const PackTable& tab, int b_first,
                        cudaStream_t s) {
  UnpackArgs a;
  a.out_pad = (const uint4*)out_pad; a.out = (uint4*)out;
  a.out_row_vec = g.Hq * g.d * elem_bytes / 16;
  a.lse_pad = lse_pad; a.lse = lse;
  a.idx_pad = idx_pad; a.idx = idx;
  a.Hq = g.Hq; a.Hkv = g.Hkv; a.K = g.K;
  dim3 grid(grid_x((long long)g.N * a.out_row_vec), tab.n, 3);
  pack_scatter_kernel<<<grid, 256, 0, s>>>(a, tab, b_first, g.N);
  return check_launch("pack_scatter");
}

// the backward's extra inputs: out and dout rows (zero past the end), idx and lse
int launch_pack_gather_bwd(const Geometry& g, int elem_bytes, const void* out, const void* dout, const int32_t* idx,
                           const float* lse, void* out_pad, void* dout_pad, int32_t* idx_pad, float* lse_pad,
                           const PackTable& tab, int b_first, cudaStream_t s) {
  PackSrc a = {};
  a.src[0] = (const uint4*)out; a.src[1] = (const uint4*)dout;
  a.dst[0] = (uint4*)out_pad; a.dst[1] = (uint4*)dout_pad;
  a.row_vec[0] = a.row_vec[1] = g.Hq * g.d * elem_bytes / 16;
  dim3 grid(grid_x((long long)g.N * a.row_vec[0]), tab.n, 2);
  pack_gather_kernel<<<grid, 256, 0, s>>>(a, tab, b_first, g.N);
  int st = check_launch("pack_gather_bwd");
  if (st != PISA_OK) return st;
  PackMeta m;
  m.idx = idx; m.idx_pad = idx_pad; m.lse = lse; m.lse_pad = lse_pad;
  m.Hq = g.Hq; m.Hkv = g.Hkv; m.K = g.K;
  dim3 grid2(grid_x((long long)g.N * g.Hkv * g.K), tab.n, 2);
  pack_gather_meta_kernel<<<grid2, 256, 0, s>>>(m, tab, b_first, g.N);
  return check_launch("pack_gather_meta");
}

// the gradients of the valid rows back to the packed tensors
int launch_pack_scatter_grads(const Geometry& g, int elem_bytes, const void* dq_pad, const void* dk_pad,
                              const void* dv_pad, void* dq, void* dk, void* dv, const PackTable& tab, int b_first,
                              cudaStream_t s) {
  PackSrc a = {};
  a.src[0] = (const uint4*)dq_pad; a.src[1] = (const uint4*)dk_pad; a.src[2] = (const uint4*)dv_pad;
  a.dst[0] = (uint4*)dq; a.dst[1] = (uint4*)dk; a.dst[2] = (uint4*)dv;
  a.row_vec[0] = g.Hq * g.d * elem_bytes / 16;
  a.row_vec[1] = a.row_vec[2] = g.Hkv * g.d * elem_bytes / 16;
  dim3 grid(grid_x((long long)g.N * a.row_vec[0]), tab.n, 3);
  pack_scatter_rows_kernel<<<grid, 256, 0, s>>>(a, tab, b_first, g.N);
  return check_launch("pack_scatter_grads");
}

}  // namespace pisa
