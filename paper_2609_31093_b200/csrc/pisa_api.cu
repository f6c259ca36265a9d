// C-ABI entry points of libpisa: argument checks, hierarchy/workspace layout, stage sequencing.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <memory>
#include <new>

#include "pisa_common.cuh"
#include "pisa_tensor.cuh"

namespace pisa {

static thread_local char g_cuda_err[512] = "";
static thread_local bool g_timing = false;
static thread_local cudaEvent_t g_ev[4] = {nullptr, nullptr, nullptr, nullptr};
static thread_local bool g_ev_valid = false;
// per-kernel marks (name of the kernel that starts at the mark, and the stream it was recorded on),
// recorded when timing is on; a kernel's time runs to the next mark on the same stream
constexpr int kMaxMarks = 192;
static thread_local cudaEvent_t g_mark_ev[kMaxMarks];
static thread_local const char* g_mark_name[kMaxMarks];
static thread_local cudaStream_t g_mark_stream[kMaxMarks];
static thread_local int g_mark_n = 0;
static thread_local bool g_mark_valid = false;

void kernel_mark(const char* name, cudaStream_t s) {
  if (!g_timing || g_mark_n >= kMaxMarks) return;
  if (!g_mark_valid) {
    for (int j = 0; j < kMaxMarks; ++j) cudaEventCreate(&g_mark_ev[j]);
    g_mark_valid = true;
  }
  g_mark_name[g_mark_n] = name;
  g_mark_stream[g_mark_n] = s;
  cudaEventRecord(g_mark_ev[g_mark_n], s);
  ++g_mark_n;
}

void record_cuda_error(const char* what, cudaError_t e) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
}

static unsigned long long g_launches = 0;   // kernels launched by this process (relaxed counter)

int check_launch(const char* what) {
  __atomic_fetch_add(&g_launches, 1ull, __ATOMIC_RELAXED);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    record_cuda_error(what, e);
    return PISA_ERR_CUDA;
  }
  return PISA_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static size_t elem_size(int dtype) { return dtype == PISA_BF16 ? 2 : 4; }

// PISA_DEBUG=1 in the environment switches the device-side index checks on for every call
static int env_debug_bits() {
  static int bits = -1;
  if (bits < 0) {
    const char* e = getenv("PISA_DEBUG");
    bits = (e != nullptr && e[0] != '\0' && e[0] != '0') ? PISA_DEBUG_BOUNDS : 0;
  }
  return bits;
}

// SM count of the current device (cached per device ordinal)
int num_sms() {
  constexpr int kMaxDev = 64;
  static int cached[kMaxDev] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) dev = 0;
  int n = __atomic_load_n(&cached[dev], __ATOMIC_RELAXED);
  if (n == 0) {
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
    __atomic_store_n(&cached[dev], n, __ATOMIC_RELAXED);
  }
  return n;
}

int resolve(const pisa_params_t* p, Geometry* g) {
  if (p == nullptr || g == nullptr) return PISA_ERR_INVALID_ARG;
  if (p->B <= 0 || p->N <= 0 || p->Hq <= 0 || p->Hkv <= 0 || p->d <= 0 || p->C <= 0) return PISA_ERR_INVALID_ARG;
  if (p->Hq % p->Hkv != 0 || p->K < 3 || p->g < 2 || !(p->scale >= 0.f)) return PISA_ERR_INVALID_ARG;
  if (p->dtype != PISA_BF16 && p->dtype != PISA_FP32) return PISA_ERR_UNSUPPORTED;
  if (p->causal != 1) return PISA_ERR_UNSUPPORTED;
  if (p->score_mode < PISA_SCORE_LSE || p->score_mode > PISA_SCORE_MEAN_VAR) return PISA_ERR_UNSUPPORTED;
  if (p->impl < PISA_IMPL_AUTO || p->impl > PISA_IMPL_TENSOR) return PISA_ERR_INVALID_ARG;
  if (p->d != 32 && p->d != 64 && p->d != 128) return PISA_ERR_UNSUPPORTED;
  const int G = p->Hq / p->Hkv;
  if (G != 1 && G != 2 && G != 4 && G != 8 && G != 16) return PISA_ERR_UNSUPPORTED;
  if (p->K > kMaxK || (long long)p->g * p->K > kMaxCand) return PISA_ERR_UNSUPPORTED;
  memset(g, 0, sizeof(*g));
  g->B = p->B; g->N = p->N; g->Hq = p->Hq; g->Hkv = p->Hkv; g->G = G; g->d = p->d;
  g->C = p->C; g->g = p->g; g->K = p->K;
  g->score_mode = p->score_mode;
  g->debug = p->debug | env_debug_bits();
  g->scale = (p->scale == 0.f) ? (float)(1.0 / sqrt((double)p->d)) : p->scale;
  g->M[0] = p->N;
  g->M[1] = (p->N + p->C - 1) / p->C;
  int L = 1;
  while (g->M[L] > 1) {
    if (L + 1 >= kMaxLevels) return PISA_ERR_UNSUPPORTED;
    g->M[L + 1] = (g->M[L] + p->g - 1) / p->g;
    ++L;
  }
  g->L = L;
  long long span = 1;
  for (int l = 1; l < kMaxLevels; ++l) {
    g->span[l] = span;
    if (span < (1LL << 40)) span *= p->g;
  }
  // levels back to back, each starting on a 256-byte boundary
  const size_t es = elem_size(p->dtype);
  size_t off = 0;
  for (int l = 1; l <= L; ++l) {
    g->level_off[l] = (long long)(off / es);
    off += align_up((size_t)p->B * p->Hkv * g->M[l] * p->d * es, 256);
  }
  auto strides = [&](const int64_t* in, long long* out, int H) {
    if (in[0] == 0 && in[1] == 0 && in[2] == 0) {
      out[2] = p->d; out[1] = (long long)H * p->d; out[0] = (long long)p->N * H * p->d;
    } else {
      out[0] = in[0]; out[1] = in[1]; out[2] = in[2];
    }
  };
  strides(p->q_stride, g->qs, p->Hq);
  strides(p->k_stride, g->ks, p->Hkv);
  strides(p->v_stride, g->vs, p->Hkv);
  strides(p->o_stride, g->os, p->Hq);
  // 16-byte vector loads need every row to start on a 16-byte boundary
  const long long vec = 16 / (long long)es;
  for (int i = 0; i < 3; ++i)
    if (g->qs[i] % vec || g->ks[i] % vec || g->vs[i] % vec || g->os[i] % vec) return PISA_ERR_INVALID_ARG;
  return PISA_OK;
}

static size_t pyramid_bytes_dtype(const Geometry& g, int dtype) {
  const size_t es = elem_size(dtype);
  return (size_t)g.level_off[g.L] * es + align_up((size_t)g.B * g.Hkv * g.M[g.L] * g.d * es, 256);
}

static bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }
// the pyramid is read with 32-byte loads
static bool misaligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) != 0; }

static bool use_tensor(const pisa_params_t* p, const Geometry& g) {
  if (p->impl == PISA_IMPL_SIMT) return false;
  return tensor_path_supported(g, p->dtype);
}

static size_t route_ws_bytes(const pisa_params_t* p, const Geometry& g) {
  size_t b = kStatusBytes;
  if (use_tensor(p, g)) b += tensor_route_workspace_bytes(g);
  return b;
}
static size_t bsa_ws_bytes(const pisa_params_t* p, const Geometry& g) {
  size_t b = kStatusBytes;
  if (use_tensor(p, g)) b += tensor_bsa_workspace_bytes(g);
  return b;
}

// Device arena of pisa_forward_host.  The call walks the KV heads (independent units of the path):
// unit u's tensors live in slot u % 4 and its kernels run on compute stream u % 2 with that stream's
// workspace and pyramid, so that two units' kernels are in flight (they fill each other's tails, as
// the chunks of pisa_forward do) while the next unit is uploaded and the previous one downloaded.
constexpr int kHostSlots = 4;
struct HostArena {
  pisa_params_t unit;          // the per-unit problem: Hkv = 1, Hq = G, dense strides
  Geometry ug;
  size_t fwd, qb, kb, lb, ib, pb;   // bytes: forward workspace, q/out, k/v, lse, idx, pyramid (one unit)
  size_t slot, total;
};
static int host_arena(const pisa_params_t* p, HostArena* a) {
  a->unit = *p;
  a->unit.Hq = p->Hq / p->Hkv;
  a->unit.Hkv = 1;
  for (int i = 0; i < 3; ++i) a->unit.q_stride[i] = a->unit.k_stride[i] = a->unit.v_stride[i] = a->unit.o_stride[i] = 0;
  int st = resolve(&a->unit, &a->ug);
  if (st != PISA_OK) return st;
  const Geometry& g = a->ug;
  const size_t es = elem_size(p->dtype);
  const size_t r = route_ws_bytes(&a->unit, g), b = bsa_ws_bytes(&a->unit, g);
  a->fwd = align_up(r > b ? r : b, 256);
  a->qb = align_up((size_t)g.B * g.N * g.Hq * g.d * es, 256);
  a->kb = align_up((size_t)g.B * g.N * g.d * es, 256);
  a->lb = align_up((size_t)g.B * g.Hq * g.N * sizeof(float), 256);
  a->ib = align_up((size_t)g.B * g.N * g.K * sizeof(int32_t), 256);
  a->pb = align_up(pyramid_bytes_dtype(g, p->dtype), 256);
  a->slot = 2 * a->qb + 2 * a->kb + a->lb + a->ib;
  a->total = 2 * (a->fwd + a->pb) + kHostSlots * a->slot;
  return PISA_OK;
}

static int clear_status(void* ws, cudaStream_t s) {
  cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, s);
  if (e != cudaSuccess) { record_cuda_error("status memset", e); return PISA_ERR_CUDA; }
  return PISA_OK;
}

static int do_route(const pisa_params_t* p, const Geometry& g, const void* q, const void* k, const void* pyr,
                    int32_t* idx, float* sel_lse, float* margin, float* lse_out, void* ws, size_t ws_bytes,
                    cudaStream_t s) {
  if (ws_bytes < route_ws_bytes(p, g)) return PISA_ERR_WORKSPACE_TOO_SMALL;
  if (use_tensor(p, g))
    return tensor_route(g, p->dtype, q, k, pyr, idx, sel_lse, margin, lse_out, (char*)ws + kStatusBytes, (int32_t*)ws, s);
  kernel_mark("route_simt", s);
  int st = launch_route_simt(g, p->dtype, q, k, pyr, idx, margin, s);
  if (st != PISA_OK || sel_lse == nullptr) return st;
  kernel_mark("sel_lse", s);
  return launch_sel_lse_simt(g, p->dtype, q, k, idx, sel_lse, (int32_t*)ws, s);
}

static int do_bsa(const pisa_params_t* p, const Geometry& g, const void* q, const void* k, const void* v,
                  const int32_t* idx, const float* sel_lse, void* out, float* lse, bool lse_ready, bool forced_present,
                  void* ws, size_t ws_bytes, cudaStream_t s) {
  if (ws_bytes < bsa_ws_bytes(p, g)) return PISA_ERR_WORKSPACE_TOO_SMALL;
  if (use_tensor(p, g))
    return tensor_bsa(g, p->dtype, q, k, v, idx, sel_lse, out, lse, lse_ready, forced_present,
                      (char*)ws + kStatusBytes, (int32_t*)ws, s);
  kernel_mark("bsa_simt", s);
  return launch_bsa_simt(g, p->dtype, q, k, v, idx, out, lse, s);
}

static void stage_mark(int i, cudaStream_t s) {
  if (!g_timing) return;
  if (!g_ev_valid) {
    for (int j = 0; j < 4; ++j) cudaEventCreate(&g_ev[j]);
    g_ev_valid = true;
  }
  cudaEventRecord(g_ev[i], s);
}

// ---------------------------------------------------------------- forward in chunks on two streams
//
// The (batch, KV head) units of a forward are independent, and its kernels load different parts of
// the machine (stage 1 of the routing: instruction issue; the two tile kernels: L2 and tensor cores).
// A large tensor-path forward is therefore cut into chunks of units that alternate between the
// caller's stream and one internal stream: while a persistent tile kernel of one chunk drains, the
// next kernels of the other chunk fill the SMs it frees.  A chunk is a rectangular sub-problem that
// is contiguous in idx and lse: whole batches, or a range of KV heads of one batch.  The pyramid is
// built once for the whole problem; a chunk's geometry points at its units inside it.
constexpr int kMaxChunks = 4;                     // measured at B=1, Hkv=8, N=128K: 2 / 4 / 8 chunks -> 46.4 / 45.2 / 46.4 ms
constexpr int kStreams = 2;                       // the caller's stream + one internal (3 or 4 streams: no gain)
constexpr int kMaxStreams = kStreams;
static thread_local int g_chunk_limit = 0;        // pisa_set_forward_chunks: 0 = automatic, 1 = never split
constexpr long long kMinChunkTokens = 65536;      // units * N per chunk below which splitting does not pay

struct Chunk { int b0, nb, h0, nh; };
struct ForwardPlan {
  int n;                        // 1 = not split
  Chunk c[kMaxChunks];
  int streams;                  // streams the chunks alternate on (the caller's + internal ones)
  size_t region;                // workspace bytes of one stream's region (largest chunk), 256-aligned
  size_t total;                 // status word + regions
};

static int chunk_problem(const pisa_params_t* p, const Geometry& g, const Chunk& c, pisa_params_t* pc, Geometry* gc) {
  *pc = *p;
  pc->B = c.nb;
  pc->Hkv = c.nh;
  pc->Hq = c.nh * g.G;
  for (int i = 0; i < 3; ++i) {
    pc->q_stride[i] = g.qs[i]; pc->k_stride[i] = g.ks[i]; pc->v_stride[i] = g.vs[i]; pc->o_stride[i] = g.os[i];
  }
  const int st = resolve(pc, gc);
  if (st != PISA_OK) return st;
  const long long unit0 = (long long)c.b0 * g.Hkv + c.h0;
  for (int l = 1; l <= g.L; ++l) gc->level_off[l] = g.level_off[l] + unit0 * g.M[l] * g.d;
  return PISA_OK;
}

constexpr int kOpRoute = 1, kOpBsa = 2, kOpBwd = 4;

static bool ops_supported(const pisa_params_t* p, const Geometry& g, int ops) {
  if (ops == kOpBwd) return p->impl != PISA_IMPL_SIMT && tensor_bwd_supported(g, p->dtype);
  return use_tensor(p, g);
}
static size_t ops_ws_bytes(const pisa_params_t* p, const Geometry& g, int ops) {     // with the status word
  size_t m = kStatusBytes;
  if (ops & kOpRoute) { const size_t r = route_ws_bytes(p, g); if (r > m) m = r; }
  if (ops & kOpBsa) { const size_t b = bsa_ws_bytes(p, g); if (b > m) m = b; }
  if (ops & kOpBwd) { const size_t b = kStatusBytes + tensor_bwd_workspace_bytes(g); if (b > m) m = b; }
  return m;
}

static int forward_plan(const pisa_params_t* p, const Geometry& g, int ops, ForwardPlan* pl) {
  pl->n = 1;
  pl->c[0] = {0, g.B, 0, g.Hkv};
  const long long units = (long long)g.B * g.Hkv;
  long long parts = units * g.N / kMinChunkTokens;
  // The attention kernel draws its work items dynamically, so it no longer leaves a tail of idle SMs for
  // another chunk to fill: two chunks (measured 44.5 ms at B=1, Hkv=8, N=128K against 45.2 with four) keep
  // the leaf-scoring kernel's tail covered.  Routing alone (stage 1 and the statically walked leaf scoring
  // fill each other's tails) and the backward kernel, which also walks its items statically, keep four.
  const int max_chunks = (ops == kOpBwd || ops == kOpRoute) ? kMaxChunks : 2;
  if (parts > max_chunks) parts = max_chunks;
  if (g_chunk_limit > 0 && parts > g_chunk_limit) parts = g_chunk_limit;
  if (parts > units) parts = units;
  if (ops_supported(p, g, ops) && parts >= 2) {
    int n = 0;
    if (g.B >= parts) {                       // whole batches
      for (int i = 0; i < parts; ++i) {
        const int b0 = (int)((long long)g.B * i / parts), b1 = (int)((long long)g.B * (i + 1) / parts);
        pl->c[n++] = {b0, b1 - b0, 0, g.Hkv};
      }
    } else {                                  // head ranges inside every batch
      int per = (int)(parts / g.B);
      if (per > g.Hkv) per = g.Hkv;
      for (int b = 0; b < g.B; ++b)
        for (int i = 0; i < per; ++i) {
          const int h0 = g.Hkv * i / per, h1 = g.Hkv * (i + 1) / per;
          pl->c[n++] = {b, 1, h0, h1 - h0};
        }
    }
    pl->n = n;
  }
  size_t region = 0;
  for (int i = 0; i < pl->n; ++i) {
    pisa_params_t pc;
    Geometry gc;
    const int st = chunk_problem(p, g, pl->c[i], &pc, &gc);
    if (st != PISA_OK) return st;
    if (pl->n > 1 && !ops_supported(&pc, gc, ops)) {   // a chunk the tensor path does not take: run unsplit
      pl->n = 1;
      pl->c[0] = {0, g.B, 0, g.Hkv};
      i = -1;
      region = 0;
      continue;
    }
    const size_t m = align_up(ops_ws_bytes(&pc, gc, ops) - kStatusBytes, 256);
    if (m > region) region = m;
  }
  pl->region = region;
  pl->streams = (pl->n > 1) ? (pl->n < kStreams ? pl->n : kStreams) : 1;
  pl->total = kStatusBytes + pl->streams * region;
  return PISA_OK;
}

// Internal streams ([0] unused) and fork / join events, per host thread AND per device: streams and
// events belong to the device that was current when they were made.  g_side / g_fork / g_join point at
// the set of the device that is current in the call being served (side_streams() selects it).
constexpr int kMaxDevices = 64;
struct SideSet { cudaStream_t side[kMaxStreams]; cudaEvent_t fork, join[kMaxStreams]; };
static thread_local SideSet g_sets[kMaxDevices] = {};
static thread_local cudaStream_t* g_side = g_sets[0].side;
static thread_local cudaEvent_t g_fork = nullptr;
static thread_local cudaEvent_t* g_join = g_sets[0].join;

static int side_streams() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { record_cuda_error("cudaGetDevice", e); return PISA_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return PISA_ERR_UNSUPPORTED;
  SideSet& ss = g_sets[dev];
  if (ss.fork == nullptr) {
    for (int i = 1; i < kMaxStreams && e == cudaSuccess; ++i) {
      e = cudaStreamCreateWithFlags(&ss.side[i], cudaStreamNonBlocking);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ss.join[i], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ss.fork, cudaEventDisableTiming);
    if (e != cudaSuccess) { record_cuda_error("internal streams", e); ss.fork = nullptr; return PISA_ERR_CUDA; }
  }
  g_side = ss.side; g_fork = ss.fork; g_join = ss.join;
  return PISA_OK;
}

// A chunk's view of the caller's tensors.
struct ChunkView {
  pisa_params_t p;
  Geometry g;
  Chunk c;
  long long unit0;              // first (batch, KV head) unit, flattened
  size_t q_off, k_off, v_off, o_off;   // byte offsets into q / k / v / out
  char* region;                 // this chunk's scratch (past any status word)
  cudaStream_t stream;
};

// Plans `ops` for (p, g), falls back to the unsplit plan when `ws_bytes` only covers that one, and
// returns the bytes the plan needs.
static int plan_for(const pisa_params_t* p, const Geometry& g, int ops, size_t ws_bytes, ForwardPlan* pl) {
  int st = forward_plan(p, g, ops, pl);
  if (st != PISA_OK) return st;
  if (pl->n > 1 && ws_bytes < pl->total) {   // a workspace sized for another length of the same problem: unsplit
    pl->n = 1;
    pl->streams = 1;
    pl->total = ops_ws_bytes(p, g, ops);
  }
  if (ws_bytes < pl->total) return PISA_ERR_WORKSPACE_TOO_SMALL;
  if (pl->n > 1) return side_streams();
  return PISA_OK;
}

// Runs fn(view) for every chunk of a split plan: chunk i on stream i % streams (the caller's, then the
// internal ones, forked here and joined before returning -- also after a failed launch, so that the
// caller's stream never runs ahead of the internal one).
template <typename F>
static int run_chunks(const pisa_params_t* p, const Geometry& g, const ForwardPlan& pl, void* ws, cudaStream_t s,
                      F&& fn) {
  cudaError_t e = cudaEventRecord(g_fork, s);
  for (int i = 1; i < pl.streams && e == cudaSuccess; ++i) e = cudaStreamWaitEvent(g_side[i], g_fork, 0);
  if (e != cudaSuccess) { record_cuda_error("fork", e); return PISA_ERR_CUDA; }
  const size_t es = elem_size(p->dtype);
  int st = PISA_OK;
  for (int i = 0; i < pl.n && st == PISA_OK; ++i) {
    const Chunk& c = pl.c[i];
    ChunkView v;
    st = chunk_problem(p, g, c, &v.p, &v.g);
    if (st != PISA_OK) break;
    const int si = i % pl.streams;
    v.c = c;
    v.stream = si ? g_side[si] : s;
    v.region = (char*)ws + kStatusBytes + (size_t)si * pl.region;
    v.unit0 = (long long)c.b0 * g.Hkv + c.h0;
    v.q_off = (size_t)((long long)c.b0 * g.qs[0] + (long long)c.h0 * g.G * g.qs[2]) * es;
    v.k_off = (size_t)((long long)c.b0 * g.ks[0] + (long long)c.h0 * g.ks[2]) * es;
    v.v_off = (size_t)((long long)c.b0 * g.vs[0] + (long long)c.h0 * g.vs[2]) * es;
    v.o_off = (size_t)((long long)c.b0 * g.os[0] + (long long)c.h0 * g.G * g.os[2]) * es;
    st = fn(v, i);
  }
  e = cudaSuccess;
  for (int i = 1; i < pl.streams; ++i) {
    kernel_mark("end", g_side[i]);
    if (e == cudaSuccess) e = cudaEventRecord(g_join[i], g_side[i]);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, g_join[i], 0);
  }
  if (e != cudaSuccess && st == PISA_OK) { record_cuda_error("join", e); st = PISA_ERR_CUDA; }
  return st;
}

static int do_route_chunked(const pisa_params_t* p, const Geometry& g, const void* q, const void* k, const void* pyr,
                            int32_t* idx, float* sel_lse, float* margin, void* ws, size_t ws_bytes, cudaStream_t s) {
  ForwardPlan pl;
  int st = plan_for(p, g, kOpRoute, ws_bytes, &pl);
  if (st != PISA_OK) return st;
  st = clear_status(ws, s);
  if (st != PISA_OK) return st;
  g_mark_n = 0;
  if (pl.n == 1) st = do_route(p, g, q, k, pyr, idx, sel_lse, margin, nullptr, ws, ws_bytes, s);
  else
    st = run_chunks(p, g, pl, ws, s, [&](const ChunkView& v, int) {
      return tensor_route(v.g, p->dtype, (const char*)q + v.q_off, (const char*)k + v.k_off, pyr,
                          idx + v.unit0 * g.N * g.K, sel_lse ? sel_lse + v.unit0 * g.G * g.N * g.K : nullptr,
                          margin ? margin + v.unit0 * g.N : nullptr, nullptr, v.region, (int32_t*)ws, v.stream);
    });
  kernel_mark("end", s);
  return st;
}

static int do_bsa_chunked(const pisa_params_t* p, const Geometry& g, const void* q, const void* k, const void* v_,
                          const int32_t* idx, const float* sel_lse, void* out, float* lse, void* ws, size_t ws_bytes,
                          cudaStream_t s) {
  ForwardPlan pl;
  int st = plan_for(p, g, kOpBsa, ws_bytes, &pl);
  if (st != PISA_OK) return st;
  st = clear_status(ws, s);
  if (st != PISA_OK) return st;
  g_mark_n = 0;
  if (pl.n == 1) st = do_bsa(p, g, q, k, v_, idx, sel_lse, out, lse, false, false, ws, ws_bytes, s);
  else
    st = run_chunks(p, g, pl, ws, s, [&](const ChunkView& v, int) {
      return tensor_bsa(v.g, p->dtype, (const char*)q + v.q_off, (const char*)k + v.k_off, (const char*)v_ + v.v_off,
                        idx + v.unit0 * g.N * g.K, sel_lse ? sel_lse + v.unit0 * g.G * g.N * g.K : nullptr,
                        (char*)out + v.o_off, lse + v.unit0 * g.G * g.N, false, false, v.region, (int32_t*)ws, v.stream);
    });
  kernel_mark("end", s);
  return st;
}

// Attention backward of one dense problem (dq, dk, dv dense like q, k, v), in chunks when it is large.
static int do_bwd(const pisa_params_t* p, const Geometry& g, const void* q, const void* k, const void* v_,
                  const int32_t* idx, const void* out, const float* lse, const void* dout, void* dq, void* dk,
                  void* dv, void* ws, size_t ws_bytes, cudaStream_t s) {
  ForwardPlan pl;
  int st = plan_for(p, g, kOpBwd, ws_bytes, &pl);
  if (st != PISA_OK) return st;
  const size_t es = elem_size(p->dtype);
  const long long dqs[3] = {(long long)g.N * g.Hq * g.d, (long long)g.Hq * g.d, g.d};
  const long long pitch = (long long)g.Hkv * g.d;
  if (pl.n == 1)
    return tensor_bsa_bwd(g, q, k, v_, idx, out, lse, dout, dq, dk, dv, dqs, pitch, (char*)ws + kStatusBytes,
                          (int32_t*)ws, s);
  return run_chunks(p, g, pl, ws, s, [&](const ChunkView& v, int) {
    const size_t dq_off = (size_t)((long long)v.c.b0 * dqs[0] + (long long)v.c.h0 * g.G * dqs[2]) * es;
    const size_t dkv_off = (size_t)((long long)v.c.b0 * g.N * pitch + (long long)v.c.h0 * g.d) * es;
    return tensor_bsa_bwd(v.g, (const char*)q + v.q_off, (const char*)k + v.k_off, (const char*)v_ + v.v_off,
                          idx + v.unit0 * g.N * g.K, (const char*)out + v.o_off, lse + v.unit0 * g.G * g.N,
                          (const char*)dout + v.o_off, (char*)dq + dq_off, (char*)dk + dkv_off, (char*)dv + dkv_off, dqs,
                          pitch, v.region, (int32_t*)ws, v.stream);
  });
}

// v_ready (optional): an event the attention stage must wait for (the values may still be on their way while
// the routing runs); routed (optional): recorded when idx is final, before the attention stage
static int do_forward(const pisa_params_t* p, const Geometry& g, const void* q, const void* k, const void* v_,
                      void* pyr, int32_t* idx, void* out, float* lse, void* ws, size_t ws_bytes,
                      cudaStream_t s, bool clear = true, cudaEvent_t v_ready = nullptr, cudaEvent_t routed = nullptr) {
  ForwardPlan pl;
  int st = plan_for(p, g, kOpRoute | kOpBsa, ws_bytes, &pl);
  if (st != PISA_OK) return st;
  st = clear ? clear_status(ws, s) : PISA_OK;
  if (st != PISA_OK) return st;
  g_mark_n = 0;
  stage_mark(0, s);
  kernel_mark("pyramid", s);
  st = launch_pyramid(g, p->dtype, k, pyr, (int32_t*)ws, s);
  if (st != PISA_OK) return st;
  stage_mark(1, s);
  if (pl.n == 1) {
    // the tensor-core routing already knows every kept leaf's per-head LSE, so it hands the rows'
    // softmax denominators to the attention stage
    st = do_route(p, g, q, k, pyr, idx, nullptr, nullptr, lse, ws, ws_bytes, s);
    if (st != PISA_OK) return st;
    cudaError_t ee = cudaSuccess;
    if (routed != nullptr) ee = cudaEventRecord(routed, s);
    if (ee == cudaSuccess && v_ready != nullptr) ee = cudaStreamWaitEvent(s, v_ready, 0);
    if (ee != cudaSuccess) { record_cuda_error("forward stage events", ee); return PISA_ERR_CUDA; }
    stage_mark(2, s);
    st = do_bsa(p, g, q, k, v_, idx, nullptr, out, lse, use_tensor(p, g) && g.score_mode == PISA_SCORE_LSE, true, ws,
                ws_bytes, s);
  } else {
    st = run_chunks(p, g, pl, ws, s, [&](const ChunkView& v, int i) {
      int32_t* ic = idx + v.unit0 * g.N * g.K;
      float* lc = lse + v.unit0 * g.G * g.N;
      int r = tensor_route(v.g, p->dtype, (const char*)q + v.q_off, (const char*)k + v.k_off, pyr, ic, nullptr, nullptr,
                           lc, v.region, (int32_t*)ws, v.stream);
      if (r != PISA_OK) return r;
      if (v_ready != nullptr) {
        const cudaError_t ee = cudaStreamWaitEvent(v.stream, v_ready, 0);
        if (ee != cudaSuccess) { record_cuda_error("forward stage events", ee); return (int)PISA_ERR_CUDA; }
      }
      if (i == 0) stage_mark(2, s);
      return tensor_bsa(v.g, p->dtype, (const char*)q + v.q_off, (const char*)k + v.k_off, (const char*)v_ + v.v_off,
                        ic, nullptr, (char*)out + v.o_off, lc, g.score_mode == PISA_SCORE_LSE, true, v.region, (int32_t*)ws,
                        v.stream);
    });
    if (st == PISA_OK && routed != nullptr) {             // (chunks: the indices count as final when all chunks have ended)
      const cudaError_t ee = cudaEventRecord(routed, s);
      if (ee != cudaSuccess) { record_cuda_error("forward stage events", ee); return PISA_ERR_CUDA; }
    }
  }
  stage_mark(3, s);
  kernel_mark("end", s);
  return st;
}

// pisa_route on the caller's stream only, never split into chunks: creates no stream or event
int route_unsplit(const pisa_params_t* p, const void* q, const void* k, const void* pyramid, int32_t* idx,
                  float* margin, void* ws, size_t ws_bytes, cudaStream_t s) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q || !k || !pyramid || !idx || !ws || misaligned(q) || misaligned(k) || misaligned32(pyramid) || misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  if (ws_bytes < route_ws_bytes(p, g)) return PISA_ERR_WORKSPACE_TOO_SMALL;
  st = clear_status(ws, s);
  if (st != PISA_OK) return st;
  return do_route(p, g, q, k, pyramid, idx, nullptr, margin, nullptr, ws, ws_bytes, s);
}
// bytes route_unsplit needs
int route_unsplit_bytes(const pisa_params_t* p, size_t* bytes) {
  Geometry g;
  const int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  *bytes = route_ws_bytes(p, g);
  return PISA_OK;
}

}  // namespace pisa

using namespace pisa;

extern "C" {

int pisa_version(void) { return PISA_VERSION; }

const char* pisa_status_string(int status) {
  switch (status) {
    case PISA_OK: return "ok";
    case PISA_ERR_INVALID_ARG: return "invalid argument";
    case PISA_ERR_UNSUPPORTED: return "unsupported configuration";
    case PISA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case PISA_ERR_CUDA: return "CUDA error";
    case PISA_ERR_TIMEOUT: return "device-side wait timed out";
    case PISA_ERR_BOUNDS: return "device-side index check failed";
    case PISA_ERR_STATIC_SCRATCH_TOO_SMALL:
      return "problem needs more scratch than the library's built-in device array holds";
    default: return "unknown status";
  }
}

const char* pisa_last_cuda_error(void) { return g_cuda_err; }

int pisa_pyramid_layout(const pisa_params_t* p, int32_t* L, int32_t* M, int64_t* level_off, size_t* bytes) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (L) *L = g.L;
  for (int l = 0; l <= g.L; ++l) {
    if (M) M[l] = g.M[l];
    if (level_off) level_off[l] = g.level_off[l];
  }
  if (bytes) *bytes = pyramid_bytes_dtype(g, p->dtype);
  return PISA_OK;
}

// ---------------------------------------------------------------- packed batches as padded batches
//
// pisa_forward_packed groups the short sequences of a packed batch by length and runs every group as a
// padded batch [B', N'] through one set of launches (the copies are in packed.cu).  N' comes from a fixed
// grid (every length up to 15, then m * 2^k, m = 8..15: at most 12.5 % apart) so that the workspace can be sized from the parameters
// alone; a group holds sequences no shorter than 3/4 of its N' and at most kPackTokens padded tokens
// (more if the longest sequence is longer).  Sequences above kPackDirectLen, and groups of one, run
// unpadded on the packed tensors themselves.
constexpr int kPackDirectLen = 8192;
constexpr long long kPackTokens = 32768;

static int pack_grid_len(int len) {
  int k = 0;
  while ((15LL << k) < len) ++k;
  const int m = (int)(((long long)len + (1LL << k) - 1) >> k);      // 8..15 for k > 0; the length itself up to 15
  return m << k;
}

// sequences one group of padded length np may hold: kPackTokens padded tokens, and (batch, KV head) units that
// still index a grid's y dimension
static long long pack_group_cap(const pisa_params_t* p, long long tokens, long long np) {
  long long b = tokens / np < 1 ? 1 : tokens / np;
  if (b * p->Hkv > 65535) b = 65535 / p->Hkv;
  return b < 1 ? 1 : b;
}

struct PackedArena {
  long long tokens;                        // padded tokens one group may hold
  size_t fwd, pyr, qb, kb, lb, ib, total;  // bytes: forward workspace, pyramid, q/out, k/v, lse, idx (one group)
};

static size_t forward_ws_bytes(const pisa_params_t* p, const Geometry& g, int* st) {
  size_t r = route_ws_bytes(p, g), a = bsa_ws_bytes(p, g);
  size_t f = r > a ? r : a;
  ForwardPlan pl;
  *st = forward_plan(p, g, kOpRoute | kOpBsa, &pl);
  if (*st == PISA_OK && pl.total > f) f = pl.total;
  return f;
}

static int packed_arena(const pisa_params_t* p, PackedArena* a) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  a->tokens = kPackTokens;
  size_t fwd = forward_ws_bytes(p, g, &st), pyr = 0;
  if (st != PISA_OK) return st;
  const int n_max = p->N < kPackDirectLen ? p->N : kPackDirectLen;
  for (int k = 0; k < 31; ++k)
    for (int m = (k == 0) ? 1 : 8; m <= 15; ++m) {
      const long long np = (long long)m << k;
      if (np > pack_grid_len(n_max)) continue;
      pisa_params_t pg = *p;
      pg.N = (int)np;
      pg.B = (int)pack_group_cap(p, a->tokens, np);
      Geometry gg;
      if ((st = resolve(&pg, &gg)) != PISA_OK) return st;
      const size_t f = forward_ws_bytes(&pg, gg, &st);
      if (st != PISA_OK) return st;
      if (f > fwd) fwd = f;
      const size_t pb = pyramid_bytes_dtype(gg, p->dtype);
      if (pb > pyr) pyr = pb;
    }
  const size_t es = elem_size(p->dtype);
  const size_t tok = (size_t)a->tokens;                                    // B' * N' <= tokens for every group
  a->fwd = align_up(fwd, 256);
  a->pyr = align_up(pyr, 256);
  a->qb = align_up(tok * g.Hq * g.d * es, 256);
  a->kb = align_up(tok * g.Hkv * g.d * es, 256);
  a->lb = align_up(tok * g.Hq * sizeof(float), 256);
  a->ib = align_up(tok * g.Hkv * g.K * sizeof(int32_t), 256);
  a->total = a->fwd + a->pyr + 2 * a->qb + 2 * a->kb + a->lb + a->ib;
  return PISA_OK;
}

// ... and what pisa_bsa_bwd_packed needs to run the same groups: the backward's workspace for any group, padded q /
// out / dout / dq, k / v / dk / dv, lse and idx
struct PackedBwdArena {
  long long tokens;
  size_t bwd, qb, kb, lb, ib, total;
};
static int packed_bwd_arena(const pisa_params_t* p, PackedBwdArena* a) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  a->tokens = kPackTokens;
  auto need = [](const pisa_params_t* pp, const Geometry& gg, size_t* out) -> int {
    if (!tensor_bwd_supported(gg, pp->dtype) || pp->impl == PISA_IMPL_SIMT) return PISA_ERR_UNSUPPORTED;
    size_t b = kStatusBytes + tensor_bwd_workspace_bytes(gg);
    ForwardPlan pl;
    const int r = forward_plan(pp, gg, kOpBwd, &pl);
    if (r != PISA_OK) return r;
    if (pl.total > b) b = pl.total;
    *out = b;
    return PISA_OK;
  };
  size_t bwd = 0;
  if ((st = need(p, g, &bwd)) != PISA_OK) return st;
  const int n_max = p->N < kPackDirectLen ? p->N : kPackDirectLen;
  for (int k = 0; k < 31; ++k)
    for (int m = (k == 0) ? 1 : 8; m <= 15; ++m) {
      const long long np = (long long)m << k;
      if (np > pack_grid_len(n_max)) continue;
      pisa_params_t pg = *p;
      pg.N = (int)np;
      pg.B = (int)pack_group_cap(p, a->tokens, np);
      Geometry gg;
      if ((st = resolve(&pg, &gg)) != PISA_OK) return st;
      size_t b = 0;
      if ((st = need(&pg, gg, &b)) != PISA_OK) return st;
      if (b > bwd) bwd = b;
    }
  const size_t es = elem_size(p->dtype), tok = (size_t)a->tokens;
  a->bwd = align_up(bwd, 256);
  a->qb = align_up(tok * g.Hq * g.d * es, 256);
  a->kb = align_up(tok * g.Hkv * g.d * es, 256);
  a->lb = align_up(tok * g.Hq * sizeof(float), 256);
  a->ib = align_up(tok * g.Hkv * g.K * sizeof(int32_t), 256);
  a->total = a->bwd + 4 * a->qb + 4 * a->kb + a->lb + a->ib;
  return PISA_OK;
}

// The grouping of pisa_forward_packed, host arithmetic only.  order: the sequences that take part in groups,
// longest first (nseq + 1 ints of scratch); group[i] / padded[i] for sequence i: its group (0, 1, ... in launch
// order) and the group's padded length, or group -1 for a sequence that runs alone (longer than kPackDirectLen, the
// only one of its length class, or empty: padded = its own length).  Returns the number of groups.
static int packed_plan(const pisa_params_t* p, const int32_t* cu, int nseq, long long tokens, int* order,
                       int32_t* group, int32_t* padded) {
  size_t n_short = 0;
  for (int i = 0; i < nseq; ++i) {
    const int len = cu[i + 1] - cu[i];
    group[i] = -1;
    padded[i] = len;
    if (len > 0 && len <= kPackDirectLen) order[n_short++] = i;
  }
  std::stable_sort(order, order + n_short, [&](int a, int b) { return cu[a + 1] - cu[a] > cu[b + 1] - cu[b]; });
  int n_groups = 0;
  size_t at = 0;
  while (at < n_short) {
    const int np = pack_grid_len(cu[order[at] + 1] - cu[order[at]]);
    const long long b_cap = pack_group_cap(p, tokens, np);
    size_t end = at + 1;
    while (end < n_short && (long long)(end - at) < b_cap) {
      const int len = cu[order[end] + 1] - cu[order[end]];
      if (4LL * len < 3LL * np) break;
      ++end;
    }
    if (end - at >= 2) {
      for (size_t j = at; j < end; ++j) { group[order[j]] = n_groups; padded[order[j]] = np; }
      ++n_groups;
    }
    at = end;
  }
  return n_groups;
}

int pisa_packed_plan(const pisa_params_t* p, const int32_t* cu_seqlens, int32_t nseq, int32_t* group, int32_t* padded,
                     int32_t* n_groups) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!cu_seqlens || nseq < 0 || !group || !padded || cu_seqlens[0] != 0) return PISA_ERR_INVALID_ARG;
  for (int i = 0; i < nseq; ++i) {
    const int len = cu_seqlens[i + 1] - cu_seqlens[i];
    if (len < 0 || len > p->N) return PISA_ERR_INVALID_ARG;
  }
  PackedArena pa;
  if ((st = packed_arena(p, &pa)) != PISA_OK) return st;
  std::unique_ptr<int[]> order(new (std::nothrow) int[(size_t)nseq + 1]);
  if (!order) return PISA_ERR_INVALID_ARG;
  const int n = packed_plan(p, cu_seqlens, nseq, pa.tokens, order.get(), group, padded);
  if (n_groups) *n_groups = n;
  return PISA_OK;
}

int pisa_workspace_bytes(const pisa_params_t* p, int op, size_t* bytes) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (bytes == nullptr) return PISA_ERR_INVALID_ARG;
  size_t r = route_ws_bytes(p, g), a = bsa_ws_bytes(p, g);
  {                                          // the chunked plans of the three calls
    ForwardPlan pl;
    if ((st = forward_plan(p, g, kOpRoute, &pl)) != PISA_OK) return st;
    if (pl.total > r) r = pl.total;
    if ((st = forward_plan(p, g, kOpBsa, &pl)) != PISA_OK) return st;
    if (pl.total > a) a = pl.total;
  }
  size_t f = r > a ? r : a;                  // one buffer sized for the forward also serves pisa_route and pisa_bsa_fwd
  {
    ForwardPlan pl;
    if ((st = forward_plan(p, g, kOpRoute | kOpBsa, &pl)) != PISA_OK) return st;
    if (pl.total > f) f = pl.total;
  }
  switch (op) {
    case PISA_OP_ROUTE: *bytes = r; break;
    case PISA_OP_BSA: *bytes = a; break;
    case PISA_OP_FORWARD: *bytes = f; break;
    case PISA_OP_FLAT: *bytes = kStatusBytes; break;
    case PISA_OP_BSA_BWD:
      if (!tensor_bwd_supported(g, p->dtype) || p->impl == PISA_IMPL_SIMT) return PISA_ERR_UNSUPPORTED;
      *bytes = kStatusBytes + tensor_bwd_workspace_bytes(g);
      {
        ForwardPlan pl;
        if ((st = forward_plan(p, g, kOpBwd, &pl)) != PISA_OK) return st;
        if (pl.total > *bytes) *bytes = pl.total;
      }
      break;
    case PISA_OP_DECODE:
      if (!decode_supported(g, p->dtype)) return PISA_ERR_UNSUPPORTED;
      *bytes = kStatusBytes + decode_workspace_bytes(g);
      break;
    case PISA_OP_BSA_BWD_PACKED: {
      PackedBwdArena pa;
      st = packed_bwd_arena(p, &pa);
      if (st != PISA_OK) return st;
      *bytes = pa.total;
      break;
    }
    case PISA_OP_FORWARD_PACKED: {
      PackedArena pa;
      st = packed_arena(p, &pa);
      if (st != PISA_OK) return st;
      *bytes = pa.total;
      break;
    }
    case PISA_OP_FORWARD_HOST: {
      HostArena a;
      st = host_arena(p, &a);
      if (st != PISA_OK) return st;
      *bytes = a.total;
      break;
    }
    default: return PISA_ERR_INVALID_ARG;
  }
  return PISA_OK;
}

int pisa_build_pyramid(const pisa_params_t* p, const void* k, void* pyramid, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (k == nullptr || pyramid == nullptr || misaligned(k) || misaligned32(pyramid)) return PISA_ERR_INVALID_ARG;
  return launch_pyramid(g, p->dtype, k, pyramid, nullptr, (cudaStream_t)stream);
}

int pisa_route(const pisa_params_t* p, const void* q, const void* k, const void* pyramid, int32_t* idx,
               float* sel_lse, float* margin, void* ws, size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q || !k || !pyramid || !idx || !ws || misaligned(q) || misaligned(k) || misaligned32(pyramid) ||
      misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  return do_route_chunked(p, g, q, k, pyramid, idx, sel_lse, margin, ws, ws_bytes, (cudaStream_t)stream);
}

int pisa_bsa_fwd(const pisa_params_t* p, const void* q, const void* k, const void* v, const int32_t* idx,
                 const float* sel_lse, void* out, float* lse, void* ws, size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q || !k || !v || !idx || !out || !lse || !ws || misaligned(q) || misaligned(k) || misaligned(v) ||
      misaligned(out) || misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  return do_bsa_chunked(p, g, q, k, v, idx, sel_lse, out, lse, ws, ws_bytes, (cudaStream_t)stream);
}

int pisa_forward(const pisa_params_t* p, const void* q, const void* k, const void* v, void* pyramid,
                 int32_t* idx, void* out, float* lse, void* ws, size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q || !k || !v || !pyramid || !idx || !out || !lse || !ws || misaligned(q) || misaligned(k) ||
      misaligned(v) || misaligned32(pyramid) || misaligned(out) || misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  return do_forward(p, g, q, k, v, pyramid, idx, out, lse, ws, ws_bytes, (cudaStream_t)stream);
}

int pisa_forward_packed(const pisa_params_t* p, const int32_t* cu_seqlens, int32_t nseq, const void* q,
                        const void* k, const void* v, void* pyramid, int32_t* idx, void* out, float* lse,
                        void* ws, size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!cu_seqlens || nseq < 0 || !q || !k || !v || !pyramid || !idx || !out || !lse || !ws || misaligned(q) ||
      misaligned(k) || misaligned(v) || misaligned32(pyramid) || misaligned(out) || misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  if (p->B != 1 || cu_seqlens[0] != 0) return PISA_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i)
    if (p->q_stride[i] || p->k_stride[i] || p->v_stride[i] || p->o_stride[i]) return PISA_ERR_INVALID_ARG;
  for (int i = 0; i < nseq; ++i) {
    const int len = cu_seqlens[i + 1] - cu_seqlens[i];
    if (len < 0 || len > p->N) return PISA_ERR_INVALID_ARG;
  }
  cudaStream_t s = (cudaStream_t)stream;
  st = clear_status(ws, s);
  if (st != PISA_OK) return st;
  const size_t es = elem_size(p->dtype);
  auto run_alone = [&](int i) -> int {        // one sequence, unpadded, on the packed tensors themselves
    const size_t t0 = (size_t)cu_seqlens[i];
    const int len = cu_seqlens[i + 1] - cu_seqlens[i];
    if (len == 0) return PISA_OK;
    pisa_params_t pi = *p;
    pi.N = len;
    Geometry gi;
    int r = resolve(&pi, &gi);
    if (r != PISA_OK) return r;
    return do_forward(&pi, gi, (const char*)q + t0 * g.Hq * g.d * es, (const char*)k + t0 * g.Hkv * g.d * es,
                      (const char*)v + t0 * g.Hkv * g.d * es, pyramid, idx + t0 * g.Hkv * g.K,
                      (char*)out + t0 * g.Hq * g.d * es, lse + t0 * g.Hq, ws, ws_bytes, s, /*clear=*/false);
  };
  PackedArena pa;
  st = packed_arena(p, &pa);
  if (st != PISA_OK) return st;
  if (ws_bytes < pa.total) {      // a workspace sized for PISA_OP_FORWARD: one sequence after the other
    for (int i = 0; i < nseq; ++i)
      if ((st = run_alone(i)) != PISA_OK) return st;
    return PISA_OK;
  }
  char* base = (char*)ws;
  char* pyr_pad = base + pa.fwd;
  char* q_pad = pyr_pad + pa.pyr;
  char* k_pad = q_pad + pa.qb;
  char* v_pad = k_pad + pa.kb;
  char* o_pad = v_pad + pa.kb;
  float* l_pad = (float*)(o_pad + pa.qb);
  int32_t* i_pad = (int32_t*)((char*)l_pad + pa.lb);
  // the plan: which sequences share a padded batch (host arithmetic, see packed_plan), then group by group
  // (no exception may cross the C boundary: plain arrays, allocated without throwing)
  std::unique_ptr<int[]> order(new (std::nothrow) int[(size_t)nseq + 1]);
  std::unique_ptr<int32_t[]> group(new (std::nothrow) int32_t[(size_t)nseq + 1]);
  std::unique_ptr<int32_t[]> padded(new (std::nothrow) int32_t[(size_t)nseq + 1]);
  if (!order || !group || !padded) return PISA_ERR_INVALID_ARG;
  packed_plan(p, cu_seqlens, nseq, pa.tokens, order.get(), group.get(), padded.get());
  for (int i = 0; i < nseq; ++i)
    if (group[i] < 0 && (st = run_alone(i)) != PISA_OK) return st;
  // `order` lists the grouped candidates longest first; the members of a group are consecutive in it
  size_t n_short = 0;
  for (int i = 0; i < nseq; ++i) {
    const int len = cu_seqlens[i + 1] - cu_seqlens[i];
    if (len > 0 && len <= kPackDirectLen) ++n_short;
  }
  size_t at = 0;
  while (at < n_short) {
    const int first = order[at];
    if (group[first] < 0) { ++at; continue; }
    size_t end = at + 1;
    while (end < n_short && group[order[end]] == group[first]) ++end;
    const int nb = (int)(end - at), np = padded[first];
    pisa_params_t pg = *p;
    pg.B = nb;
    pg.N = np;
    Geometry gg;
    if ((st = resolve(&pg, &gg)) != PISA_OK) return st;
    PackTable tab;
    for (int b0 = 0; b0 < nb; b0 += kPackSeqs) {
      tab.n = nb - b0 < kPackSeqs ? nb - b0 : kPackSeqs;
      for (int j = 0; j < tab.n; ++j) {
        const int sq = order[at + (size_t)b0 + j];
        tab.off[j] = cu_seqlens[sq];
        tab.len[j] = cu_seqlens[sq + 1] - cu_seqlens[sq];
      }
      if ((st = launch_pack_gather(gg, (int)es, q, k, v, q_pad, k_pad, v_pad, tab, b0, s)) != PISA_OK) return st;
    }
    st = do_forward(&pg, gg, q_pad, k_pad, v_pad, pyr_pad, i_pad, o_pad, l_pad, ws, pa.fwd, s, /*clear=*/false);
    if (st != PISA_OK) return st;
    for (int b0 = 0; b0 < nb; b0 += kPackSeqs) {
      tab.n = nb - b0 < kPackSeqs ? nb - b0 : kPackSeqs;
      for (int j = 0; j < tab.n; ++j) {
        const int sq = order[at + (size_t)b0 + j];
        tab.off[j] = cu_seqlens[sq];
        tab.len[j] = cu_seqlens[sq + 1] - cu_seqlens[sq];
      }
      if ((st = launch_pack_scatter(gg, (int)es, o_pad, l_pad, i_pad, out, lse, idx, tab, b0, s)) != PISA_OK) return st;
    }
    at = end;
  }
  return PISA_OK;
}

int pisa_forward_host(const pisa_params_t* p, const void* q_host, const void* k_host, const void* v_host,
                      void* out_host, float* lse_host, int32_t* idx_host, void* ws, size_t ws_bytes,
                      void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q_host || !k_host || !v_host || !out_host || !lse_host || !ws || misaligned(ws)) return PISA_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i)
    if (p->q_stride[i] || p->k_stride[i] || p->v_stride[i] || p->o_stride[i]) return PISA_ERR_INVALID_ARG;
  HostArena A;
  st = host_arena(p, &A);
  if (st != PISA_OK) return st;
  if (ws_bytes < A.total) return PISA_ERR_WORKSPACE_TOO_SMALL;
  if ((st = side_streams()) != PISA_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t es = elem_size(p->dtype);
  char* base = (char*)ws;                                          // [fwd 0][fwd 1][pyramid 0][pyramid 1][slots]
  char* dpyr = base + 2 * A.fwd;
  char* slot0 = dpyr + 2 * A.pb;
  const int U = g.Hkv, G = g.G;
  const size_t rows = (size_t)g.B * g.N;                         // tokens of all batches
  const size_t q_w = (size_t)G * g.d * es, q_pitch = (size_t)g.Hq * g.d * es;
  const size_t k_w = (size_t)g.d * es, k_pitch = (size_t)g.Hkv * g.d * es;
  const size_t l_w = (size_t)G * g.N * sizeof(float), l_pitch = (size_t)g.Hq * g.N * sizeof(float);
  const size_t i_w = (size_t)g.N * g.K * sizeof(int32_t), i_pitch = (size_t)g.Hkv * i_w;

  // copy streams and the events that order the three stages of every unit
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_begin = nullptr, ev_in[kHostSlots] = {}, ev_v[kHostSlots] = {}, ev_routed[kHostSlots] = {},
              ev_done[kHostSlots] = {}, ev_out[kHostSlots] = {};
  cudaError_t e = cudaSuccess;
  const char* what = "copy streams";
  auto ok = [&](cudaError_t r, const char* w) { if (e == cudaSuccess && r != cudaSuccess) { e = r; what = w; } return e == cudaSuccess; };
  ok(cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking), "stream create");
  ok(cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking), "stream create");
  ok(cudaEventCreateWithFlags(&ev_begin, cudaEventDisableTiming), "event create");
  cudaStream_t cs[2] = {s, g_side[1]};                             // compute streams
  for (int i = 0; i < kHostSlots; ++i) {
    ok(cudaEventCreateWithFlags(&ev_in[i], cudaEventDisableTiming), "event create");
    ok(cudaEventCreateWithFlags(&ev_v[i], cudaEventDisableTiming), "event create");
    ok(cudaEventCreateWithFlags(&ev_routed[i], cudaEventDisableTiming), "event create");
    ok(cudaEventCreateWithFlags(&ev_done[i], cudaEventDisableTiming), "event create");
    ok(cudaEventCreateWithFlags(&ev_out[i], cudaEventDisableTiming), "event create");
  }
  // work already queued on the caller's stream comes first
  if (e == cudaSuccess) {
    ok(cudaEventRecord(ev_begin, s), "event record");
    ok(cudaStreamWaitEvent(s_in, ev_begin, 0), "stream wait");
    ok(cudaStreamWaitEvent(s_out, ev_begin, 0), "stream wait");
  }
  st = (e == cudaSuccess) ? clear_status(ws, s) : PISA_OK;
  if (e == cudaSuccess && st == PISA_OK) st = clear_status(base + A.fwd, s);   // the second workspace's status word
  if (e == cudaSuccess) {
    ok(cudaEventRecord(ev_begin, s), "event record");
    ok(cudaStreamWaitEvent(cs[1], ev_begin, 0), "stream wait");
  }
  for (int u = 0; u < U && e == cudaSuccess && st == PISA_OK; ++u) {
    const int sl = u % kHostSlots, ci = u & 1;
    char* dq = slot0 + sl * A.slot;
    char* dout = dq + A.qb;
    char* dk = dout + A.qb;
    char* dv = dk + A.kb;
    char* dl = dv + A.kb;
    char* di = dl + A.lb;
    // stage 1: inputs of unit u (its slot was last read by the kernels of the unit that had it before)
    if (u >= kHostSlots) ok(cudaStreamWaitEvent(s_in, ev_done[sl], 0), "stream wait");
    // keys and queries first: the pyramid and the routing start on them while the values are still copied
    ok(cudaMemcpy2DAsync(dk, k_w, (const char*)k_host + (size_t)u * k_w, k_pitch, k_w, rows, cudaMemcpyHostToDevice, s_in), "h2d copy");
    ok(cudaMemcpy2DAsync(dq, q_w, (const char*)q_host + (size_t)u * q_w, q_pitch, q_w, rows, cudaMemcpyHostToDevice, s_in), "h2d copy");
    ok(cudaEventRecord(ev_in[sl], s_in), "event record");
    ok(cudaMemcpy2DAsync(dv, k_w, (const char*)v_host + (size_t)u * k_w, k_pitch, k_w, rows, cudaMemcpyHostToDevice, s_in), "h2d copy");
    ok(cudaEventRecord(ev_v[sl], s_in), "event record");
    // stage 2: the kernels (the slot's outputs were last read by the copies of its previous unit); the
    // workspace and pyramid of this compute stream were last used by unit u-2, earlier on the same stream
    ok(cudaStreamWaitEvent(cs[ci], ev_in[sl], 0), "stream wait");
    if (u >= kHostSlots) ok(cudaStreamWaitEvent(cs[ci], ev_out[sl], 0), "stream wait");
    if (e != cudaSuccess) break;
    st = do_forward(&A.unit, A.ug, dq, dk, dv, dpyr + ci * A.pb, (int32_t*)di, dout, (float*)dl, base + ci * A.fwd,
                    A.fwd, cs[ci], /*clear=*/false, ev_v[sl], ev_routed[sl]);
    if (st != PISA_OK) break;
    ok(cudaEventRecord(ev_done[sl], cs[ci]), "event record");
    // stage 3: results of unit u; the indices leave as soon as the routing has written them
    if (idx_host) {
      ok(cudaStreamWaitEvent(s_out, ev_routed[sl], 0), "stream wait");
      ok(cudaMemcpy2DAsync((char*)idx_host + (size_t)u * i_w, i_pitch, di, i_w, i_w, (size_t)g.B, cudaMemcpyDeviceToHost, s_out), "d2h copy");
    }
    ok(cudaStreamWaitEvent(s_out, ev_done[sl], 0), "stream wait");
    ok(cudaMemcpy2DAsync((char*)out_host + (size_t)u * q_w, q_pitch, dout, q_w, q_w, rows, cudaMemcpyDeviceToHost, s_out), "d2h copy");
    ok(cudaMemcpy2DAsync((char*)lse_host + (size_t)u * l_w, l_pitch, dl, l_w, l_w, (size_t)g.B, cudaMemcpyDeviceToHost, s_out), "d2h copy");
    ok(cudaEventRecord(ev_out[sl], s_out), "event record");
  }
  // everything this call queued must be finished before its streams and events go away
  if (s_in) ok(cudaStreamSynchronize(s_in), "stream sync");
  ok(cudaStreamSynchronize(s), "stream sync");
  ok(cudaStreamSynchronize(cs[1]), "stream sync");
  if (s_out) ok(cudaStreamSynchronize(s_out), "stream sync");
  // a device-side error of the second compute stream shows in the status word the caller reads
  if (e == cudaSuccess) {
    int32_t w1 = 0, w0 = 0;
    ok(cudaMemcpy(&w1, base + A.fwd, sizeof(w1), cudaMemcpyDeviceToHost), "status read");
    ok(cudaMemcpy(&w0, base, sizeof(w0), cudaMemcpyDeviceToHost), "status read");
    if (e == cudaSuccess && w1 != 0 && w0 == 0) ok(cudaMemcpy(base, &w1, sizeof(w1), cudaMemcpyHostToDevice), "status write");
  }
  for (int i = 0; i < kHostSlots; ++i) {
    if (ev_in[i]) cudaEventDestroy(ev_in[i]);
    if (ev_v[i]) cudaEventDestroy(ev_v[i]);
    if (ev_routed[i]) cudaEventDestroy(ev_routed[i]);
    if (ev_done[i]) cudaEventDestroy(ev_done[i]);
    if (ev_out[i]) cudaEventDestroy(ev_out[i]);
  }
  if (ev_begin) cudaEventDestroy(ev_begin);
  if (s_in) cudaStreamDestroy(s_in);
  if (s_out) cudaStreamDestroy(s_out);
  if (e != cudaSuccess) { record_cuda_error(what, e); return PISA_ERR_CUDA; }
  return st;
}

int pisa_bsa_bwd(const pisa_params_t* p, const void* q, const void* k, const void* v, const int32_t* idx,
                 const void* out, const float* lse, const void* dout, void* dq, void* dk, void* dv,
                 void* ws, size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q || !k || !v || !idx || !out || !lse || !dout || !dq || !dk || !dv || !ws) return PISA_ERR_INVALID_ARG;
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out) || misaligned(dout) || misaligned(dq) ||
      misaligned(dk) || misaligned(dv) || misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  if (!tensor_bwd_supported(g, p->dtype) || p->impl == PISA_IMPL_SIMT) return PISA_ERR_UNSUPPORTED;
  {
    ForwardPlan pl;                            // sizes are checked before anything is queued
    if ((st = plan_for(p, g, kOpBwd, ws_bytes, &pl)) != PISA_OK) return st;
  }
  cudaStream_t s = (cudaStream_t)stream;
  st = clear_status(ws, s);
  if (st != PISA_OK) return st;
  g_mark_n = 0;
  st = do_bwd(p, g, q, k, v, idx, out, lse, dout, dq, dk, dv, ws, ws_bytes, s);
  kernel_mark("end", s);
  return st;
}

int pisa_bsa_bwd_packed(const pisa_params_t* p, const int32_t* cu_seqlens, int32_t nseq, const void* q,
                        const void* k, const void* v, const int32_t* idx, const void* out, const float* lse,
                        const void* dout, void* dq, void* dk, void* dv, void* ws, size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!cu_seqlens || nseq < 0 || !q || !k || !v || !idx || !out || !lse || !dout || !dq || !dk || !dv || !ws)
    return PISA_ERR_INVALID_ARG;
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out) || misaligned(dout) || misaligned(dq) ||
      misaligned(dk) || misaligned(dv) || misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  if (p->B != 1 || cu_seqlens[0] != 0) return PISA_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i)
    if (p->q_stride[i] || p->k_stride[i] || p->v_stride[i] || p->o_stride[i]) return PISA_ERR_INVALID_ARG;
  if (p->impl == PISA_IMPL_SIMT) return PISA_ERR_UNSUPPORTED;
  // everything is checked before anything is queued
  for (int i = 0; i < nseq; ++i) {
    const int len = cu_seqlens[i + 1] - cu_seqlens[i];
    if (len < 0 || len > p->N) return PISA_ERR_INVALID_ARG;
    if (len == 0) continue;
    pisa_params_t pi = *p;
    pi.N = len;
    Geometry gi;
    st = resolve(&pi, &gi);
    if (st != PISA_OK) return st;
    if (!tensor_bwd_supported(gi, p->dtype)) return PISA_ERR_UNSUPPORTED;
    if (ws_bytes < kStatusBytes + tensor_bwd_workspace_bytes(gi)) return PISA_ERR_WORKSPACE_TOO_SMALL;
  }
  cudaStream_t s = (cudaStream_t)stream;
  st = clear_status(ws, s);
  if (st != PISA_OK) return st;
  g_mark_n = 0;
  const size_t es = elem_size(p->dtype);
  auto run_alone = [&](int i, size_t wsb) -> int {
    const size_t t0 = (size_t)cu_seqlens[i];
    const int len = cu_seqlens[i + 1] - cu_seqlens[i];
    if (len == 0) return PISA_OK;
    pisa_params_t pi = *p;
    pi.N = len;
    Geometry gi;
    const int r = resolve(&pi, &gi);
    if (r != PISA_OK) return r;
    const size_t oq = t0 * g.Hq * g.d * es, ok = t0 * g.Hkv * g.d * es;
    return do_bwd(&pi, gi, (const char*)q + oq, (const char*)k + ok, (const char*)v + ok, idx + t0 * g.Hkv * g.K,
                  (const char*)out + oq, lse + t0 * g.Hq, (const char*)dout + oq, (char*)dq + oq, (char*)dk + ok,
                  (char*)dv + ok, ws, wsb, s);
  };
  // With a workspace sized for PISA_OP_BSA_BWD_PACKED the short sequences run in the forward's padded groups (a
  // padded query row gets idx = -1: it has no blocks and adds nothing to any key's gradient); with the smaller
  // PISA_OP_BSA_BWD one, one sequence after the other.
  PackedBwdArena pa;
  const bool grouped = packed_bwd_arena(p, &pa) == PISA_OK && ws_bytes >= pa.total;
  if (!grouped) {
    for (int i = 0; i < nseq; ++i)
      if ((st = run_alone(i, ws_bytes)) != PISA_OK) return st;
    kernel_mark("end", s);
    return PISA_OK;
  }
  std::unique_ptr<int[]> order(new (std::nothrow) int[(size_t)nseq + 1]);
  std::unique_ptr<int32_t[]> group(new (std::nothrow) int32_t[(size_t)nseq + 1]);
  std::unique_ptr<int32_t[]> padded(new (std::nothrow) int32_t[(size_t)nseq + 1]);
  if (!order || !group || !padded) return PISA_ERR_INVALID_ARG;
  packed_plan(p, cu_seqlens, nseq, pa.tokens, order.get(), group.get(), padded.get());
  for (int i = 0; i < nseq; ++i)
    if (group[i] < 0 && (st = run_alone(i, pa.bwd)) != PISA_OK) return st;
  char* q_pad = (char*)ws + pa.bwd;
  char* o_pad = q_pad + pa.qb;
  char* do_pad = o_pad + pa.qb;
  char* dq_pad = do_pad + pa.qb;
  char* k_pad = dq_pad + pa.qb;
  char* v_pad = k_pad + pa.kb;
  char* dk_pad = v_pad + pa.kb;
  char* dv_pad = dk_pad + pa.kb;
  float* l_pad = (float*)(dv_pad + pa.kb);
  int32_t* i_pad = (int32_t*)((char*)l_pad + pa.lb);
  size_t n_short = 0;
  for (int i = 0; i < nseq; ++i) {
    const int len = cu_seqlens[i + 1] - cu_seqlens[i];
    if (len > 0 && len <= kPackDirectLen) ++n_short;
  }
  size_t at = 0;
  while (at < n_short) {
    const int first = order[at];
    if (group[first] < 0) { ++at; continue; }
    size_t end = at + 1;
    while (end < n_short && group[order[end]] == group[first]) ++end;
    const int nb = (int)(end - at), np = padded[first];
    pisa_params_t pg = *p;
    pg.B = nb;
    pg.N = np;
    Geometry gg;
    if ((st = resolve(&pg, &gg)) != PISA_OK) return st;
    PackTable tab;
    auto fill = [&](int b0) {
      tab.n = nb - b0 < kPackSeqs ? nb - b0 : kPackSeqs;
      for (int j = 0; j < tab.n; ++j) {
        const int sq = order[at + (size_t)b0 + j];
        tab.off[j] = cu_seqlens[sq];
        tab.len[j] = cu_seqlens[sq + 1] - cu_seqlens[sq];
      }
    };
    for (int b0 = 0; b0 < nb; b0 += kPackSeqs) {
      fill(b0);
      if ((st = launch_pack_gather(gg, (int)es, q, k, v, q_pad, k_pad, v_pad, tab, b0, s)) != PISA_OK) return st;
      st = launch_pack_gather_bwd(gg, (int)es, out, dout, idx, lse, o_pad, do_pad, i_pad, l_pad, tab, b0, s);
      if (st != PISA_OK) return st;
    }
    st = do_bwd(&pg, gg, q_pad, k_pad, v_pad, i_pad, o_pad, l_pad, do_pad, dq_pad, dk_pad, dv_pad, ws, pa.bwd, s);
    if (st != PISA_OK) return st;
    for (int b0 = 0; b0 < nb; b0 += kPackSeqs) {
      fill(b0);
      st = launch_pack_scatter_grads(gg, (int)es, dq_pad, dk_pad, dv_pad, dq, dk, dv, tab, b0, s);
      if (st != PISA_OK) return st;
    }
    at = end;
  }
  kernel_mark("end", s);
  return PISA_OK;
}

int pisa_decode_step(const pisa_params_t* p, int32_t pos, const void* q, const void* k_cache,
                     const void* v_cache, void* pyramid, int32_t* idx, void* out, float* lse,
                     void* ws, size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q || !k_cache || !v_cache || !pyramid || !idx || !out || !lse || !ws) return PISA_ERR_INVALID_ARG;
  if (misaligned(q) || misaligned(k_cache) || misaligned(v_cache) || misaligned32(pyramid) || misaligned(ws))
    return PISA_ERR_INVALID_ARG;
  if (pos < 0 || pos >= g.N) return PISA_ERR_INVALID_ARG;
  if (!decode_supported(g, p->dtype)) return PISA_ERR_UNSUPPORTED;
  if (ws_bytes < kStatusBytes + decode_workspace_bytes(g)) return PISA_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t s = (cudaStream_t)stream;
  kernel_mark("decode_step", s);
  st = launch_decode_step(g, pos, q, k_cache, v_cache, pyramid, idx, out, lse, (char*)ws + kStatusBytes, s);
  kernel_mark("end", s);
  return st;
}

int pisa_pyramid_regrow(const pisa_params_t* p_old, const pisa_params_t* p_new, const void* pyramid_old,
                        void* pyramid_new, void* stream) {
  Geometry go, gn;
  int st = resolve(p_old, &go);
  if (st != PISA_OK) return st;
  st = resolve(p_new, &gn);
  if (st != PISA_OK) return st;
  if (!pyramid_old || !pyramid_new || misaligned32(pyramid_old) || misaligned32(pyramid_new)) return PISA_ERR_INVALID_ARG;
  if (go.B != gn.B || go.Hkv != gn.Hkv || go.d != gn.d || go.C != gn.C || go.g != gn.g ||
      p_old->dtype != p_new->dtype || gn.N < go.N)
    return PISA_ERR_INVALID_ARG;
  const size_t es = elem_size(p_old->dtype);
  for (int l = 1; l <= go.L; ++l) {
    const size_t w = (size_t)go.M[l] * go.d * es;           // one (b, KV head) of the old level
    cudaError_t e = cudaMemcpy2DAsync((char*)pyramid_new + (size_t)gn.level_off[l] * es, (size_t)gn.M[l] * gn.d * es,
                                      (const char*)pyramid_old + (size_t)go.level_off[l] * es, w, w,
                                      (size_t)go.B * go.Hkv, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
    if (e != cudaSuccess) { record_cuda_error("pyramid regrow", e); return PISA_ERR_CUDA; }
  }
  return PISA_OK;
}

int pisa_flat_select(const pisa_params_t* p, const void* q, const void* pyramid, int32_t* idx, void* ws,
                     size_t ws_bytes, void* stream) {
  Geometry g;
  int st = resolve(p, &g);
  if (st != PISA_OK) return st;
  if (!q || !pyramid || !idx || !ws || misaligned(q) || misaligned32(pyramid)) return PISA_ERR_INVALID_ARG;
  if (ws_bytes < kStatusBytes) return PISA_ERR_WORKSPACE_TOO_SMALL;
  st = clear_status(ws, (cudaStream_t)stream);
  if (st != PISA_OK) return st;
  if (p->impl != PISA_IMPL_SIMT && flat_tc_supported(g, p->dtype)) {
    kernel_mark("flat_tc", (cudaStream_t)stream);
    st = launch_flat_tc(g, q, pyramid, idx, (int32_t*)ws, (cudaStream_t)stream);
    kernel_mark("end", (cudaStream_t)stream);
    return st;
  }
  return launch_flat_simt(g, p->dtype, q, pyramid, idx, (cudaStream_t)stream);
}

int pisa_read_status(const void* ws, int32_t* status) {
  if (!ws || !status) return PISA_ERR_INVALID_ARG;
  int32_t word = 0;
  cudaError_t e = cudaMemcpy(&word, ws, sizeof(word), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) { record_cuda_error("status read", e); return PISA_ERR_CUDA; }
  *status = word;
  return PISA_OK;
}

int pisa_debug_wait_timeout(void* ws, unsigned long long limit_ns, void* stream) {
  if (!ws || misaligned(ws)) return PISA_ERR_INVALID_ARG;
  if (limit_ns < 1000ull) limit_ns = 1000ull;
  if (limit_ns > 1000000000ull) limit_ns = 1000000000ull;
  int st = clear_status(ws, (cudaStream_t)stream);
  if (st != PISA_OK) return st;
  return launch_wait_timeout((int32_t*)ws, limit_ns, (cudaStream_t)stream);
}

int pisa_get_kernel_ms(int i, char* name, size_t name_len, float* ms) {
  if (!g_timing || !g_mark_valid || i < 0 || i >= g_mark_n) return PISA_ERR_INVALID_ARG;
  int j = i + 1;
  while (j < g_mark_n && g_mark_stream[j] != g_mark_stream[i]) ++j;
  float t = 0.f;
  if (j < g_mark_n) {
    cudaError_t e = cudaEventSynchronize(g_mark_ev[j]);
    if (e != cudaSuccess) { record_cuda_error("kernel events", e); return PISA_ERR_CUDA; }
    cudaEventElapsedTime(&t, g_mark_ev[i], g_mark_ev[j]);
  }
  if (ms) *ms = t;
  if (name && name_len > 0) snprintf(name, name_len, "%s", (j < g_mark_n) ? g_mark_name[i] : "end");
  return PISA_OK;
}

int pisa_set_forward_chunks(int max_chunks) {
  if (max_chunks < 0) return PISA_ERR_INVALID_ARG;
  g_chunk_limit = max_chunks;
  return PISA_OK;
}

unsigned long long pisa_launch_count(void) { return __atomic_load_n(&g_launches, __ATOMIC_RELAXED); }

int pisa_set_stage_timing(int enable) {
  g_timing = enable != 0;
  return PISA_OK;
}

int pisa_get_stage_ms(float* pyramid_ms, float* route_ms, float* attn_ms) {
  if (!g_timing || !g_ev_valid) return PISA_ERR_INVALID_ARG;
  cudaError_t e = cudaEventSynchronize(g_ev[3]);
  if (e != cudaSuccess) { record_cuda_error("stage events", e); return PISA_ERR_CUDA; }
  float a = 0, b = 0, c = 0;
  cudaEventElapsedTime(&a, g_ev[0], g_ev[1]);
  cudaEventElapsedTime(&b, g_ev[1], g_ev[2]);
  cudaEventElapsedTime(&c, g_ev[2], g_ev[3]);
  if (pyramid_ms) *pyramid_ms = a;
  if (route_ms) *route_ms = b;
  if (attn_ms) *attn_ms = c;
  return PISA_OK;
}

}  // extern "C"
