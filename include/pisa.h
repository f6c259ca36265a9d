/*
 * libpisa — Pyramid Sparse Attention (PISA) on NVIDIA B200 (sm_100a): the forward hot path (pyramid,
 * routing, block-sparse attention), the decoding step and the attention backward.
 *
 * C ABI.  Every pointer is caller-owned.  "device" pointers are CUDA global memory of the
 * current device, "host" pointers are ordinary host memory.  The library never allocates or
 * frees device memory and, except where stated, never synchronises: all work is enqueued on
 * `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).  Scratch comes
 * from a caller-provided workspace whose size is queried with pisa_workspace_bytes().
 *
 * Notation follows the paper (Sec. 3.1-3.2): N tokens, Hq query heads, Hkv KV heads
 * (G = Hq/Hkv heads share KV head h: heads h*G .. h*G+G-1), head dim d, leaf block size C,
 * pooling fan-in g above the leaves, block budget K, M_1 = ceil(N/C) leaf blocks,
 * M_{l+1} = ceil(M_l/g), L = first level with M_L = 1.  Everything is 0-based.
 *
 * Tensor layouts (d contiguous, strides in elements, order (b, n, h)):
 *   q, out : [B, N, Hq,  d]      k, v : [B, N, Hkv, d]
 *   idx    : int32 [B, Hkv, N, K]   ascending leaf-block ids, padded with -1
 *   lse    : float [B, Hq, N]       natural-log softmax denominator
 *   pyramid: levels 1..L back to back, level l = [B, Hkv, M_l, d] in the input dtype,
 *            at the element offsets pisa_pyramid_layout() reports.
 *
 * All functions return a pisa_status (0 = OK).  Nothing aborts, throws or traps the GPU.
 */
#ifndef PISA_H_
#define PISA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PISA_VERSION 100

typedef enum {
  PISA_OK = 0,
  PISA_ERR_INVALID_ARG = -1,         /* null pointer, non-positive size, Hq % Hkv != 0, K < 3, g < 2 */
  PISA_ERR_UNSUPPORTED = -2,         /* causal = 0, d / G / g*K outside the built range, unknown dtype */
  PISA_ERR_WORKSPACE_TOO_SMALL = -3,
  PISA_ERR_CUDA = -4,                /* a launch or copy failed; pisa_last_cuda_error() has the text */
  PISA_ERR_TIMEOUT = -5,             /* a bounded device-side wait gave up (read from the status word) */
  PISA_ERR_BOUNDS = -6,              /* a device-side index check failed (read from the status word) */
  PISA_ERR_STATIC_SCRATCH_TOO_SMALL = -7  /* pisa_route_static: the problem needs more scratch than the
                                             library's built-in device array holds */
} pisa_status;

enum { PISA_BF16 = 0, PISA_FP32 = 1 };
/* Block score (Sec. 4.3, App. A.2): PISA = log-sum-exp, PISA-1 = mean logit, PISA-2 = mean + var/2 */
enum { PISA_SCORE_LSE = 0, PISA_SCORE_MEAN = 1, PISA_SCORE_MEAN_VAR = 2 };
/* operations a workspace can be sized for */
enum { PISA_OP_ROUTE = 0, PISA_OP_BSA = 1, PISA_OP_FORWARD = 2, PISA_OP_FLAT = 3, PISA_OP_FORWARD_HOST = 4,
       PISA_OP_DECODE = 5, PISA_OP_BSA_BWD = 6, PISA_OP_FORWARD_PACKED = 7,
       PISA_OP_BSA_BWD_PACKED = 8 };
/* implementation selector (params.impl): AUTO picks the tensor-core path where it applies */
enum { PISA_IMPL_AUTO = 0, PISA_IMPL_SIMT = 1, PISA_IMPL_TENSOR = 2 };
/*
 * params.debug bits.  PISA_DEBUG_BOUNDS: every index a kernel is about to gather or scatter with (token
 * positions, node / leaf ids read from idx, from the inverted lists or from intermediate routing
 * results, list slots) is range-checked on the device first; a value out of range is not used, the
 * access is skipped and PISA_ERR_BOUNDS lands in the workspace's status word (pisa_read_status).
 * Nothing traps.  In this mode an idx entry other than -1 that names a leaf which does not exist or
 * starts after the row's own leaf counts as out of range (without it such entries are silently
 * ignored).  The environment variable PISA_DEBUG=1 sets the bit for every call of the process.
 * Costs a few percent; meant for tests and for chasing a suspected stray index (no memory checker
 * can be attached to these kernels everywhere).
 */
enum { PISA_DEBUG_BOUNDS = 1 };

typedef struct {
  int32_t B, N, Hq, Hkv, d, C, g, K; /* prefill self-attention: N queries = N keys            */
  int32_t causal;                    /* must be 1: the paper defines only the causal LM case   */
  int32_t dtype;                     /* PISA_BF16 | PISA_FP32: q, k, v, out, summaries share it */
  int32_t score_mode;                /* PISA_SCORE_*                                            */
  int32_t impl;                      /* PISA_IMPL_*                                             */
  float   scale;                     /* logit scale, > 0; 0 => 1/sqrt(d)  (Eq. "block scores")  */
  int32_t debug;                     /* PISA_DEBUG_* bits; 0 = off                              */
  int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3]; /* elements, (b, n, h); all 0 => dense */
} pisa_params_t;

int pisa_version(void);
const char* pisa_status_string(int status);
/* text of the last CUDA error seen by this thread's calls ("" if none) */
const char* pisa_last_cuda_error(void);

/*
 * Hierarchy of Sec. 3.2 "Fine-to-coarse block aggregation".
 * Host-only.  Writes L, M[0..L] (M[0] = N; caller provides >= 34 entries) and level_off[0..L]
 * (element offset of level l inside the pyramid buffer; level_off[0] is unused), and the
 * buffer size in bytes.  Any output pointer may be NULL.  The pyramid buffer itself must start on
 * a 32-byte boundary wherever it is passed (every entry point that takes a pyramid checks it and
 * returns PISA_ERR_INVALID_ARG otherwise: the routing kernels read the summaries with 32-byte
 * loads); tensor pointers need 16 bytes.
 */
int pisa_pyramid_layout(const pisa_params_t* p, int32_t* L, int32_t* M, int64_t* level_off, size_t* bytes);

/* Host-only.  Bytes of device workspace `op` needs for these parameters (256-byte aligned base). */
int pisa_workspace_bytes(const pisa_params_t* p, int op, size_t* bytes);

/*
 * Eq. "mean pyramid": level 1 = mean of each leaf block's keys, level l+1 = unweighted mean of
 * the valid level-l children (fp32 accumulation, each level rounded to the input dtype and pooled
 * from the stored level below).  k: device [B,N,Hkv,d]; pyramid: device, pisa_pyramid_layout bytes.
 */
int pisa_build_pyramid(const pisa_params_t* p, const void* k, void* pyramid, void* stream);

/*
 * Coarse-to-fine Top-K block selection (Sec. 3.2 "Coarse-to-fine block selection", Eq. "direct
 * child LSE", Eq. "grouped score", App. B "Causal masking"): per (b, KV head, query token) start
 * from the root, drop candidates that do not exist or start after the query's leaf, keep all if
 * at most K remain, else keep the forced nodes (ancestors of the first / previous / current leaf,
 * never scored, counted inside K) plus the best of the rest by the group-summed score of their
 * children (g child summaries above the leaves, the C raw keys at the leaves), ties to the smaller
 * index; expand the kept nodes' children; the kept leaves are the result.
 *   q, k, pyramid : device inputs            idx : device int32 [B,Hkv,N,K] output
 *   sel_lse       : device float [B,Hq,N,K] or NULL — for every query head and kept slot s the
 *                   natural-log softmax denominator of the visible keys (j <= t) of leaf idx[b,h,t,s]
 *                   alone (-inf for a -1 slot).  The leaf scores of the LSE mode are exactly these
 *                   numbers, so the tensor-core routing has them for free; handing them to
 *                   pisa_bsa_fwd saves its own scoring pass over the selected blocks
 *   margin        : device float [B,Hkv,N] or NULL — smallest relative gap between the last kept
 *                   and the first dropped score over the scored levels (+inf if nothing was cut);
 *                   gap = (u_kept - u_dropped) / max(|u_kept|, 1)
 *   ws / ws_bytes : device workspace sized for PISA_OP_ROUTE
 */
int pisa_route(const pisa_params_t* p, const void* q, const void* k, const void* pyramid,
               int32_t* idx, float* sel_lse, float* margin, void* ws, size_t ws_bytes, void* stream);

/*
 * Eq. "selected sparse attention" with the causal mask inside selected blocks (App. B): for every
 * query head, softmax over the tokens j <= t of the leaf blocks idx[b, h, t, :] (entries < 0 are
 * skipped) with logits q.k*scale, fp32 accumulation.  out: device [B,N,Hq,d] in the input dtype;
 * lse: device float [B,Hq,N].  Workspace sized for PISA_OP_BSA.
 *   sel_lse : device float [B,Hq,N,K] or NULL — per-block denominators of exactly these idx as
 *             pisa_route wrote them; with them the tensor-core path skips its own pass over the
 *             selected blocks that would compute them (the exact-fp32 path ignores the argument)
 */
int pisa_bsa_fwd(const pisa_params_t* p, const void* q, const void* k, const void* v, const int32_t* idx,
                 const float* sel_lse, void* out, float* lse, void* ws, size_t ws_bytes, void* stream);

/*
 * pisa_route for callers that cannot provide a workspace because they are not allowed to allocate
 * device memory where they run (a memory pool that is fully assigned, a serving plugin that forbids
 * allocation after start-up, a loop that cannot afford cudaMalloc's implicit synchronisation).
 * (No counterpart in the paper: this is a property of the library, not of the method.)
 *
 * Same arguments and results as pisa_route, without ws / ws_bytes: the scratch is a 32 MiB device
 * array built into the library (pisa_route_static_capacity()), present on every GPU that loads the
 * library until the process exits.  The call allocates nothing, on the host or on the device.
 *  - Problems whose PISA_OP_ROUTE workspace exceeds the capacity are refused with
 *    PISA_ERR_STATIC_SCRATCH_TOO_SMALL before anything is launched.
 *  - The first call on each device looks up the array's device address (the device that is current
 *    at the call); make that first call outside any stream capture.
 *  - All calls on one device share the array, which keeps whatever the last call left in it; each
 *    call zeroes what it needs zeroed, on `stream`, before use.  Two calls that can overlap on the
 *    GPU (different streams, or different host threads without ordering) race on it: serialise them.
 *  - The device status word of this variant is not exposed; use pisa_route with your own workspace
 *    where you need pisa_read_status.  Keep stage timing off (the default) for an allocation-free call.
 */
int pisa_route_static(const pisa_params_t* p, const void* q, const void* k, const void* pyramid,
                      int32_t* idx, float* margin, void* stream);
size_t pisa_route_static_capacity(void);

/*
 * pyramid -> route -> attention in one call.  pyramid and idx are outputs too (kept for reuse).
 * A large tensor-path problem is cut into up to four chunks of (batch, KV head) units that alternate
 * between `stream` and one stream the library owns (created on the first such call, per host
 * thread): the chunks' kernels stress different parts of the GPU and fill each other's tails.  The
 * internal stream forks from `stream` after the pyramid and joins it before the call's last
 * operation, so the call still behaves as ordered work on `stream` (and can be captured into a CUDA
 * graph).  The workspace query for PISA_OP_FORWARD covers both streams' scratch.  pisa_route and
 * pisa_bsa_fwd split large problems the same way.
 */
int pisa_forward(const pisa_params_t* p, const void* q, const void* k, const void* v, void* pyramid,
                 int32_t* idx, void* out, float* lse, void* ws, size_t ws_bytes, void* stream);

/*
 * Packed variable-length batches: `nseq` sequences laid back to back along the token axis.
 * Boundary rule (the paper leaves packed inputs open): every sequence has its own block grid that
 * starts at its first token, its own hierarchy and its own causal order; nothing is shared across
 * sequences, i.e. the result is what pisa_forward gives on each sequence alone.
 *
 *   p           : B must be 1 and strides dense; p->N is the LONGEST sequence (it sizes the pyramid
 *                 scratch and the workspace)
 *   cu_seqlens  : HOST int32 [nseq + 1], cu[0] = 0, non-decreasing; sequence i is tokens cu[i]..cu[i+1]-1
 *                 (empty sequences are skipped)
 *   q, out      : device [total, Hq, d];  k, v : device [total, Hkv, d]   (total = cu[nseq])
 *   pyramid     : device scratch sized by pisa_pyramid_layout for p (overwritten per sequence)
 *   idx         : device int32, sequence-major: sequence i's [Hkv, len_i, K] block starts at element
 *                 Hkv * K * cu[i]; block ids are relative to the sequence
 *   lse         : device float, sequence-major: sequence i's [Hq, len_i] block starts at Hq * cu[i]
 *   ws          : device workspace sized for PISA_OP_FORWARD_PACKED with p (N = the longest sequence)
 *
 * Launches.  The method is causal (Sec. 3.2: a query only ever scores nodes that lie wholly in its
 * past; the nodes on its own path are forced, not scored), so a sequence gives the same rows when it is
 * the head of a longer, zero-filled batch element.  Sequences of at most 8192 tokens are therefore
 * grouped by length (a group's members are no shorter than 3/4 of its padded length, padded lengths come
 * from the grid 1, 2, .., 15, then m * 2^k with m = 8..15, and a group holds at most 32768 padded tokens and at most 65535 / Hkv sequences), copied into a padded
 * batch inside the workspace, run through ONE set of launches of the batched forward, and the valid rows
 * copied back.  Longer sequences, and groups of one, run unpadded on the packed tensors.  With a
 * workspace sized for PISA_OP_FORWARD only (too small for the padded copies) the call runs the sequences
 * one after the other instead; the results are the same rows either way (up to the rounding order of
 * the fp32 partial sums).
 */
/*
 * The grouping pisa_forward_packed applies, as host arithmetic only (no GPU work, nothing allocated on the
 * device): for sequence i, group[i] = the padded batch it runs in (0, 1, ... in launch order) and
 * padded[i] = that batch's padded length; group[i] = -1 (padded[i] = its own length) for a sequence that
 * runs alone -- longer than 8192 tokens, alone in its length class, or empty.
 *   p, cu_seqlens, nseq : as for pisa_forward_packed
 *   group, padded       : HOST int32 [nseq], written
 *   n_groups            : HOST, nullable; receives the number of padded batches
 * Returns PISA_ERR_INVALID_ARG for null pointers, cu_seqlens[0] != 0, or a length outside [0, p->N].
 */
int pisa_packed_plan(const pisa_params_t* p, const int32_t* cu_seqlens, int32_t nseq, int32_t* group,
                     int32_t* padded, int32_t* n_groups);

int pisa_forward_packed(const pisa_params_t* p, const int32_t* cu_seqlens, int32_t nseq, const void* q,
                        const void* k, const void* v, void* pyramid, int32_t* idx, void* out, float* lse,
                        void* ws, size_t ws_bytes, void* stream);

/*
 * The same forward pass for callers that hold HOST tensors.  KV heads are independent units of the
 * path (Sec. 3.3: one selected set per KV head), so the call walks them one at a time: the strided
 * slice of q, k, v that belongs to head h is copied into one of four slots of the device arena
 * (`ws`, sized for PISA_OP_FORWARD_HOST: four slots of per-head tensors, two per-head pyramids and
 * two per-head forward workspaces), pisa_forward runs on it, and out, lse and (if not NULL) idx of
 * that head are copied back into their places in the host tensors.  The copies run on two internal
 * streams and the kernels of consecutive heads alternate between `stream` and a third internal
 * stream, so two heads' kernels are in flight while the next head is uploaded and the previous one
 * downloaded.  A head's keys and queries are copied first: its pyramid and routing start on them while
 * its values are still on the way, and its indices are copied back while its attention runs.
 * Host buffers should be pinned (pageable memory makes the copies synchronous); strides must be
 * dense.  Work already queued on `stream` is ordered before the call; the call returns after
 * everything it queued has finished.  This is the one entry point that synchronises.
 */
int pisa_forward_host(const pisa_params_t* p, const void* q_host, const void* k_host, const void* v_host,
                      void* out_host, float* lse_host, int32_t* idx_host,
                      void* ws, size_t ws_bytes, void* stream);

/*
 * Backward of the block-sparse attention (App. B).  idx is treated as a constant: only q, k and v
 * receive gradients, each through the softmax attention over its row's selected, visible keys.
 *
 *   q, k, v, idx   : as for pisa_bsa_fwd
 *   out, lse       : what pisa_bsa_fwd / pisa_forward produced for these idx (out with o_stride)
 *   dout           : gradient of the loss w.r.t. out, device, same dtype and strides as out
 *   dq             : device [B, N, Hq, d], dense, input dtype
 *   dk, dv         : device [B, N, Hkv, d], dense, input dtype; keys no query selected get zeros
 *   ws             : device workspace sized for PISA_OP_BSA_BWD (holds fp32 accumulators of all
 *                    three gradients; partial sums are added with fp32 reductions, so results are
 *                    reproducible to fp32 rounding, not bitwise)
 *
 * bf16, d in {64, 128}, C in {64, 128}; other configurations return PISA_ERR_UNSUPPORTED.
 * Asynchronous on `stream`.
 */
int pisa_bsa_bwd(const pisa_params_t* p, const void* q, const void* k, const void* v, const int32_t* idx,
                 const void* out, const float* lse, const void* dout, void* dq, void* dk, void* dv,
                 void* ws, size_t ws_bytes, void* stream);

/*
 * pisa_bsa_bwd for a packed variable-length batch laid out as for pisa_forward_packed (same boundary
 * rule: nothing is shared across sequences).
 *
 *   p, cu_seqlens, nseq : as for pisa_forward_packed (B = 1, dense strides, p->N the longest sequence)
 *   q, out, dout, dq    : device [total, Hq, d];  k, v, dk, dv : device [total, Hkv, d]
 *   idx, lse            : sequence-major, as pisa_forward_packed wrote them
 *   ws                  : device workspace sized for PISA_OP_BSA_BWD_PACKED with p: the short sequences then run in
 *                         the groups pisa_packed_plan reports, each group as one padded batch (a padded query row is
 *                         given idx = -1 and so contributes to no gradient); a workspace sized for PISA_OP_BSA_BWD
 *                         is accepted too and runs one backward per sequence
 *
 * All sequences are validated before anything is queued; one unsupported sequence fails the call.
 */
int pisa_bsa_bwd_packed(const pisa_params_t* p, const int32_t* cu_seqlens, int32_t nseq, const void* q,
                        const void* k, const void* v, const int32_t* idx, const void* out, const float* lse,
                        const void* dout, void* dq, void* dk, void* dv, void* ws, size_t ws_bytes, void* stream);

/*
 * Decoding (Sec. 3.3 "Decoding", App. B "Decode cache"): one new token per sequence, one kernel launch.
 *
 *   p->N             : CAPACITY of the caches in tokens (the pyramid layout is that of
 *                      pisa_pyramid_layout for this N); B, Hq, Hkv, d, C, g, K, scale as usual
 *   pos              : 0-based position of the new token, pos < p->N
 *   q                : device [B, Hq, d], dense (q_stride is ignored)
 *   k_cache, v_cache : device [B, N, Hkv, d] (k_stride / v_stride honoured); rows 0..pos hold the
 *                      sequence, the new token's key and value already written at row pos; rows
 *                      after pos are never read
 *   pyramid          : the cached pyramid, updated in place: the summary of the leaf that holds pos
 *                      becomes the mean of the keys it holds so far and each of its ancestors the mean
 *                      of its children up to the path (every other node is left as it is).  Nodes
 *                      that lie entirely after pos are never read, so the buffer needs no
 *                      initialisation: a cache built by calling this for pos = 0, 1, 2, ... , or by
 *                      pisa_build_pyramid over the first tokens followed by steps from there on,
 *                      holds the pyramid of keys 0..pos after every step
 *   idx              : device int32 [B, Hkv, K], ascending, -1 padded
 *   out, lse         : device [B, Hq, d] (input dtype), float [B, Hq]
 *   ws               : device workspace sized for PISA_OP_DECODE
 *
 * The step selects exactly what the prefill path selects for row pos of the same sequence (every
 * scored node lies strictly in the past of the query) and attends over keys <= pos of the selected
 * blocks.  bf16, every score mode, d in {64, 128}, C in {32, 64, 128}, group size <= 16; other
 * configurations return PISA_ERR_UNSUPPORTED.  Asynchronous on `stream`; allocates nothing.
 */
int pisa_decode_step(const pisa_params_t* p, int32_t pos, const void* q, const void* k_cache,
                     const void* v_cache, void* pyramid, int32_t* idx, void* out, float* lse,
                     void* ws, size_t ws_bytes, void* stream);

/*
 * Capacity growth of a cached pyramid (App. B "Decode cache": every level's buffer grows when more
 * space is needed): copies every level of `pyramid_old` (layout of p_old, capacity p_old->N) into
 * the layout of p_new (same shape parameters, p_new->N >= p_old->N) in `pyramid_new`.  The two
 * buffers must not overlap.  Levels that only the larger hierarchy has are rebuilt by the next
 * decoding steps along the path, as any other ancestor.
 */
int pisa_pyramid_regrow(const pisa_params_t* p_old, const pisa_params_t* p_new, const void* pyramid_old,
                        void* pyramid_new, void* stream);

/*
 * Flat block selection (Sec. 3.1, the O(N^2/C) reference point): score every eligible leaf with
 * q . level-1 summary * scale, softmax over the eligible leaves within each query head (App. C),
 * sum over the group's heads, keep the forced leaves plus the best of the rest.
 */
int pisa_flat_select(const pisa_params_t* p, const void* q, const void* pyramid, int32_t* idx,
                     void* ws, size_t ws_bytes, void* stream);

/*
 * Reads the device status word a workspace carries (written by bounded waits and index checks).
 * Call after the stream has been synchronised.  *status receives a pisa_status.
 */
int pisa_read_status(const void* ws, int32_t* status);

/*
 * Device time of the stages of the last pisa_forward / pisa_forward_host issued by this thread,
 * in milliseconds: pyramid, route, attention (measured with CUDA events on the call's stream).
 * Recording is off unless pisa_set_stage_timing(1) was called; the getter waits for the events.
 */
int pisa_set_stage_timing(int enable);
int pisa_get_stage_ms(float* pyramid_ms, float* route_ms, float* attn_ms);

/*
 * With stage timing on, pisa_forward also brackets its main kernels with events.  After a forward
 * call, entry i (0-based) gives the name of the i-th bracket and its device time in milliseconds
 * (from its event to the next one on the same stream; a name occurs once per chunk; the last bracket
 * of a stream is named "end" and has no time); PISA_ERR_INVALID_ARG past the last entry.  The getter
 * waits for the events.
 */
int pisa_get_kernel_ms(int i, char* name, size_t name_len, float* ms);

/*
 * Upper limit on the chunks pisa_forward, pisa_route and pisa_bsa_fwd cut a problem into, for the
 * calling host thread:
 * 0 = automatic (the default), 1 = never split (every kernel runs alone on `stream`, which is what a
 * per-kernel measurement wants).  Workspace sizes queried before stay sufficient.
 */
int pisa_set_forward_chunks(int max_chunks);

/* Number of kernels this process has launched through the library so far (host counter). */
unsigned long long pisa_launch_count(void);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper).  Every wait inside the
 * kernels (on an mbarrier another warp or the tensor pipe is to complete) gives up after a time
 * limit, records PISA_ERR_TIMEOUT in the workspace's status word, releases what it holds and lets
 * the kernel return, so that a scheduling bug can never hang the GPU.  This entry point launches one
 * CTA that waits, with the limit `limit_ns` (clamped to [1 us, 1 s]), on a barrier nobody arrives
 * at: after the stream has been synchronised pisa_read_status(ws) reports PISA_ERR_TIMEOUT and the
 * device remains usable.  ws: at least 256 bytes of device memory.
 */
int pisa_debug_wait_timeout(void* ws, unsigned long long limit_ns, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PISA_H_ */
