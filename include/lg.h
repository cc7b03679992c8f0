/*
 * lg.h -- C ABI of the LongGen efficient-layer attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the attention of LongGen's sparse layers (paper Section 3.1: a
 * static, block-wise pattern that is the same for every head -- attention sink plus
 * sliding window, or blockwise strided plus local blocks), the plain causal attention of
 * its full layers, and the serving side of Section 3.2 (a rolling-buffer KV cache for the
 * window with the sink kept beside it, and a bandwidth-bound decode over it).
 *
 * Conventions for every entry point
 *   - Pointers named in a signature as device pointers are device memory OWNED BY THE
 *     CALLER; the library allocates nothing that outlives a call and keeps no state
 *     between calls except what it writes into the caller's workspace.  Two exceptions, both
 *     documented where they are declared: the fixed scratch array of lg_sparse_decode_static
 *     (shared by all its calls on a device) and a diagnostic launch counter.
 *   - `stream` is a cudaStream_t (0 = default stream).  Calls enqueue work and return;
 *     the return value covers validation and launch only.  A device-side wait that gave
 *     up (every wait in the kernels is bounded) is reported by lg_last_status().
 *   - All tensors are bf16 with the head dimension D contiguous; device pointers must be
 *     16-byte aligned.  Results are bitwise reproducible for fixed inputs and parameters.
 *   - No exception crosses this boundary.  A call with invalid arguments launches nothing.
 */
#ifndef LG_H_
#define LG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LG_OK = 0,
  LG_ERR_INVALID_ARG = -1,    /* null / misaligned pointer, inconsistent sizes              */
  LG_ERR_UNSUPPORTED = -2,    /* valid problem outside what the kernels cover (e.g. D)      */
  LG_ERR_WORKSPACE = -3,      /* workspace_bytes smaller than the matching *_workspace_bytes */
  LG_ERR_CUDA = -4,           /* a CUDA runtime / driver call failed                         */
  LG_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait expired (see lg_last_status)     */
  LG_ERR_ARCH = -6            /* current device is not compute capability 10.x               */
} lg_status;

typedef enum {
  LG_MODE_FULL_CAUSAL = 0,   /* key j visible to query i iff j <= i (the full-attention layers)  */
  LG_MODE_SINK_WINDOW = 1,   /* Section 3.1 "Attention Sink": first blocks + most recent blocks   */
  LG_MODE_STRIDED_LOCAL = 2  /* Section 3.1 "block sparse": every stride-th block + local blocks  */
} lg_mode;

/*
 * Problem statement of one attention call (Sections 3.1 and 4.1).
 * With Bs = block, qb = i / Bs, kb = j / Bs, query i may attend key j iff j <= i and
 *   FULL_CAUSAL   : (nothing more)
 *   SINK_WINDOW   : kb < sink_tokens/Bs  or  qb - kb < window_tokens/Bs
 *                   (the window is block-granular and counts the query's own block: Section 4.1
 *                    keeps one sink block and the 32 latest blocks, the query's included);
 *                   with window_exact != 0 the second condition is i - j < window_tokens,
 *                   the token-exact window of the rolling-buffer cache (Section 3.2), so
 *                   that a model can be trained on exactly the keys lg_sparse_decode reads
 *   STRIDED_LOCAL : qb - kb < local_blocks  or  kb % stride_blocks == 0
 * Grouped-query attention: query head h reads kv head h / (Hq / Hkv).
 */
typedef struct {
  int32_t B, Hq, Hkv, L, D;   /* Hq % Hkv == 0; D in {64, 128}; L >= 1 (the last block may be partial) */
  int32_t block;              /* pattern granularity in tokens: 64 or 128                    */
  int32_t mode;               /* lg_mode                                                     */
  int32_t sink_tokens;        /* SINK_WINDOW: multiple of block (may be 0)                   */
  int32_t window_tokens;      /* SINK_WINDOW: multiple of block, >= block                    */
  int32_t stride_blocks;      /* STRIDED_LOCAL: >= 1                                         */
  int32_t local_blocks;       /* STRIDED_LOCAL: >= 1 (the diagonal block is always active)   */
  int32_t window_exact;       /* SINK_WINDOW: 0 = block-granular window, 1 = token-exact     */
  int32_t lists_prepared;     /* 0: the call builds the block lists itself (any workspace);
                                 1: the workspace was filled by lg_sparse_attn_prepare() for
                                 this pattern and the call only launches its attention kernels */
  float   scale;              /* softmax scale; 0 selects 1/sqrt(D)                          */
  /* Strides in ELEMENTS of (batch, head, token) for Q, K, V, O; dO and dQ use the O / Q
     strides, dK / dV the K / V strides.  All zero selects contiguous [B, H, L, D].
     Every stride must be a multiple of 8 elements (16 bytes).                              */
  int64_t q_strides[3], k_strides[3], v_strides[3], o_strides[3];
  /* Packed documents (optional; the paper packs documents, each opened by <bos>, into one
     sample and describes no masking between them): NULL, or a DEVICE int32 array [B, L],
     contiguous, with doc_start[b][i] = position of the first token of the document token i
     belongs to (non-decreasing in i, <= i).  When given, a query sees no key of an earlier
     document, on top of the pattern (which stays in absolute positions: the sink blocks are
     those of the sample, so only its first document sees them).  The calls drop every key
     block that ends before the earliest document of a query block starts; as the lists then
     differ between sequences, a call with B > 1 runs sequence by sequence (its workspace is
     B slices of the B == 1 size).
     lg_build_block_index ignores this field.                                                */
  const int32_t* doc_start;
} lg_attn_params;

/* ---- block-index builder (Section 3.2: the mask is kept in compressed-sparse-row form,
 *      O(N) memory, static for all heads) ---------------------------------------------- */

/* Number of active blocks (nnz) of the pattern, computed on the host; < 0 = lg_status. */
int64_t lg_block_index_nnz(const lg_attn_params* p);

/* Bytes needed for the four int32 arrays below, laid out back to back:
 * row_ptr[nB+1], col_idx[nnz], col_ptr[nB+1], row_idx[nnz] (nB = L / block). 0 on error. */
size_t lg_block_index_bytes(const lg_attn_params* p);

/* Fill the CSR lists (for each query block, the ascending KV blocks it attends) and the
 * CSC transpose (for each KV block, the ascending query blocks that attend it).
 * All four arrays are DEVICE int32 arrays of the sizes above, written by a kernel on
 * `stream`.  nnz_out_host (HOST, nullable) receives nnz.                                 */
lg_status lg_build_block_index(const lg_attn_params* p, int32_t* row_ptr, int32_t* col_idx,
                               int32_t* col_ptr, int32_t* row_idx, int64_t* nnz_out_host,
                               void* stream);

/* ---- training / prefill attention (Section 3.2: FlashAttention-style kernel that skips
 *      every block whose mask is zero, in the forward and in the backward) -------------- */

/* Workspace bytes for lg_sparse_attn_fwd (want_bwd == 0) or lg_sparse_attn_bwd (!= 0). */
size_t lg_sparse_attn_workspace_bytes(const lg_attn_params* p, int want_bwd);

/* Build the block lists and the kernels' tile schedules once (Section 3.2: the mask is static
 * and the same for all heads, so nothing has to be rebuilt from step to step).  Afterwards
 * lg_sparse_attn_fwd (and, with want_bwd != 0, lg_sparse_attn_bwd) called with the same
 * workspace, the same pattern (L, block, mode, sink / window / stride / local counts,
 * window_exact, doc_start pointer) and lists_prepared = 1 launch their attention kernels only:
 * one kernel for the forward, three for the backward.  The lists do not depend on the head
 * counts, on D or on the strides.  With doc_start the lists also depend on the CONTENTS of that
 * array: prepare again whenever they change.  The workspace keeps a fingerprint of what it was
 * prepared for; a call with lists_prepared = 1 whose pattern does not match it launches kernels
 * that do nothing, and lg_last_status() then returns LG_ERR_WORKSPACE.  In this mode the status
 * word is not cleared from call to call: a failure stays visible until lg_last_status() reads it,
 * and calls made in between do nothing.  workspace: device, 256-byte aligned,
 * lg_sparse_attn_workspace_bytes(p, want_bwd) bytes.                                       */
lg_status lg_sparse_attn_prepare(const lg_attn_params* p, void* workspace, size_t workspace_bytes,
                                 int want_bwd, void* stream);

/* O = softmax(scale * Q K^T + mask) V;  LSE_i = ln sum_j exp(scale * q_i . k_j) over the
 * visible keys.  q [B,Hq,L,D], k, v [B,Hkv,L,D], o [B,Hq,L,D] bf16 (device);
 * lse [B,Hq,L] fp32 contiguous (device).  workspace: device, 256-byte aligned.           */
lg_status lg_sparse_attn_fwd(const lg_attn_params* p, const void* q, const void* k, const void* v,
                             void* o, float* lse, void* workspace, size_t workspace_bytes,
                             void* stream);

/* Gradients of sum(O * dO): dq [B,Hq,L,D], dk, dv [B,Hkv,L,D] bf16 (device), from the
 * forward's inputs, its outputs o and lse, and d_o [B,Hq,L,D] bf16.  dK and dV of a kv head
 * are summed over the query heads of its group.  Keys a query may not see receive exactly
 * zero from it.  Accumulation order is fixed (no atomics).                               */
lg_status lg_sparse_attn_bwd(const lg_attn_params* p, const void* q, const void* k, const void* v,
                             const void* o, const float* lse, const void* d_o,
                             void* dq, void* dk, void* dv,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Which of its two equivalent backward variants lg_sparse_attn_bwd runs for `p` (the workspace size
 * reflects the choice): 0 = two passes, the dQ pass recomputing S and dP; 2 = the dK/dV pass also
 * writes dS (bf16, 2 bytes per pair of every block of the pattern and query head) to the workspace and
 * the dQ pass is the single product dQ = dS K.  The second is chosen when that buffer takes at most
 * 40 % of the current device's memory (or LG_KEEP_DS_MAX_GB gigabytes, where the environment sets it;
 * 48 GB where no device can be asked) and the block lists are shared by the batch; the environment
 * variable LG_BWD_VARIANT = two_pass | keep_ds overrides the choice.  Both give bitwise reproducible
 * results; they differ from one another in the last bits (dS is rounded to bf16 once either way, but the
 * order of the fp32 sums differs).  < 0 = lg_status.  (The paper has no counterpart.)            */
int32_t lg_sparse_attn_bwd_variant(const lg_attn_params* p);

/* Same computation as lg_sparse_attn_bwd; in addition the CUDA events of the caller are recorded on
 * `stream` around its kernels: events[0] before the first one, events[1] after the pre-pass
 * (delta), events[2] after the dK/dV pass, events[3] after the dQ pass.  `events` is a HOST array
 * of four cudaEvent_t created by the caller (with timing enabled if durations are wanted).  The
 * call creates nothing and does not synchronise; the caller reads the events when the stream has
 * passed them.  With doc_start and B > 1 (sequence-by-sequence execution) the events bracket the
 * first sequence only.  (The paper has no counterpart; a benchmark uses it to report per-kernel
 * durations.)                                                                              */
lg_status lg_sparse_attn_bwd_marked(const lg_attn_params* p, const void* q, const void* k,
                                    const void* v, const void* o, const float* lse,
                                    const void* d_o, void* dq, void* dk, void* dv,
                                    void* workspace, size_t workspace_bytes, void* stream,
                                    void* const* events);

/* ---- a whole training step on HOST buffers ---------------------------------------------- */

/*
 * Forward + backward of one attention call whose inputs and results live in HOST memory (pinned,
 * for the copies to overlap): q, k, v, d_o are copied to the device, lg_sparse_attn_fwd and
 * lg_sparse_attn_bwd run there, and o, lse, dq, dk, dv are copied back.  (The paper has no
 * counterpart: its kernels sit inside a trainer whose activations are already on the GPU; this is
 * the end-to-end form of the same two calls for a caller who holds host tensors.)
 *
 * Heads are independent, so the step is cut into `head_groups` groups of kv heads (with their
 * query heads) that move through three streams: while one group computes on `stream_compute`, the
 * next one's inputs arrive on `stream_in` and the previous one's results leave on `stream_out`;
 * the two copy directions share the link.  head_groups must divide Hkv (1 = no pipelining).
 *
 *   host tensors   : contiguous [B,H,L,D] bf16 (lse_host [B,Hq,L] fp32); the strides in `p` are
 *                    ignored.  doc_start in `p` (a DEVICE array, as always) is honoured.
 *   dev            : DEVICE staging buffers of the same shapes, owned by the caller, and one
 *                    workspace of lg_sparse_attn_fwd_bwd_host_workspace_bytes() bytes (256-byte
 *                    aligned), which the call cuts into one slice per group.
 *   streams        : three cudaStream_t of the caller.  The call waits for nothing that was
 *                    enqueued on them before; it creates a few timing-less CUDA events for the
 *                    hand-over between the streams and destroys them before returning.  On
 *                    return everything is enqueued; the host results are complete when
 *                    stream_out is idle (stream_in and stream_compute are then idle too).
 * Results are bit-identical to the two device calls on the whole tensors.  lg_last_status() on
 * dev->workspace reports a device-side failure of any group.
 */
typedef struct {
  void* q; void* k; void* v; void* d_o;      /* inputs  [B,Hq,L,D], [B,Hkv,L,D] x2, [B,Hq,L,D] */
  void* o; float* lse; void* dq; void* dk; void* dv;
  void* workspace;
  size_t workspace_bytes;
} lg_device_step_buffers;

size_t lg_sparse_attn_fwd_bwd_host_workspace_bytes(const lg_attn_params* p, int head_groups);

lg_status lg_sparse_attn_fwd_bwd_host(const lg_attn_params* p,
                                      const void* q_host, const void* k_host, const void* v_host,
                                      const void* d_o_host,
                                      void* o_host, float* lse_host, void* dq_host, void* dk_host,
                                      void* dv_host,
                                      const lg_device_step_buffers* dev, int head_groups,
                                      void* stream_in, void* stream_compute, void* stream_out);

/* ---- serving: rolling-buffer cache and decode (Section 3.2) --------------------------- */

/*
 * Cache layout: K and V each [B, Hkv, sink_tokens + window_tokens, D] bf16, contiguous.
 * Token j of a sequence lives in slot(j) = j < sink ? j : sink + (j - sink) % window.
 * A plain linear cache of `cap` tokens is sink_tokens = 0, window_tokens = cap.
 */
typedef struct {
  int32_t B, Hq, Hkv, D;       /* D in {64, 128}; Hq % Hkv == 0                              */
  int32_t sink_tokens;         /* >= 0                                                       */
  int32_t window_tokens;       /* >= 1                                                       */
  int32_t block_tokens;        /* 0: the query attends every token the cache holds (the token-exact
                                  window of Section 3.2's rolling buffer, the same keys as
                                  window_exact = 1 in training).  Bs > 0: the block-granular window
                                  of Section 4.1 that the default training mask uses -- the query at
                                  position n - 1 attends the sink and the tokens j with
                                  (n-1)/Bs - j/Bs < window_tokens/Bs; sink_tokens and window_tokens
                                  must be multiples of Bs.  The cache layout is the same either way
                                  (the ring still holds window_tokens tokens; up to Bs - 1 of the
                                  oldest are then read but not attended).  lg_kv_ring_append
                                  ignores this field.                                         */
  float   scale;               /* 0 selects 1/sqrt(D)                                        */
} lg_decode_params;

/* Append T_new tokens per sequence: k_new, v_new [B, Hkv, T_new, D] bf16 (device);
 * n_tokens_before (device int64 [B]) = tokens already appended to each sequence.  The
 * result equals appending one token at a time; writes that a later token of the same
 * call would overwrite are skipped.  A sequence whose count is negative is left untouched. */
lg_status lg_kv_ring_append(const lg_decode_params* p, void* k_cache, void* v_cache,
                            const void* k_new, const void* v_new, int32_t T_new,
                            const int64_t* n_tokens_before, void* stream);

size_t lg_sparse_decode_workspace_bytes(const lg_decode_params* p);

/* A decode workspace must be zero-filled once before its first use (this call, or any memset);
 * every lg_sparse_decode call leaves it ready for the next one, so a serving loop pays no
 * clearing per token.  (The first bytes hold the status word and one arrival counter per
 * (sequence, kv head, head group); the CTA that completes a unit resets its counter.)  Call it
 * again after a launch that failed.                                                       */
lg_status lg_sparse_decode_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* One query token per sequence attends to every valid slot of its cache:
 * q [B,Hq,D], o [B,Hq,D] bf16; n_tokens (device int64 [B]) counts the tokens appended so
 * far, the current one included; slots holding no token yet are ignored; n_tokens == 0
 * gives o = 0, lse = -inf.  lse [B,Hq] fp32 is optional (NULL to skip).                 */
lg_status lg_sparse_decode(const lg_decode_params* p, const void* q, const void* k_cache,
                           const void* v_cache, const int64_t* n_tokens, void* o, float* lse,
                           void* workspace /* initialised, see above */, size_t workspace_bytes, void* stream);

/* ---- a chunk of new tokens served against the cache (Section 3.2: in serving, the sparse
 *      layers keep only the sink and the most recent window of K,V) ---------------------- */

/*
 * T new tokens of every sequence attend to what the sink + window ring holds and, causally,
 * to themselves: the token at position i sees the sink tokens and the positions j with
 * 0 <= i - j < window_tokens.  That is what T single-token steps (append, then lg_sparse_decode)
 * would have seen; the chunk is NOT appended by this call (use lg_kv_ring_append afterwards).
 * It is the step that prefills a long prompt chunk by chunk with a cache of fixed size.
 *
 * q_chunk, o [B,Hq,T,D]; k_chunk, v_chunk [B,Hkv,T,D]; caches as above (may be NULL when
 * n_tokens_before == 0); all bf16, contiguous, device.  lse [B,Hq,T] fp32 (device).
 * n_tokens_before (HOST value, the same for every sequence) = tokens appended so far.
 * Limits: sink_tokens and window_tokens are multiples of 64 (window_tokens >= 64), otherwise
 * LG_ERR_UNSUPPORTED; T >= 1 and n_tokens_before >= 0 are free.  The call copies the ring's tokens in
 * time order, followed by the chunk, into the workspace and runs the sparse forward kernel
 * with the token-exact window over them, for the chunk's rows only.  workspace: device,
 * 256-byte aligned, lg_chunk_prefill_workspace_bytes() bytes (0 = invalid arguments);
 * lg_last_status(workspace, stream) reports a device-side timeout as for the forward.
 */
size_t lg_chunk_prefill_workspace_bytes(const lg_decode_params* p, int32_t T, int64_t n_tokens_before);
lg_status lg_chunk_prefill(const lg_decode_params* p, const void* q_chunk, const void* k_chunk,
                           const void* v_chunk, const void* k_cache, const void* v_cache, int32_t T,
                           int64_t n_tokens_before, void* o, float* lse, void* workspace,
                           size_t workspace_bytes, void* stream);

/* ---- decode for callers that may not allocate -------------------------------------- */

/* Size of the scratch array that lg_sparse_decode_static uses instead of a workspace.  It
 * is part of the library image: every GPU on which the library is used keeps this much
 * device memory from the first use until the process exits.                              */
#define LG_DECODE_STATIC_SCRATCH_BYTES (4u << 20)

/*
 * lg_sparse_decode without a workspace argument.  (The paper has no counterpart; this is a
 * convenience of this library.)
 *
 * Who needs it: code that runs where device memory cannot be requested at call time -- a
 * serving loop whose memory pool is handed out entirely at start-up, a plug-in that has no
 * allocator handle of its host framework, a latency-critical step where cudaMalloc's implicit
 * synchronisation is not acceptable.  Such a caller still owns q, the caches, n_tokens, o and
 * lse and passes them exactly as to lg_sparse_decode; only the split-KV partials, which
 * lg_sparse_decode keeps in the caller's workspace, go to a fixed array inside the library.
 * The call itself requests no device or host memory (no cudaMalloc / cudaFree, no allocating
 * library routine).
 *
 * Limits and rules
 *   - The problem must satisfy lg_sparse_decode_workspace_bytes(p) <=
 *     LG_DECODE_STATIC_SCRATCH_BYTES (the Llama-2-70B-shaped decode of 16 sequences over a
 *     128 + 4096 token ring needs about 2.7 MB); otherwise LG_ERR_WORKSPACE is returned and
 *     nothing is launched.  Larger problems use lg_sparse_decode with their own workspace.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and remembers it; make that first call outside any stream capture.
 *   - All calls on one device share the one array, and it keeps whatever the previous call
 *     left in it.  The array starts zero-filled (it is a static object), every call resets the
 *     arrival counters it used and overwrites every partial it later reads, so back-to-back
 *     calls on one stream are fine; two calls that can run
 *     on the GPU at the same time (different streams, no dependency) race on the array and
 *     give undefined results.
 *   - The decode kernels contain no device-side waits, so there is no device status to read
 *     back for this call (lg_last_status needs a workspace pointer and does not apply).
 *   - If a launch on the array ends abnormally (a CUDA error reported for the stream, the
 *     process interrupted in mid-kernel and the context kept), arrival counters in the array may
 *     be left non-zero, and later calls would then merge too early or never.  The workspace
 *     variant is repaired by lg_sparse_decode_workspace_init; this array by
 *     lg_sparse_decode_static_reset(stream), which clears it with one memset on `stream`
 *     (no allocation either) and may be called at any time no static call is in flight.
 * Results are bit-identical to lg_sparse_decode on the same inputs.
 */
lg_status lg_sparse_decode_static(const lg_decode_params* p, const void* q, const void* k_cache,
                                  const void* v_cache, const int64_t* n_tokens, void* o, float* lse,
                                  void* stream);
lg_status lg_sparse_decode_static_reset(void* stream);

/* ---- self-test of the error path -------------------------------------------------------- */

/* (The paper has no counterpart; this exists so that the error path can be exercised without
 * breaking anything.)  Every device-side wait of the kernels has a time limit; when one expires,
 * the waiting thread writes its site into the status word at the start of the workspace, all
 * roles leave their loops, and lg_last_status() reports LG_ERR_DEVICE_TIMEOUT.  This call runs a
 * one-warp kernel whose only wait can never be satisfied and whose limit is about a millisecond:
 * afterwards lg_last_status(workspace, stream) must return LG_ERR_DEVICE_TIMEOUT once (and LG_OK
 * on the next call), and the CUDA context is as usable as before.  workspace: device, 256-byte
 * aligned, at least 256 bytes.                                                              */
lg_status lg_selftest_wait_timeout(void* workspace, void* stream);

/* ---- status ------------------------------------------------------------------------- */

/* Synchronises `stream`, reads the status words the kernels keep at the start of
 * `workspace` (attention or decode workspace) and clears them.  LG_OK;
 * LG_ERR_DEVICE_TIMEOUT if a bounded wait expired in a kernel that used the workspace since
 * the last call of this function (a later call on the same workspace does not hide it);
 * LG_ERR_WORKSPACE if a call with lists_prepared = 1 found lists of another pattern.       */
lg_status lg_last_status(void* workspace, void* stream);

const char* lg_status_string(lg_status s);

/* Diagnostic (the paper has no counterpart): the number of CUDA kernels this library has launched
 * in the calling process so far, over all entry points and devices.  A benchmark takes the
 * difference around its timed region.  The counter is the one piece of process-wide state the
 * library keeps besides the fixed array of lg_sparse_decode_static; nothing depends on it.   */
int64_t lg_debug_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* LG_H_ */
