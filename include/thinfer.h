/*
 * thinfer.h - C ABI of the B200 (sm_100a) FP16 Llama-style decoder forward.
 *
 * The library runs the two phases of the paper's Prefill-Buffer-Decode pipeline
 * (Section 3.4.2) for one decoder layer or a stack of them on ONE GPU:
 *
 *   prefill  dense projections on tcgen05 tensor cores + causal attention
 *            (Eq. 6, the staged attention of Section 3.3.2)
 *   decode   one token per request: weight-streaming GEMV / skinny GEMM
 *            (the small-M path of Section 3.2.2) + attention over the FP16
 *            KV cache, with the density-driven fusion units of Section 3.3.1:
 *            RMSNorm -> QKV -> RoPE + cache append (Algorithm 1), attention,
 *            O-projection + residual, RMSNorm -> gate/up -> SwiGLU,
 *            down-projection + residual.
 *
 * Conventions
 *   - Plain C.  No exception or abort crosses the boundary.  Every call
 *     returns 0 (THINFER_OK) or a negative thinfer_err; thinfer_last_error()
 *     gives a text for the most recent failure of a context.
 *   - "device" pointers are CUDA device memory of the current device, owned by
 *     the caller, 256-byte aligned unless stated otherwise.  "host" pointers
 *     are ordinary host memory.  The library allocates no device memory except
 *     one pinned, host-mapped status word per context.
 *   - Arguments are validated on the host before anything is enqueued.
 *     Compute is enqueued on `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream) and the call returns without
 *     synchronising.  Calls on one context must be issued from one thread at
 *     a time; work of one context must stay ordered on the device (use one
 *     stream, or order the streams with events).
 *   - Storage is a 16-bit floating-point type, accumulation and the norm /
 *     softmax reductions are FP32 (Section 3.2.4, which describes the operator
 *     variants side by side: same kernels, different element type).  The
 *     library is built once per storage type with the same exports:
 *     libthinfer.so stores IEEE FP16, libthinfer_bf16.so stores BF16
 *     (thinfer_storage_type() tells which one is loaded); wherever this
 *     header says "FP16" the BF16 build reads and writes BF16 instead.  Matrices are row-major [out, in] (the paper's
 *     Y = X W, Section 3.2.1, with W stored transposed so that the contraction
 *     index is contiguous for both operands).
 *   - Device-side waits are bounded: a pipeline that does not make progress
 *     writes THINFER_ETIMEOUT to the status word and the kernel returns.
 */
#ifndef THINFER_H
#define THINFER_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  THINFER_OK = 0,
  THINFER_EINVAL = -1,       /* NULL pointer, bad size, bad slot, wrong mode      */
  THINFER_EUNSUPPORTED = -2, /* shape outside what the kernels cover              */
  THINFER_ECAPACITY = -3,    /* batch > max_batch, or the sequence would exceed max_seq, or a workspace is too small */
  THINFER_EBUSY = -4,        /* prefill into a slot that has not been released (back-pressure, Section 3.4.2) */
  THINFER_ECUDA = -5,        /* a CUDA runtime / driver call failed               */
  THINFER_ETIMEOUT = -6      /* a bounded device-side wait expired                */
} thinfer_err;

typedef struct thinfer_ctx thinfer_ctx; /* opaque host object */

/* Layer shapes (Section 4.1: Llama-2 family).  Supported: head_dim 64 or 128;
 * n_q_heads a multiple of n_kv_heads; hidden, ffn and n_q_heads*head_dim
 * multiples of 8; max_batch <= 64 (decode rows); max_seq >= 1. */
typedef struct {
  int32_t hidden, n_q_heads, n_kv_heads, head_dim, ffn, n_layers;
  int32_t vocab;      /* 0: layer-only mode, hidden states in and out; > 0: token ids in, next ids / logits out */
  float rms_eps;      /* inside the square root */
  float rope_base;    /* angle of pair j at position p = p * rope_base^(-2j/head_dim) */
  int32_t max_batch;  /* requests per slot */
  int32_t max_seq;    /* KV positions per request */
  int32_t buf_slots;  /* Buf_max: number of KV slots in the bounded buffer, >= 1 */
} thinfer_config;

/* Device pointers, FP16, caller-owned, read-only, must outlive the context.
 * Norm gains are [hidden]; wq [n_q_heads*head_dim, hidden]; wk, wv
 * [n_kv_heads*head_dim, hidden]; wo [hidden, n_q_heads*head_dim]; w_gate, w_up
 * [ffn, hidden]; w_down [hidden, ffn]. */
typedef struct {
  const void *attn_norm, *wq, *wk, *wv, *wo;
  const void *ffn_norm, *w_gate, *w_up, *w_down;
} thinfer_layer_weights;

typedef struct {
  const thinfer_layer_weights* layers; /* host array [n_layers] (copied by thinfer_create) */
  const void *embed;                   /* device FP16 [vocab, hidden]; NULL when vocab == 0 */
  const void *final_norm;              /* device FP16 [hidden];        NULL when vocab == 0 */
  const void *lm_head;                 /* device FP16 [vocab, hidden]; NULL when vocab == 0 */
} thinfer_weights;

/* Storage type of the loaded build (Section 3.2.4): 0 = IEEE FP16, 1 = BF16. */
int thinfer_storage_type(void);

/* Sizes of the two caller-allocated device regions.
 * kv_bytes: buf_slots x n_layers x {K,V} x [max_batch][n_kv_heads][max_seq][head_dim] FP16
 * (K is stored after RoPE, Algorithm 1).  scratch_bytes: activations, RoPE
 * table, split-KV partials, staging for the *_host calls.  Host pointers out. */
int thinfer_workspace_bytes(const thinfer_config* cfg, size_t* kv_bytes, size_t* scratch_bytes);

/* Builds a context for one model (Section 4.1: Llama-2 7B / 13B / 70B shapes, FP16 weights shared by all
 * requests of a batch, Section 3.4.1) with buf_slots KV slots of max_batch x max_seq positions, the
 * bounded buffer between the prefill and the decode stage (Section 3.4.2).  cfg, weights: host.
 * kv_workspace, scratch: device, at least the sizes above (else THINFER_ECAPACITY); the context uses them until
 * thinfer_destroy.  Synchronises the device once (table set-up).  *out is set
 * only on success. */
int thinfer_create(const thinfer_config* cfg, const thinfer_weights* weights,
                   void* kv_workspace, size_t kv_bytes, void* scratch, size_t scratch_bytes,
                   thinfer_ctx** out);

/* Prefill (Section 3.4.2: the Prefill pool produces the first token and the
 * initial KV cache).  Processes `batch` prompts of uniform length `seq_len`
 * (Section 4.1: prompts padded to one length; every position is a real token,
 * position = index in the sequence) and fills KV slot `slot` for positions
 * 0..seq_len-1.
 *   vocab == 0: input  device FP16 [batch, seq_len, hidden];
 *               out_primary device FP16 [batch, seq_len, hidden] (layer-stack output); out_logits must be NULL.
 *   vocab  > 0: input  device int32 [batch, seq_len] token ids in [0, vocab);
 *               out_primary device int32 [batch] greedy next ids of the last position (may be NULL);
 *               out_logits  device FP32 [batch, vocab] logits of the last position (may be NULL).
 * Errors: THINFER_EBUSY if the slot holds an unreleased sequence;
 * THINFER_ECAPACITY if batch > max_batch or seq_len > max_seq. */
int thinfer_prefill(thinfer_ctx* ctx, int32_t slot, const void* input, int32_t batch, int32_t seq_len,
                    void* out_primary, void* out_logits, void* cuda_stream);

/* Prefill of prompts of DIFFERENT lengths (Section 3.4.1: attention is per request, each with its own KV
 * cache; the paper pads prompts to one length only for its experiment, Section 4.1).  `input` is laid out as
 * for thinfer_prefill with seq_len = the padded length; seq_lens: host int32 [batch], 1 <= seq_lens[b] <=
 * seq_len.  Rows past a request's length are padding: they are computed but mean nothing, and with vocab == 0
 * the hidden-state output of those rows is unspecified; with vocab > 0 the logits / next ids are those of each
 * request's own last token.  Later decode steps continue every request from its own length: the new token of
 * request b sits at position seq_lens[b] + (decode steps so far).  The slot is full when the LONGEST request
 * reaches max_seq.  Launch mode 2 uses the per-unit kernels for such a slot. */
int thinfer_prefill_ragged(thinfer_ctx* ctx, int32_t slot, const void* input, int32_t batch, int32_t seq_len,
                           const int32_t* seq_lens, void* out_primary, void* out_logits, void* cuda_stream);

/* Host query: positions each request of the slot holds (lens_out: host int32 [batch of the slot]). */
int thinfer_slot_lengths(const thinfer_ctx* ctx, int32_t slot, int32_t* lens_out);

/* Batch sizes.  Decode steps of up to 16 requests run on the weight-streaming skinny projections and are
 * what the library is tuned and measured for (75 - 94 % of the device's copy bandwidth depending on the model);
 * 17 .. 64 requests run on the stream-K tensor-core path, which is correct and tested but measured at 62 - 66 %
 * (a step of 17 requests costs about 30 % more than one of 16).  Split larger batches into slots of 16. */
/* One decode step for every request of `slot` (Section 3.4.1, selective
 * batching: projections batched over requests, attention per request).  The
 * new token sits at position cur_len (the number of positions the slot holds);
 * its key and value are appended and cur_len grows by one.
 *   vocab == 0: input device FP16 [batch, hidden]; out_primary device FP16 [batch, hidden].
 *   vocab  > 0: input device int32 [batch];        out_primary int32 [batch] / out_logits FP32 [batch, vocab].
 * Errors: THINFER_EINVAL if the slot is empty; THINFER_ECAPACITY if cur_len == max_seq. */
int thinfer_decode_step(thinfer_ctx* ctx, int32_t slot, const void* input,
                        void* out_primary, void* out_logits, void* cuda_stream);

/* The same two calls with HOST buffers: the input is copied to a staging area
 * in `scratch`, the step runs, and out_primary (and out_logits if not NULL) is
 * copied back, all enqueued on cuda_stream; the host buffers may be read once
 * the stream has been synchronised.  Pinned host memory makes the copies
 * asynchronous. */
int thinfer_prefill_host(thinfer_ctx* ctx, int32_t slot, const void* host_input, int32_t batch, int32_t seq_len,
                         void* host_out_primary, void* host_out_logits, void* cuda_stream);
int thinfer_decode_step_host(thinfer_ctx* ctx, int32_t slot, const void* host_input,
                             void* host_out_primary, void* host_out_logits, void* cuda_stream);

/* Bounded buffer of Section 3.4.2: marks `slot` free so that a later prefill
 * may reuse it (until then a prefill into the slot returns THINFER_EBUSY: the
 * back-pressure).  Pass the stream on which the slot's decode steps ran: an
 * event recorded there makes a later prefill of the slot - on any stream -
 * wait on the device until those steps have finished.
 *
 * Stage hand-off.  Prefill and decode use separate activation buffers inside
 * `scratch`, and every prefill records an event that the slot's first decode
 * step waits for.  A prefill of one slot and the decode steps of another slot
 * may therefore be enqueued on two different streams and overlap on the GPU
 * (the Prefill -> Buffer -> Decode schedule on one device).  Calls of the same
 * stage (two prefills, or decode steps of two slots) still share buffers: keep
 * each stage on one stream, or order them yourself. */
int thinfer_release_slot(thinfer_ctx* ctx, int32_t slot, void* cuda_stream);

/* Host queries (no device work).  *batch / *cur_len: what the slot holds (0, 0 when free). */
int thinfer_slot_state(const thinfer_ctx* ctx, int32_t slot, int32_t* batch, int32_t* cur_len);

/* Device address of K (which = 0) or V (which = 1) of `layer` in `slot`:
 * FP16 [max_batch][n_kv_heads][max_seq][head_dim].  For inspection by tests. */
int thinfer_kv_pointer(const thinfer_ctx* ctx, int32_t slot, int32_t layer, int32_t which, void** device_ptr);

/* Reads the device status word (0, or a thinfer_err a kernel wrote) without
 * synchronising; meaningful after the caller synchronised the stream.  (The paper's pipeline avoids failure
 * by back-pressure, Section 3.4.2, and describes no error path; this word is how a bounded device-side
 * wait that ran out is reported.) */
int thinfer_status(thinfer_ctx* ctx, int32_t* device_status);

/* The status word is sticky: once a kernel has written a code it stays non-zero until it is cleared (a
 * later failure may replace the code by its own), and a
 * kernel that gave up may have left arrival counters or the grid barrier of launch mode 2 half-way, so
 * later steps of the context are not meaningful until it is cleared.  thinfer_clear_status synchronises the
 * device, puts the counters, the grid barrier and the status word back to their initial state and returns;
 * the KV slots keep their contents and lengths (release and prefill them again to be safe).  Call it with
 * no work of the context in flight. */
int thinfer_clear_status(thinfer_ctx* ctx);

/* Self-test of the bounded device-side wait (no counterpart in the paper).  Enqueues a one-CTA kernel that
 * waits, for at most limit_ns nanoseconds (1 us .. 100 ms), on a barrier nobody arrives on.  The wait gives
 * up, the kernel returns normally and THINFER_ETIMEOUT is left in the status word: after synchronising the
 * stream thinfer_status reports it, thinfer_clear_status clears it, and the context works as before.  This is
 * the same wait, with a shorter limit, that guards every TMA / tensor-core pipeline of the library. */
int thinfer_selftest_bounded_wait(thinfer_ctx* ctx, int64_t limit_ns, void* cuda_stream);

/* Inspection hook for tests (Section 3.4.3's per-layer view: the hidden state between layers never leaves
 * the library otherwise).  After layer layers[i] of every later prefill or decode step - layers[i] = -1
 * means the input of layer 0, i.e. the embedding rows when vocab > 0 - the hidden state is copied, on the
 * call's stream, to device_bufs[i]: device FP16 [batch x seq_len, hidden] (prefill) or [batch, hidden]
 * (decode), caller-owned and large enough.  n = 0 removes all captures.  layers, device_bufs: host arrays
 * [n], copied.  In launch mode 2 a decode step of up to 16 requests runs all layers in one kernel: only
 * the last layer's state (and -1) can be captured there, other layers give THINFER_EUNSUPPORTED. */
int thinfer_capture_hidden(thinfer_ctx* ctx, int32_t n, const int32_t* layers, void* const* device_bufs);

/* Unified launch (Section 3.3.3: one creation + launch for the whole operator
 * graph instead of one per operator).  mode 0: one plain launch per fusion
 * unit; 1: the same launches chained with programmatic dependent launch (each
 * kernel starts early and waits on the device); 2: a decode step of up to 16
 * requests runs every unit of every layer in ONE cooperative, persistent
 * kernel with grid-wide barriers between units (larger batches and prefill
 * fall back to mode 1). */
int thinfer_set_launch_mode(thinfer_ctx* ctx, int32_t mode);

/* Per-kernel timing for roofline reports.  When `kernel_id` >= 0 every launch
 * of that kernel (thinfer_kernel_id) is bracketed by CUDA events on its own
 * stream; thinfer_profile_read synchronises those events and returns the count
 * and the summed duration since the last read.  -1 switches it off.
 * (THINFER_K_ATTN_COMBINE is kept for numbering only: the split-KV merge runs
 * inside the decode attention kernel and has no launches of its own.) */
typedef enum {
  THINFER_K_RMSNORM = 0, THINFER_K_QKV = 1, THINFER_K_ATTN = 2, THINFER_K_ATTN_COMBINE = 3,
  THINFER_K_OPROJ = 4, THINFER_K_GATEUP = 5, THINFER_K_DOWN = 6, THINFER_K_HEAD = 7,
  THINFER_K_EMBED = 8, THINFER_K_ARGMAX = 9, THINFER_K_DECODE_UNIFIED = 10, THINFER_K_COUNT = 11
} thinfer_kernel_id;
int thinfer_profile_select(thinfer_ctx* ctx, int32_t kernel_id);
int thinfer_profile_read(thinfer_ctx* ctx, int32_t* launches, float* total_ms);

/* Trace of the unified decode kernel (launch mode 2).  enable != 0: CTA 0 of every later unified
 * launch stores the nanosecond device timer at each unit boundary into a scratch area.  If host_out is
 * not NULL, the area is copied to it first (synchronous copy; call after synchronising the stream):
 * entry 0 = kernel end, 1 = start, 2 = prep done, 3 = after the first grid barrier, then per layer
 * QKV done, barrier, attention done, barrier, O done, barrier, gate/up done, barrier, down done
 * (, barrier).  While tracing is on, the stream-K projections of the per-unit decode path also store, per
 * thinfer_kernel_id k, in entries 16k+10 .. 16k+15: earliest CTA start, earliest pass of the dependency wait,
 * latest load issued, latest MMA issued, latest accumulator ready, latest epilogue end.  max_entries <= 4352: entries
 * from 256 on hold, for the kernel id named by the environment variable THINFER_TRACE_CTA_KID at thinfer_create, four
 * values per CTA of its last launch (SM id, time past the dependency wait, last warp's stream end, end).
 * Host pointer; tracing aid, not part of the hot path. */
int thinfer_trace_unified(thinfer_ctx* ctx, int32_t enable, uint64_t* host_out, int32_t max_entries);

/* Number of kernels this context has launched so far (host counter). */
int64_t thinfer_launch_count(const thinfer_ctx* ctx);

const char* thinfer_last_error(const thinfer_ctx* ctx);

/* Ends a context (the paper has no counterpart: its pools live for the whole run, Section 3.4.2).  Frees the
 * host object, its events and the status word; the caller's weights, KV workspace and scratch are untouched
 * and may be freed afterwards.  No work of the context may be in flight.  NULL is allowed. */
void thinfer_destroy(thinfer_ctx* ctx);

/* ------------------------------------------------------------------------ *
 * Single operators (the paper's operator layer, Section 3.2), exposed for
 * parity tests and micro-benchmarks at the shapes of Tables 8 and 9.  All
 * pointers are device pointers; work is enqueued on cuda_stream.
 * ------------------------------------------------------------------------ */

/* y[rows, n_out] = x[rows, k] * w[n_out, k]^T  (Section 3.2.1).  FP16 in,
 * FP16 out (out_fp32 == 0) or FP32 out.  path 0: tcgen05 tensor-core tiles
 * (any rows); path 1: the weight-streaming FMA GEMV (rows <= 16); path 2: the
 * weight-streaming skinny GEMM on warp-level tensor-core fragments (rows <= 16),
 * the kernel the decode projections of up to 16 requests use.  k % 8 == 0,
 * n_out even. */
int thinfer_op_linear(const void* x, const void* w, void* y, int32_t rows, int32_t n_out, int32_t k,
                      int32_t out_fp32, int32_t path, void* cuda_stream);

/* The same product for callers that must not allocate (the paper has no
 * counterpart: this entry point exists for the integration, not the method).
 * Some hosts of this library cannot call cudaMalloc at the point where they
 * need a projection: code running while a CUDA graph is being captured on
 * another stream of the process, real-time loops that forbid calls which may
 * synchronise the device, and allocators that hand a fixed arena to each
 * plug-in.  For them the split-K partial sums and arrival counters of the
 * stream-K kernel live in a fixed array inside the library image instead of a
 * caller workspace; nothing is allocated or freed, by this call or by anything
 * it uses.
 *   Limits: rows <= 16, n_out <= 16384, k % 8 == 0, n_out even.  Larger sizes
 *   return THINFER_ECAPACITY (text in thinfer_last_error(NULL)).  The array is
 *   about 2.3 MB and stays resident on every GPU that loads the library until
 *   the process exits.
 *   The first call on a device resolves the array's device address (with that
 *   device current) and should therefore come before any stream capture; later
 *   calls only enqueue a 1 KB clear of the counters and the kernel.
 *   All calls on a device share the array: calls whose kernels may overlap on
 *   the GPU (different streams without ordering) race on it.  Keep them on one
 *   stream or order them with events.
 * x, w, y: device pointers as for thinfer_op_linear (tensor-core path). */
int thinfer_op_linear_noalloc(const void* x, const void* w, void* y, int32_t rows, int32_t n_out, int32_t k,
                              int32_t out_fp32, void* cuda_stream);

/* Causal attention of Eq. 6 for a batch: q FP16 [batch, n_q_heads, seq, head_dim],
 * k, v FP16 [batch, n_kv_heads, kv_stride, head_dim] (first seq positions used),
 * out FP16 [batch, seq, n_q_heads*head_dim]. */
int thinfer_op_attention_prefill(const void* q, const void* k, const void* v, void* out,
                                 int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t seq,
                                 int32_t kv_stride, int32_t head_dim, void* cuda_stream);

/* Decode attention alone (Eq. 6 for one query row per request and head, Section 3.4.1: per request, over its own
 * cache), for parity tests of the split-KV schedules: q device FP16 [batch, n_q_heads, head_dim] (already rotated)
 * attends the first t_len positions of every request in the K/V cache of (`slot`, `layer`) of `ctx` - written
 * beforehand by a prefill, or directly through thinfer_kv_pointer - and out device FP16 [batch, n_q_heads*head_dim]
 * receives the result.  seq_lens (host int32 [batch], may be NULL): request b attends seq_lens[b] keys instead
 * (the slot's per-request length array on the device is overwritten: use a slot that holds no ragged sequence).
 * Uses the context's split-KV scratch: order it with the context's other work. */
int thinfer_op_attention_decode(thinfer_ctx* ctx, int32_t slot, int32_t layer, const void* q, void* out, int32_t batch,
                                int32_t t_len, const int32_t* seq_lens, void* cuda_stream);

/* Greedy pick of the stack's last step (the paper is silent on sampling): ids[r] = the lowest index at
 * which logits[r, :] is largest.  logits device FP32 [rows, n]; ids device int32 [rows]. */
int thinfer_op_argmax(const void* logits, void* ids, int32_t rows, int32_t n, void* cuda_stream);

/* y = x * gain / sqrt(mean(x^2) + eps), rows of length n (Section 3.2.4). */
int thinfer_op_rmsnorm(const void* x, const void* gain, void* y, int32_t rows, int32_t n, float eps,
                       void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* THINFER_H */
