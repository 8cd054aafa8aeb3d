/*
 * videoscan.h -- C ABI of the B200 (sm_100a) streaming attention path of VideoScan
 * (arXiv 2503.09387): one semantic-carrier token per frame, a bounded bank of carrier
 * K/V, visual tokens discarded after their own prefill.
 *
 * Conventions
 *  - Every call returns an int status: VS_OK (0) or a negative VS_ERR_* code.  Nothing
 *    throws, aborts or sets errno.  vs_status_string() names a code.
 *  - Pointers marked DEVICE are CUDA device pointers on `vs_config.device`; pointers
 *    marked HOST are ordinary host memory.  All tensors are bf16 (2 bytes, upper half of
 *    an IEEE fp32) unless stated otherwise, row-major, densely packed.
 *  - The library borrows memory, it owns none on the device: weights, the workspace,
 *    inputs and outputs are allocated and freed by the caller, and weights and workspace
 *    must outlive the handle.  No call allocates device memory.
 *  - vs_frame_prefill / vs_decode_step only enqueue work on `cuda_stream` (a
 *    cudaStream_t passed as void*; NULL is the default stream) and return without
 *    synchronising.  vs_bank_state synchronises that stream.  All calls on one handle
 *    must use the same CUDA stream (or be ordered by the caller).
 *  - A handle is not thread safe.  Distinct handles share no state.
 *  - Device-side waits are bounded; if one ever expires the kernel records
 *    VS_ERR_DEVICE_TIMEOUT in a device status word that vs_bank_state reports.
 *    A handle that has reported it holds unspecified state: destroy it.
 *  - The projection of a step whose K split spans several thread blocks lets those
 *    blocks wait for one another, which needs all of them on the GPU at once: a
 *    handle expects the whole GPU while a step runs.  In particular the steps of two
 *    handles on one GPU must not overlap (same stream, or ordered by events): two such
 *    projections holding half the SMs each would wait for blocks that cannot start,
 *    and both would end with VS_ERR_DEVICE_TIMEOUT.
 */
#ifndef VIDEOSCAN_H_
#define VIDEOSCAN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VS_OK                   0
#define VS_ERR_INVALID_ARG     -1   /* NULL pointer, bad size, bad stream id, duplicate id   */
#define VS_ERR_STATE           -2   /* call not legal in the stream's current phase         */
#define VS_ERR_CAPACITY        -3   /* prefix / text tail / workspace too small             */
#define VS_ERR_CUDA            -4   /* a CUDA runtime or driver call failed                 */
#define VS_ERR_DEVICE_TIMEOUT  -5   /* a bounded device-side wait expired                   */
#define VS_ERR_UNSUPPORTED     -6   /* shape outside what the kernels are built for         */
#define VS_ERR_BOUNDS          -7   /* checked build (-DVS_DEBUG_BOUNDS) only: a kernel tried to store outside the buffer
                                       it was writing, or the guard words behind a workspace region were overwritten */

#define VS_MAX_BATCH           64   /* most streams one call may list                       */
#define VS_N_KERNEL_CLASSES    10   /* kernel classes reported by vs_profile_read           */
#define VS_STATIC_MAX_BANK   4096   /* most carriers vs_evict_choose_static can score       */

typedef struct vs_stream vs_stream;   /* opaque handle: a batch of n_streams independent video streams */

/* Model shape and stream limits.  Multi-head attention with grouped KV heads and rotary
 * position embedding is the Qwen2 backbone the paper builds on (Section 4.1); Eq. (1) is
 * applied per head with d_k = head_dim. */
typedef struct {
  int32_t n_layers;              /* attention layers chained through a residual stream (>= 1)      */
  int32_t d_model;               /* hidden size d; multiple of 64                                    */
  int32_t n_q_heads;             /* query heads Hq                                                   */
  int32_t n_kv_heads;            /* KV heads Hkv; Hq % Hkv == 0, Hq / Hkv <= 8                       */
  int32_t head_dim;              /* D: 64 or 128                                                     */
  int32_t max_tokens_per_frame;  /* largest N one frame may bring (N + 1 <= 256)                     */
  int32_t max_prefix;            /* prompt-prefix capacity in tokens                                 */
  int32_t max_text;              /* question + answer tail capacity in tokens, per turn              */
  int32_t max_step_tokens;       /* largest T of one vs_decode_step call (per stream)                */
  int32_t bank_capacity;         /* M of Section 3.3 (memory mechanism); 0 = keep no carriers        */
  int32_t n_streams;             /* independent streams held by the handle (1 .. VS_MAX_BATCH)       */
  int32_t agg_mode;              /* 0: carrier = mean of the frame's tokens (Section 3.3);
                                    1: carrier = last visual token (ablation "w/o emb", Table 4)     */
  int32_t evict_policy;          /* 0: discard the stored carrier most cosine-similar to the incoming
                                       one; 1: discard the older member of the most similar adjacent
                                       pair (both readings of Section 3.3); 2: FIFO (test aid)       */
  int32_t use_rmsnorm;           /* 1: QKV = RMSNorm(h) W (pre-attention norm); 0: QKV = h W         */
  int32_t residual;              /* 1: h <- h + O between layers (needs Hq*D == d_model); required
                                       when n_layers > 1                                             */
  float   rope_theta;            /* rotary base (Qwen2: 1e6)                                         */
  float   rms_eps;               /* RMSNorm epsilon                                                  */
  int32_t device;                /* CUDA device ordinal                                              */
  int32_t evict_log_capacity;    /* eviction-log entries kept per stream (most recent); may be 0     */
  int32_t out_dtype;             /* element type of `out`: 0 = bf16, 1 = fp32.  Attention outputs reach
                                    |y| > 4 on LLaVA-Video-shaped inputs, where bf16 storage alone
                                    rounds by up to 1.6e-2; fp32 keeps the fp32-accumulated value    */
  int32_t max_chunk_frames;      /* most frames one vs_frame_prefill_chunk call may bring (0 or 1:
                                    that call is not used); sizes the per-step scratch              */
  int32_t d_ff;                  /* 0: attention sub-block only.  > 0: width of the SwiGLU MLP of the full
                                    decoder block (Section 4.1: the backbone is a Qwen2 decoder); a multiple
                                    of 64; needs residual = 1, d_model a multiple of 128 and the four block
                                    weight arrays of vs_weights                                         */
  int32_t vocab;                 /* 0: no language-model head.  > 0: rows of the vocabulary projection used by
                                    vs_lm_head; a multiple of 128; needs vs_weights.w_lm                */
} vs_config;

/* DEVICE pointers to bf16 weights, one entry per layer.  The arrays of pointers themselves
 * are HOST arrays of length n_layers and are copied at create. */
typedef struct {
  const void* const* w_qkv;      /* [n_layers] each [E_out, d_model] row-major ("out x in"),
                                    E_out = (Hq + 2*Hkv) * D, rows ordered Q heads, K heads, V heads;
                                    16-byte aligned                                                  */
  const void* const* b_qkv;      /* [n_layers] each [E_out], or NULL (whole array or any entry)      */
  const void* const* norm_w;     /* [n_layers] each [d_model] RMSNorm gain, or NULL = all ones       */
  /* the rest of the decoder block, read only when d_ff > 0 (all "out x in", row-major, 16-byte aligned):
   *   h1 = h + A W_o^T (A: the layer's attention rows),  h2 = h1 + (SiLU(n W_gate^T) * (n W_up^T)) W_down^T,
   *   n = RMSNorm(h1) when use_rmsnorm.  A step's `out` then receives the last layer's h2 ([..][d_model]). */
  const void* const* w_o;        /* [n_layers] each [d_model, Hq*D]                                  */
  const void* const* w_gate;     /* [n_layers] each [d_ff, d_model]                                  */
  const void* const* w_up;       /* [n_layers] each [d_ff, d_model]                                  */
  const void* const* w_down;     /* [n_layers] each [d_model, d_ff]                                  */
  const void* const* norm2_w;    /* [n_layers] each [d_model] gain of the post-attention RMSNorm, or NULL */
  /* the language-model head, read only when vocab > 0 (single DEVICE pointers, not per layer): */
  const void* w_lm;              /* [vocab, d_model] row-major, 16-byte aligned                      */
  const void* norm_f_w;          /* [d_model] gain of the final RMSNorm, or NULL = all ones          */
} vs_weights;

/* Filled by vs_bank_state (HOST). */
typedef struct {
  int32_t count;                 /* carriers in the bank == min(frames_seen, capacity)               */
  int32_t capacity;
  int64_t frames_seen;
  int64_t evictions;
  int64_t next_pos;              /* position id the next frame (or prefix token) starts at           */
  int64_t prefix_len;
  int64_t text_len;
  int32_t last_victim_frame;     /* frame id discarded by the last frame step, -1 if none            */
  int32_t device_status;         /* 0, or VS_ERR_DEVICE_TIMEOUT (or VS_ERR_BOUNDS in a checked build)  */
  uint64_t persistent_bytes;     /* bytes of the workspace that hold stream state; constant          */
  uint64_t workspace_bytes;      /* whole workspace; constant for the life of the handle             */
} vs_bank_info;

/* Bytes of DEVICE workspace vs_create_stream needs for `cfg` (256-byte aligned base). */
int vs_workspace_bytes(const vs_config* cfg, size_t* out_bytes);

/* Builds a handle over caller memory: carves `workspace` (DEVICE, >= vs_workspace_bytes,
 * 256-byte aligned) into bank, prefix, tail, metadata and per-step scratch, clears the
 * metadata (synchronously) and encodes the TMA descriptors of the weights.  Nothing is
 * allocated on the device, so memory use does not depend on stream length (the constant
 * memory footprint that Section 3.3 claims for the method holds by construction). */
int vs_create_stream(const vs_config* cfg, const vs_weights* weights,
                     void* workspace, size_t workspace_bytes, vs_stream** out);

/* One frame per listed stream -- the prefilling phase of Section 3.3:
 *   carrier C = (1/N) sum_i E_i appended after the N visual tokens (Sections 3.2, 3.3);
 *   per layer: Q,K,V projection, RoPE, softmax attention (Eq. 1) of the N+1 tokens over
 *   [prompt prefix | carriers in the bank | own frame, causal];
 *   then the carrier's K/V of every layer enters the bank (evicting first when the bank is
 *   full) and everything else of the frame is dropped.
 * stream_ids: HOST [n_active], distinct ids in [0, n_streams).
 * hidden:     DEVICE bf16 [n_active][N][d_model].
 * carrier_override: DEVICE bf16 [n_active][d_model] used as the carrier token instead of
 *             the mean (e.g. projector(mean) computed by the caller), or NULL.
 * out:        DEVICE [n_active][N+1][Hq*D] of `out_dtype`, last layer's attention output, row N
 *             being the carrier's; may be NULL.  On a handle with d_ff > 0: the hidden state that
 *             leaves the last decoder block (Hq*D == d_model there), a bf16 storage point widened
 *             to `out_dtype`.
 * Errors: VS_ERR_STATE if a listed stream has an open text turn (call vs_end_turn first);
 *         VS_ERR_CAPACITY if N > max_tokens_per_frame. */
int vs_frame_prefill(vs_stream* h, const int32_t* stream_ids, int32_t n_active,
                     const void* hidden, int32_t N, const void* carrier_override,
                     void* out, void* cuda_stream);

/* F consecutive frames of ONE stream in one call -- the offline form of the prefilling phase
 * (Section 3.3; the paper's offline benchmarks of Section 4 feed whole videos).  The result is
 * that of F vs_frame_prefill calls in a row: each frame attends over [prefix | the bank as the
 * frames before it left it | own frame], evictions included, because the eviction rule looks
 * only at carrier embeddings, which are all known once the frames are pooled.  Per layer the
 * Q/K/V projection of all F*(N+1) rows is one GEMM and the attention of all F frames is one launch
 * (each frame with its own view of the bank).
 * hidden: DEVICE bf16 [F][N][d_model];  out: DEVICE [F][N+1][Hq*D] of `out_dtype`, or NULL.
 * The chunk's bank updates are enqueued on a stream that the handle owns, forked from and joined
 * back into `cuda_stream` by events, so that they run beside the projection; the handle's first
 * call of this function creates that stream and its two events (no device memory).
 * Errors: as vs_frame_prefill; VS_ERR_CAPACITY also if F > max_chunk_frames or if
 *         bank_capacity + 1 + F > 8192. */
int vs_frame_prefill_chunk(vs_stream* h, int32_t stream_id, const void* hidden, int32_t F, int32_t N,
                           void* out, void* cuda_stream);

/* The bank's carriers as ordinary tokens, without their stored K/V (Section 3.4, stage 1: the
 * visual input is the semantic carrier tokens only; Section 4.3, inference without KV reuse):
 * the stored carrier embeddings of ONE stream, in temporal order, one token per frame at
 * positions prefix_len + i, go through the layers, each attending over the prompt prefix and the
 * carriers up to itself.  Reads the bank, changes nothing.
 * out: DEVICE [count][Hq*D] of `out_dtype` (count = carriers in the bank; vs_bank_state tells).
 * count = 0 is not an error: nothing is launched. */
int vs_bank_forward(vs_stream* h, int32_t stream_id, void* out, void* cuda_stream);

/* T text tokens per listed stream -- the decoding phase of Section 3.3 (T = 1) and the
 * text part of prefilling (T > 1).  Token i attends to [prefix | bank | tail tokens up to
 * itself]; no visual-token K/V exists any more.  Before a stream's first frame the tokens
 * extend the prompt prefix instead (the system instruction comes first, Section 3.3) and
 * stay for the life of the stream.
 * hidden: DEVICE bf16 [n_active][T][d_model];  out: DEVICE [n_active][T][Hq*D] of `out_dtype`.
 * All listed streams must be in the same phase (all before or all after their first frame).
 * Errors: VS_ERR_CAPACITY on prefix / tail overflow or T > max_step_tokens. */
int vs_decode_step(vs_stream* h, const int32_t* stream_ids, int32_t n_active,
                   const void* hidden, int32_t T, void* out, void* cuda_stream);

/* Language-model head -- what turns the hidden state of a last position into the next answer token in
 * the decoding phase of Section 3.3.  The paper prints no formula for it; it is the head of the Qwen2
 * backbone named in Section 4.1:  logits = (RMSNorm(hidden) * norm_f_w) W_lm^T  (no norm when
 * use_rmsnorm = 0),  next_token = the index of the largest logit, the lowest index among equals, a NaN
 * ranking below every number.
 * hidden: DEVICE [rows][d_model] of `out_dtype` (so the rows a step wrote to `out` can be passed on as
 *         they are); each value is rounded to bf16 on entry -- a hidden state is a stored tensor;
 *         8-byte aligned.  rows: 1 .. 256, and no more than the handle's largest step.
 * logits: DEVICE fp32 [rows][vocab], 16-byte aligned, the caller's; always written.
 * next_token: DEVICE int32 [rows], or NULL.
 * Uses the step scratch of the handle: enqueue it on the handle's stream like any other step.
 * Errors: VS_ERR_UNSUPPORTED on a handle created with vocab = 0; VS_ERR_CAPACITY for too many rows. */
int vs_lm_head(vs_stream* h, const void* hidden, int32_t rows, void* logits, int32_t* next_token,
               void* cuda_stream);

/* Ends a question/answer turn: the text tail is dropped, prefix and bank stay, frame
 * positions do not move.  Host-only bookkeeping. */
int vs_end_turn(vs_stream* h, const int32_t* stream_ids, int32_t n_active);

/* Starts the listed streams over (a new video): empty bank, no prefix, positions from 0.
 * Asynchronous on cuda_stream; the memory mechanism of Section 3.3 simply begins again. */
int vs_reset_stream(vs_stream* h, const int32_t* stream_ids, int32_t n_active, void* cuda_stream);

/* Synchronises the handle's CUDA stream and reports one stream's bank (Section 3.3,
 * memory mechanism) in temporal order (oldest carrier first).  All outputs are HOST and
 * optional (NULL skips them):
 *   frame_ids, positions, slots : [capacity] -- first `count` entries valid; `slots` are the
 *                                 physical slot numbers (implementation defined);
 *   evict_log : [evict_log_cap][2] int32 (frame step, victim frame id), oldest kept first;
 *               *evict_log_n receives the number written;
 *   emb_out   : bf16 [count][d_model] carrier embeddings;
 *   k_out, v_out : bf16 [count][Hkv][D] of `layer`. */
int vs_bank_state(vs_stream* h, int32_t stream_id, vs_bank_info* info,
                  int32_t* frame_ids, int64_t* positions, int32_t* slots,
                  int32_t* evict_log, int32_t evict_log_cap, int32_t* evict_log_n,
                  void* emb_out, int32_t layer, void* k_out, void* v_out);

/* Test aids.  vs_last_step_kv copies the rotated K and V rows that the most recent
 * vs_frame_prefill / vs_decode_step left in scratch for the LAST layer to HOST buffers
 * bf16 [rows][Hkv*D] (rows = n_active*(N+1) or n_active*T), synchronising first; it lets a
 * test check that the bank append is a pure copy.  vs_poison_scratch overwrites every
 * per-step scratch region with NaN patterns (asynchronously on cuda_stream): later steps
 * must not change, which shows that no visual-token state survives a step. */
int vs_last_step_kv(vs_stream* h, void* k_out, void* v_out, int32_t rows);
int vs_poison_scratch(vs_stream* h, void* cuda_stream);

/* Launch accounting (no counterpart in the paper; measurement aid).  Every kernel launch is
 * counted per class.  With profiling enabled each launch is also bracketed by a pair of CUDA
 * events on the launching stream, at most `max_launches` pairs between two reads (host-side
 * event objects are created on enable; no device memory).  vs_profile_read synchronises and
 * returns, per class and since the previous read: summed device milliseconds of the timed
 * launches (HOST double[VS_N_KERNEL_CLASSES]), how many were timed, and how many were
 * launched (HOST int64[VS_N_KERNEL_CLASSES] each); any pointer may be NULL. */
int vs_profile_enable(vs_stream* h, int32_t on, int32_t max_launches);
int vs_profile_read(vs_stream* h, double* ms, int64_t* timed, int64_t* launches);
const char* vs_kernel_class_name(int32_t k);

/* Eviction decision without any allocation (the paper has no counterpart; it is the rule of
 * Section 3.3's memory mechanism offered as a stand-alone call).  It is meant for callers
 * that hold no workspace and may not call cudaMalloc: a real-time frame loop, where an
 * allocation would stall the device; a component that was handed a fixed memory budget up
 * front; a plug-in that must not go around its host framework's allocator.  Such a caller
 * can still ask which stored carrier the bank would discard for an incoming one.
 *   bank_emb  : DEVICE bf16 [count][d_model], carriers in temporal order (oldest first);
 *   incoming  : DEVICE bf16 [d_model];
 *   policy    : as vs_config.evict_policy (0 similarity to the incoming carrier, 1 most
 *               similar adjacent pair, 2 FIFO);
 *   victim_out: DEVICE int32[1], receives the temporal index to discard (ties: oldest; a carrier
 *               holding Inf or NaN has no cosine, its score counts as 0; always < count).
 * The call only enqueues work on cuda_stream.  Its scratch (count fp64 scores and one block
 * counter) lives in a static device array of the library, VS_STATIC_MAX_BANK * 8 + 256
 * bytes, which every GPU that loads the library holds until the process exits; count above
 * VS_STATIC_MAX_BANK returns VS_ERR_CAPACITY.  The first call on a device looks the array's
 * device address up (cudaGetSymbolAddress, with that device current) and should therefore
 * come before any stream capture.  All calls on a device share the array: it keeps the last
 * call's scores, the counter is cleared at the start of every call, and two calls that
 * overlap on the GPU (different streams) race -- order them.  Calls no cudaMalloc, cudaFree
 * or other allocating routine. */
int vs_evict_choose_static(const void* bank_emb, const void* incoming, int32_t count, int32_t d_model,
                           int32_t policy, int32_t* victim_out, void* cuda_stream);

int vs_destroy_stream(vs_stream* h);

const char* vs_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif  /* VIDEOSCAN_H_ */
