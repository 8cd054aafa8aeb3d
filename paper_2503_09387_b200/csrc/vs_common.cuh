// Shared declarations of the CUDA path: workspace carve-up, per-call batch parameters,
// launch wrappers.  Nothing here is shared with the CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>

#include "../../include/videoscan.h"

namespace vs {

typedef __nv_bfloat16 bf16;

// ---- device-resident metadata of one stream (Section 3.3, memory mechanism) ------------
// `slots` = bank_capacity + 1 physical slots, so the incoming carrier can be written while
// the victim is still readable.
struct StreamMeta {
  int32_t count;              // carriers currently in the bank
  int32_t free_slot;          // physical slot the next carrier is written to
  int32_t victim_logical;     // temporal index chosen by the scoring kernel, -1 = none
  int32_t last_victim_frame;  // frame id discarded by the last step, -1 = none
  int64_t frames_seen;
  int64_t evictions;
  int32_t log_count;          // evictions ever logged (ring position = log_count % cap)
  int32_t score_ticket;       // blocks of the scoring kernel that have finished
  int32_t pad[4];
};

// ---- per-call description of the listed streams (passed by value to kernels) -----------
struct BatchParams {
  int32_t n_active;
  int32_t rows_per_stream;             // N + 1 for a frame step, T for a text step
  int32_t stream_id[VS_MAX_BATCH];
  int32_t count[VS_MAX_BATCH];         // carriers in the bank before this step (host mirror)
  int32_t prefix_len[VS_MAX_BATCH];
  int32_t text_len[VS_MAX_BATCH];      // tail length before this step
  int64_t pos_base[VS_MAX_BATCH];      // position id of the step's first token
  int64_t frame_id[VS_MAX_BATCH];      // frames_seen before this step
#ifdef VS_TRACE
  unsigned long long* trace;           // timeline log of a -DVS_TRACE build, or null
  unsigned trace_seq;                  // sequence number of the launch
#endif
#ifdef VS_DEBUG_BOUNDS
  struct DebugTable* dbg;              // workspace regions of a checked build
#endif
};

// ---- checked stores (only in a -DVS_DEBUG_BOUNDS build; the product build compiles none of it) ----
// Stand-in for a memory checker: every store of a kernel into the workspace names the region it
// means to write; a store outside that region is skipped and the first one is recorded (region,
// byte offset from the region's start) -- no trap.  Behind every region lie 256 guard bytes that
// vs_bank_state verifies.  Either finding is reported as VS_ERR_BOUNDS.
enum DbgRegion { DR_BANK_K = 0, DR_BANK_V, DR_PREFIX_K, DR_PREFIX_V, DR_TAIL_K, DR_TAIL_V, DR_EMB, DR_META, DR_ORDER,
                 DR_SLOT_FRAME, DR_SLOT_POS, DR_EVICT_LOG, DR_SCORES, DR_STEP_SLOT, DR_CHUNK_SLOT, DR_CHUNK_VICTIM,
                 DR_GEMM_FLAGS, DR_HBUF0, DR_HBUF1, DR_XN, DR_ROW_SS, DR_Q, DR_Q_LO, DR_Q_TILED, DR_KF, DR_VF, DR_ROPE,
                 DR_OBUF, DR_EMB_STAGE, DR_CHUNK_SCORES, DR_GEMM_XCHG, DR_ACT, DR_COUNT };
struct DebugTable {
  unsigned long long begin[DR_COUNT], end[DR_COUNT];   // device addresses
  int bad_region;                                      // -1, or the region of the first refused store
  long long bad_offset;
};
#if defined(VS_DEBUG_BOUNDS) && defined(__CUDACC__)
__device__ __forceinline__ bool vs_store_ok(const BatchParams& bp, int region, const void* p, size_t bytes) {
  if (bp.dbg == nullptr) return true;
  const unsigned long long a = reinterpret_cast<unsigned long long>(p);
  if (a >= bp.dbg->begin[region] && a + bytes <= bp.dbg->end[region]) return true;
  if (atomicCAS(&bp.dbg->bad_region, -1, region) == -1) bp.dbg->bad_offset = (long long)(a - bp.dbg->begin[region]);
  return false;
}
#define VS_STORE_OK(bp, region, p, bytes) vs_store_ok(bp, region, p, bytes)
#else
#define VS_STORE_OK(bp, region, p, bytes) true
#endif

// ---- shapes ----------------------------------------------------------------------------
struct Dims {
  int L, d, Hq, Hkv, D, G, E_out;
  int d_ff;                                      // 0, or the SwiGLU width of the full decoder block
  int vocab;                                     // 0, or the rows of the vocabulary projection (language-model head)
  int ss_parts;                                  // parts a row's sum of squares comes in: Hkv (from the attention kernel) or d / 128
  int maxN, maxP, maxT, maxStepT, M, slots, S, maxChunk;   // maxP / maxT: allocated rows (>= 1)
  int capP, capT;                                // caller's prefix / tail capacities
  int rows_per_stream_max, R_max;
  int log_cap;
  int agg_mode, evict_policy, use_rmsnorm, residual, out_fp32;
  float rope_theta, rms_eps;
};

constexpr int KSPLIT_MAX = 4;   // CTAs sharing one output tile of the projection along K
constexpr int DEC_SPLIT_MAX = 8;      // key splits of the decode attention = CTAs of one cluster
constexpr int GEMM_BLOCK_M = 128;
constexpr int GEMM_BLOCK_K = 64;
constexpr int GEMM_XCHG_CTAS = 160;   // most CTAs a K-split projection launches (one per SM)

// ---- workspace layout (byte offsets from the workspace base) ----------------------------
struct Layout {
  // persistent: stream state
  size_t bank_k, bank_v;        // bf16 [L][S][Hkv][slots][D]
  size_t prefix_k, prefix_v;    // bf16 [L][S][Hkv][maxP][D]
  size_t tail_k, tail_v;        // bf16 [L][S][Hkv][maxT][D]
  size_t emb;                   // bf16 [S][slots][d]
  size_t meta;                  // StreamMeta [S]
  size_t order;                 // int32 [S][slots]  temporal index -> physical slot
  size_t slot_frame;            // int32 [S][slots]  frame id held by a slot, -1 = free
  size_t slot_pos;              // int64 [S][slots]  position id of the carrier
  size_t evict_log;             // int32 [S][log_cap][2]
  size_t scores;                // f64   [S][slots]
  size_t inv_freq;              // f64   [D/2]
  size_t status;                // int32 [8]
  size_t step_slot;             // int32 [S]  free slot as the running frame step found it
  size_t chunk_slot;            // int32 [VS_MAX_BATCH]  chunked prefill: slot each frame's carrier went to
  size_t chunk_victim;          // int32 [VS_MAX_BATCH]  ... and whom its bank update evicted (index on the bank axis)
  size_t gemm_flags;            // int32 [GEMM_XCHG_CTAS]  projection K split: partials delivered per slice owner
  size_t lm_keys, lm_tickets;   // uint64 [256], int32 [256]  language-model head: greedy-choice keys and tickets per row
  size_t persistent_end;
  // per-step scratch
  size_t hbuf[2];               // bf16 [R_max][d]  residual ping-pong; hbuf[0] holds [E; carrier]
  size_t xn;                    // bf16 [R_max][d]  layer input times the RMSNorm gain (only with a gain vector)
  size_t row_ss;                // f32  [2][R_max][ss_parts] parts of the rows' sums of squares (RMSNorm; second half: the
                                //      post-attention norm of the full decoder block)
  size_t act;                   // bf16 [R_max][d_ff]  gated activation of the full decoder block
  size_t q;                     // bf16 [R_max][Hq*D]
  size_t q_lo;                  // bf16 [R_max][Hq*D]  low-order half of the rotated query
  size_t q_tiled;               // bf16 [row tiles][Hkv][hi | lo][128][D]  the pair as the tensor-core attention reads it
  size_t kf, vf;                // bf16 [R_max][Hkv*D]
  size_t rope;                  // float2 [R_max][D/2]
  size_t obuf;                  // f32  [R_max][Hq*D] (holds bf16 or fp32 rows)
  size_t emb_stage;             // bf16 [max_chunk][d]  chunked prefill: carrier embeddings before they have a slot
  size_t chunk_scores;          // f64  [max_chunk][slots + max_chunk]  chunked prefill: cosines of (frame, candidate) pairs
  size_t gemm_xchg;             // f32  [GEMM_XCHG_CTAS][256][128]  projection K split: partial tiles
  size_t scratch_begin, scratch_end;
  size_t total;
  // checked build: the regions as the kernels name them, and the table the kernels read
  size_t region_begin[DR_COUNT], region_end[DR_COUNT];
  size_t dbg_table;
};

// ---- timeline trace (only in a -DVS_TRACE build; the product build compiles none of it) ----------
// The first and the last CTA of a launch store the global time (ns) of a few phases into fixed slots
// of a log the host reads back -- slot = (kernel, phase, first / last CTA, launch sequence number
// modulo VS_TRACE_RING) -- with programmatic dependent launch left as it is.  A plain store: the
// stamping thread waits for nothing.
#if defined(VS_TRACE) && defined(__CUDACC__)
constexpr unsigned VS_TRACE_RING = 64;
constexpr unsigned VS_TRACE_WORDS = 8 * 16 * 2 * VS_TRACE_RING;
__device__ __forceinline__ void vs_stamp(const BatchParams& bp, unsigned kernel, unsigned phase, unsigned thread = 0) {
  if (bp.trace == nullptr || threadIdx.x != thread) return;
  const bool first = (blockIdx.x | blockIdx.y | blockIdx.z) == 0;
  const bool last = blockIdx.x == gridDim.x - 1 && blockIdx.y == gridDim.y - 1 && blockIdx.z == gridDim.z - 1;
  if (!first && !last) return;
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  bp.trace[(((kernel & 7u) * 16u + (phase & 15u)) * 2u + (last ? 1u : 0u)) * VS_TRACE_RING + (bp.trace_seq % VS_TRACE_RING)] = t;
}
#define VS_STAMP(bp, kernel, phase) vs_stamp(bp, kernel, phase)
#define VS_STAMP_BY(bp, kernel, phase, thread) vs_stamp(bp, kernel, phase, thread)
#else
#define VS_STAMP(bp, kernel, phase)
#define VS_STAMP_BY(bp, kernel, phase, thread)
#endif

// ---- programmatic dependent launch ------------------------------------------------------
// Every kernel of a step is launched with programmatic stream serialisation: it may be
// scheduled while its predecessor in the stream is still running.  The rules that keep this
// safe:
//  * a CTA lets the dependents start (pdl_launch_dependents) only after its own pdl_wait, or by
//    exiting; so when a kernel starts, every kernel older than its predecessor has completed and
//    flushed, and completion is transitive along the stream;
//  * before its pdl_wait a kernel may do set-up (barriers, tensor memory, descriptor prefetch,
//    arithmetic on its parameters) and may READ what neither its predecessor nor it writes: the
//    weights, K/V rows and bank metadata of earlier steps;
//  * everything the predecessor writes is read, and everything any earlier kernel may still read
//    is written, only after pdl_wait.  CTAs that need nothing from the predecessor (the bank
//    update beside the attention) skip the wait.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Asks the memory system to bring [p, p + bytes) into L2 (no destination, no completion to wait
// for).  p 16-byte aligned, bytes a multiple of 16.  Used for weight rows: the matrices are
// constant, so the request needs no ordering with any other kernel.
__device__ __forceinline__ void prefetch_l2_bulk(const void* p, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// ---- launch wrappers (each returns the cudaError_t of the launch) -----------------------
struct PoolArgs {
  const bf16* hidden;            // [n_active][N][d]
  const bf16* carrier_override;  // [n_active][d] or null
  bf16* x;                       // [n_active][N+1][d]
  bf16* emb;                     // [S][slots][d]
  const StreamMeta* meta;        // [S]
  int32_t* step_slot;            // [S] copy of meta.free_slot for the rest of the step
  bf16* emb_stage;               // chunked prefill: [n_active][d] carrier embeddings parked here instead of the
                                 // bank (their slots are only known as the bank updates run); else null
  const double* inv_freq;        // [D/2]
  float2* rope;                  // [n_active][N+1][D/2]
  int N, d, D, slots, M, agg_mode;
};
cudaError_t launch_pool(const PoolArgs& a, const BatchParams& bp, cudaStream_t st);

struct RopeArgs {
  const double* inv_freq;
  float2* rope;                  // [n_active][T][D/2]
  int D;
};
cudaError_t launch_rope_table(const RopeArgs& a, const BatchParams& bp, cudaStream_t st);

// sum of squares of every row -> row_ss[row][parts] (part 0; the other parts zero); with a gain vector hg = bf16(h * gain)
cudaError_t launch_rms_stats(const bf16* h, const bf16* gain, bf16* hg, float* row_ss, int parts, int rows, int d,
                             cudaStream_t st);
// Input of the language-model head: xn[row] = bf16(h[row]) (times gain, rounded again, with a gain vector), the
// sum of squares of bf16(h[row]) in part 0 of row_ss[row][parts].  h is fp32 or bf16.
cudaError_t launch_lm_norm(const void* h, int h_fp32, const bf16* gain, bf16* xn, float* row_ss, int parts, int rows, int d,
                           cudaStream_t st);
// token[row] = index of the largest of logits[row][0..vocab), the lowest index among equals, NaN below everything.
// keys[rows] and tickets[rows] are scratch that is zero between calls (the kernel leaves it so).
cudaError_t launch_argmax_rows(const float* logits, int32_t* token, unsigned long long* keys, int* tickets, int rows, int vocab,
                               cudaStream_t st);

// What the projection epilogue writes (finished rows: bias, RoPE, bf16) and where rows persist.
struct ProjectionOut {
  const bf16* bias;              // [E_out] or null
  const float* row_ss;           // [rows][ss_parts] parts of each row's sum of squares (RMSNorm: the accumulated row is
                                 // scaled by 1 / sqrt(sum / d + norm_eps), the parts added in index order), or null
  int ss_parts;
  int norm_inline;               // matrix-vector kernel only: it computes the RMSNorm scale (and h * gain) itself
  const bf16* norm_gain;         // [d] or null
  float norm_eps;
  const float2* rope;            // [rows][D/2] (cos, sin); null: the kernel derives them from inv_freq (few rows only)
  const double* inv_freq;        // [D/2]
  bf16* q;                       // [rows][Hq*D]  rotated query, leading bf16 part
  bf16* q_lo;                    // [rows][Hq*D]  bf16(query - q): the pair carries 16 mantissa bits
  bf16* q_tiled;                 // tensor-core GEMM only, or null: the pair in the attention kernel's operand layout
                                 // instead (see AttnArgs::q_tiled); rows_per_stream rows per batch entry
  bf16* kf;                      // [rows][Hkv*D] rotated keys of this step
  bf16* vf;                      // [rows][Hkv*D]
  bf16* bank_k; bf16* bank_v;    // layer base [S][Hkv][slots][D]
  bf16* text_k; bf16* text_v;    // layer base [S][Hkv][text_cap][D]: prefix or tail
  const int32_t* free_slot;      // free slot of stream s at free_slot[s * free_slot_stride]
  int free_slot_stride;
  int Hq, Hkv, D, slots, text_cap, M;
  int mode;                      // 0 frame step (carrier row -> bank), 1 text -> prefix, 2 text -> tail,
                                 // 3 chunk of frames (nothing kept here: a commit kernel copies the carrier rows),
                                 // 4 plain linear layer + residual, 5 SwiGLU gate/up pair (the rest of the decoder block),
                                 // 6 plain linear layer, fp32 rows to final_out[row][E_out] (the vocabulary projection)
  // modes 4 and 5: lin_out[row][E] = bf16(acc * row scale + lin_res[row][E]) (mode 4, E = E_out), or
  // lin_out[row][E_out / 2] = bf16(SiLU(gate) * up) (mode 5: every 128-row weight tile is 64 gate rows, then 64 up rows)
  bf16* lin_out; const bf16* lin_res;
  int lin_out_region;            // checked build: the workspace region lin_out lies in
  void* final_out; int final_fp32;   // mode 4: the rows also go here (the step's output), or null
  float* ss_out;                 // mode 4: sum of squares of the stored rows, one part per 128-feature tile:
  int ss_out_parts;              //   ss_out[row][ss_out_parts], this launch's tile m at part m; or null
  const bf16* next_gain; bf16* xn_out;   // mode 4 with ss_out: xn_out = bf16(stored row * next_gain), or null
};

struct GemmArgs {
  CUtensorMap tm_w2;             // mode 5: the up matrix (tm_w is then the gate matrix, both with boxes of 64 rows)
  CUtensorMap tm_w;              // [E_out, d] bf16, box 64 x 128, 128-byte swizzle
  CUtensorMap tm_x;              // [rows, d] bf16, box 64 x tile_n, 128-byte swizzle
  ProjectionOut out;
  int rows, E_out, d;
  int tile_n, n_tiles, ksplit;   // ksplit = CTAs per output tile along K: 1, 2 or 4
  int m_sub;                     // 1: 128 weight rows per CTA; 2: 256 (two accumulators), only without a K split
  float* xchg;                   // [m_tiles*n_tiles][ksplit][tile_n][128] fp32, needed when ksplit > 1
  int* flags;                    // [m_tiles*n_tiles][ksplit], zero between launches
  int n_sms;
  int* status;
};
cudaError_t launch_qkv_gemm(const GemmArgs& a, const BatchParams& bp, cudaStream_t st);
cudaError_t qkv_gemm_init();     // opt-in shared memory attribute, once per process/device
// Projection of one to four rows of a text step as a matrix-vector product (no RoPE table needed).
bool qkv_gemv_supported(const ProjectionOut& o, int rows, int d);
cudaError_t qkv_gemv_init();     // opt-in shared memory attribute, once per process/device
cudaError_t launch_qkv_gemv(const bf16* W, const bf16* x, const ProjectionOut& o, const BatchParams& bp, int rows, int E_out,
                            int d, bool l2_ahead, cudaStream_t st);   // l2_ahead: the matrix comes from HBM (several layers): ask for
                                                                       // all of it before the wait on the stream's earlier kernels

struct BankUpdateArgs {
  const bf16* emb;               // [S][slots][d]
  StreamMeta* meta;
  const int32_t* step_slot;      // [S] the slot the incoming carrier was written to
  // chunked prefill: the incoming carrier's embedding is still parked at `incoming_emb`; the slot
  // is meta.free_slot, recorded in *record_slot, and the embedding moves into the bank here
  const bf16* incoming_emb;
  int32_t* record_slot;
  // ... and whom the update evicted, as an index on the chunk's bank axis: the slot for a carrier
  // that was in the bank before the chunk, chunk_l1 + i for the carrier of the chunk's frame i,
  // -1 for nobody
  int32_t* record_victim;
  long long chunk_first_frame;
  int chunk_l1;                  // bank slots on the key axis of the chunk's frames
  // ... planned by ONE block for all frames in turn: the cosine of every (frame, candidate) pair was
  // worked out beforehand, pre_scores[b * pre_stride + index on the chunk's bank axis]; else null
  const double* pre_scores;
  int pre_stride;
  int32_t* order; int32_t* slot_frame; int64_t* slot_pos; int32_t* evict_log; double* scores;
  int d, slots, M, policy, log_cap;
};
// One segment of the attention's key axis.  Its K and V rows are reached through tensor maps with
// dimensions {head_dim, rows, Z} and a box of {64, ATTN_KEY_BOX, 1} elements (128-byte swizzle):
// prefix / bank / tail maps span every layer, stream and KV head on Z; the step's own rows
// ([rows][Hkv * D]) put the KV head on Z.
constexpr int ATTN_KEY_BOX = 64;   // key rows per bulk tensor copy; segments start on multiples of it on the key axis
struct AttnSegment {
  CUtensorMap tk, tv;
  int kind;                      // 0 prefix, 1 bank, 2 tail (earlier tokens of the turn), 3 this step's rows (causal),
                                 // 4 carriers of the chunk's earlier frames (entry b sees b of them)
  int rows_per_batch;            // row coordinate of batch entry b's first key: b * rows_per_batch
  int z0, z_per_stream;          // Z coordinate = z0 + stream id * z_per_stream + KV head
};
struct AttnArgs {
  const bf16* q;                 // [rows][Hq*D]
  const bf16* q_lo;
  const bf16* q_tiled;           // or: the query as the projection's GEMM leaves it for this kernel, one block per
                                 // (batch entry, 16-token row tile, KV head): [hi | lo][128 rows = g * 16 + token][D],
                                 // 128-byte swizzled like the MMA operand, fetched by one bulk copy
  AttnSegment seg[4];
  int n_seg;
  void* out;                     // [rows][Hq*D], bf16 or fp32
  int out_fp32;
  const bf16* h_in;              // residual input [rows][d] or null
  bf16* h_out;                   // residual output or null
  // RMSNorm of the layer that follows (needs h_out): the sum of squares of every stored residual row over this KV
  // head's query heads -> ss_out[row][Hkv]; with a gain vector also xn_out = bf16(h_out * next_gain); or null
  float* ss_out;
  const bf16* next_gain;
  bf16* xn_out;
  int h_out_region;              // checked build: which residual buffer h_out is (DR_HBUF0 / DR_HBUF1)
  const int32_t* free_slot;      // free slot of stream s at free_slot[s * free_slot_stride]
  int free_slot_stride;
  int Hq, Hkv, D, slots, M;
  float scale_log2e;
  // CTAs that share the key tiles of one (row tile, KV head, batch entry): a thread-block cluster of 1 .. 4
  // whose members each take a contiguous run of key tiles and combine through distributed shared memory
  int nsplit;
  // frame steps, last layer: the bank update (it needs the carrier embeddings only) is done by the CTAs of one more
  // plane of the grid (blockIdx.y == Hkv), which take its bank_blocks blocks of work in turn; 0: none
  BankUpdateArgs bank;
  int bank_blocks;
  // chunk of frames in ONE launch (entry b = frame b): the bank segment is the bank as it was
  // before the chunk (chunk_count0 carriers) for every frame; what frame b must not see -- the slot
  // that was free, and whoever the updates of frames 0 .. b-1 evicted (chunk_victim) -- is masked
  int chunk_mode, chunk_count0;
  const int32_t* chunk_victim;
};
// chunked prefill: the bank update of one frame as a launch of its own (it precedes the projection)
cudaError_t launch_bank_update(const BankUpdateArgs& a, const BatchParams& bp, bool full, cudaStream_t st);
// chunked prefill, policies that score against the incoming carrier only: all cosines of the chunk
// in one launch (frame b against bank slots 0 .. l1-1 and the chunk's carriers 0 .. b-1), then the
// F bank updates in turn by one block
cudaError_t launch_chunk_scores(const BankUpdateArgs& a, const BatchParams& bp, const bf16* emb_stage, double* out, cudaStream_t st);
cudaError_t launch_chunk_plan(const BankUpdateArgs& a, const BatchParams& bp, cudaStream_t st);
// chunked prefill, after a layer's attention: the K/V rows of the chunk's carriers that are still in
// the bank go to their slots
struct ChunkKvCommitArgs {
  const bf16* kf; const bf16* vf;          // step K/V [F][N+1][Hkv*D]
  bf16* bank_k; bf16* bank_v;              // this layer's bank [S][Hkv][slots][D]
  const int32_t* chunk_slot; const int32_t* chunk_victim;
  int F, N, Hkv, D, slots, sid, l1;
};
cudaError_t launch_chunk_kv_commit(const ChunkKvCommitArgs& a, cudaStream_t st);
constexpr int ATTN_EXCL_BITS = 8192;   // most (bank slots + chunk frames) the one-launch chunk attention can mask
cudaError_t launch_prefill_attention_tc(const AttnArgs& a, const BatchParams& bp, int* status, cudaStream_t st);
cudaError_t prefill_attention_tc_init();
int prefill_attention_max_clusters(int head_dim, int s);
constexpr int ATTN_MAX_SPLIT = 2;   // clusters of 3 or 4 do not all fit on the GPU at once (one CTA per SM, clusters inside a GPC)

struct DecodeArgs {
  const bf16* q;                 // [n_active][Hq*D]
  const bf16* q_lo;
  const bf16* prefix_k; const bf16* prefix_v;  // layer base [S][Hkv][maxP][D]
  const bf16* bank_k;   const bf16* bank_v;    // [S][Hkv][slots][D]
  const bf16* tail_k;   const bf16* tail_v;    // [S][Hkv][maxT][D]
  void* out;                     // [n_active][Hq*D], bf16 or fp32
  int out_fp32;
  const bf16* h_in; bf16* h_out;
  int h_out_region;              // checked build: which residual buffer h_out is (DR_HBUF0 / DR_HBUF1)
  const StreamMeta* meta;
  int Hq, Hkv, D, slots, M, maxP, maxT;
  int nsplit;                    // CTAs sharing one row's keys (a cluster): 1, 2, 4 or 8
  int to_prefix;                 // 1: the keys are the prefix alone (incl. the new token)
  float scale_log2e;
};
cudaError_t launch_decode_attention(const DecodeArgs& a, const BatchParams& bp, cudaStream_t st);


// rows i < count of x = emb[sid][order[i]]: the bank's carrier embeddings in temporal order
cudaError_t launch_gather_carriers(const bf16* emb, const int32_t* order, bf16* x, int sid, int slots, int d, int count,
                                   cudaStream_t st);
cudaError_t launch_poison(void* p, size_t bytes, cudaStream_t st);
cudaError_t launch_reset(StreamMeta* meta, int32_t* slot_frame, int slots, const BatchParams& bp, cudaStream_t st);

}  // namespace vs
