// Host layer of the C ABI: argument checks, workspace carve-up, launch sequencing.
// Per frame (Section 3.3, prefilling): pool -> per layer [norm] -> QKV GEMM (epilogue: RoPE,
// carrier K/V into the bank's free slot) -> attention [-> residual] -> bank update (eviction
// scoring when the bank is full, then append).  Per text step (Section 3.3, decoding): RoPE
// table -> per layer [norm] -> GEMM (epilogue: K/V appended to prefix or tail) -> attention.  Nothing here allocates device memory or synchronises, except
// create / bank_state / last_step_kv.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "vs_common.cuh"

using namespace vs;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct HostStream {
  int64_t frames_seen = 0, next_pos = 0, prefix_len = 0, text_len = 0;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int fill_dims(const vs_config* c, Dims& D) {
  if (c == nullptr) return VS_ERR_INVALID_ARG;
  if (c->n_layers < 1 || c->d_model < 64 || c->n_q_heads < 1 || c->n_kv_heads < 1) return VS_ERR_INVALID_ARG;
  if (c->n_streams < 1 || c->n_streams > VS_MAX_BATCH) return VS_ERR_INVALID_ARG;
  if (c->max_tokens_per_frame < 1 || c->max_prefix < 0 || c->max_text < 0 || c->bank_capacity < 0) return VS_ERR_INVALID_ARG;
  if (c->max_step_tokens < 1 || c->evict_log_capacity < 0) return VS_ERR_INVALID_ARG;
  if (c->out_dtype < 0 || c->out_dtype > 1) return VS_ERR_INVALID_ARG;
  if (c->max_chunk_frames < 0 || c->max_chunk_frames > VS_MAX_BATCH) return VS_ERR_INVALID_ARG;
  if (c->agg_mode < 0 || c->agg_mode > 1 || c->evict_policy < 0 || c->evict_policy > 2) return VS_ERR_INVALID_ARG;
  if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return VS_ERR_INVALID_ARG;
  if (c->d_model % 64 != 0) return VS_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return VS_ERR_UNSUPPORTED;
  if (c->n_q_heads % c->n_kv_heads != 0 || c->n_q_heads / c->n_kv_heads > 8) return VS_ERR_UNSUPPORTED;
  if (c->max_tokens_per_frame + 1 > 256) return VS_ERR_UNSUPPORTED;
  if (c->n_layers > 1 && !c->residual) return VS_ERR_INVALID_ARG;
  if (c->residual && c->n_q_heads * c->head_dim != c->d_model) return VS_ERR_INVALID_ARG;
  D.L = c->n_layers; D.d = c->d_model; D.Hq = c->n_q_heads; D.Hkv = c->n_kv_heads; D.D = c->head_dim;
  D.G = D.Hq / D.Hkv; D.E_out = (D.Hq + 2 * D.Hkv) * D.D;
  D.maxN = c->max_tokens_per_frame; D.maxP = c->max_prefix > 0 ? c->max_prefix : 1;
  D.maxT = c->max_text > 0 ? c->max_text : 1; D.maxStepT = c->max_step_tokens;
  D.capP = c->max_prefix; D.capT = c->max_text;
  D.M = c->bank_capacity; D.slots = D.M + 1; D.S = c->n_streams;
  D.rows_per_stream_max = (D.maxN + 1 > D.maxStepT) ? D.maxN + 1 : D.maxStepT;
  D.maxChunk = c->max_chunk_frames > 1 ? c->max_chunk_frames : 1;
  D.R_max = D.rows_per_stream_max * D.S;
  if (D.maxChunk * (D.maxN + 1) > D.R_max) D.R_max = D.maxChunk * (D.maxN + 1);
  if (D.M > D.R_max) D.R_max = D.M;               // vs_bank_forward runs the whole bank as one step
  D.log_cap = c->evict_log_capacity;
  D.agg_mode = c->agg_mode; D.evict_policy = c->evict_policy; D.use_rmsnorm = c->use_rmsnorm ? 1 : 0;
  D.residual = c->residual ? 1 : 0; D.out_fp32 = c->out_dtype == 1 ? 1 : 0; D.rope_theta = c->rope_theta; D.rms_eps = c->rms_eps;
  D.d_ff = c->d_ff;
  if (c->d_ff < 0) return VS_ERR_INVALID_ARG;
  if (c->d_ff > 0 && (!c->residual || c->n_q_heads * c->head_dim != c->d_model)) return VS_ERR_INVALID_ARG;
  if (c->d_ff > 0 && (c->d_ff % 64 != 0 || c->d_model % 128 != 0)) return VS_ERR_UNSUPPORTED;
  D.ss_parts = D.d_ff > 0 ? D.d / 128 : D.Hkv;
  D.vocab = c->vocab;
  if (c->vocab < 0) return VS_ERR_INVALID_ARG;
  if (c->vocab > 0 && c->vocab % GEMM_BLOCK_M != 0) return VS_ERR_UNSUPPORTED;
  return VS_OK;
}

// Checked build: 256 guard bytes behind every region (vs_bank_state verifies them).
#ifdef VS_DEBUG_BOUNDS
constexpr size_t kGuardBytes = 256;
#else
constexpr size_t kGuardBytes = 0;
#endif
constexpr unsigned char kGuardByte = 0xC5;

void fill_layout(const Dims& D, Layout& Lo) {
  size_t off = 0;
  size_t last_bytes = 0;
  auto take = [&](size_t bytes) { size_t o = off; last_bytes = bytes; off = align_up(off + bytes, 256) + kGuardBytes; return o; };
  for (int r = 0; r < DR_COUNT; ++r) { Lo.region_begin[r] = 0; Lo.region_end[r] = 0; }
  auto reg = [&](int r, size_t o) { Lo.region_begin[r] = o; Lo.region_end[r] = o + last_bytes; return o; };
  const size_t kv_bank = (size_t)D.L * D.S * D.Hkv * D.slots * D.D * 2;
  const size_t kv_pre = (size_t)D.L * D.S * D.Hkv * D.maxP * D.D * 2;
  const size_t kv_tail = (size_t)D.L * D.S * D.Hkv * D.maxT * D.D * 2;
  Lo.bank_k = reg(DR_BANK_K, take(kv_bank)); Lo.bank_v = reg(DR_BANK_V, take(kv_bank));
  Lo.prefix_k = reg(DR_PREFIX_K, take(kv_pre)); Lo.prefix_v = reg(DR_PREFIX_V, take(kv_pre));
  Lo.tail_k = reg(DR_TAIL_K, take(kv_tail)); Lo.tail_v = reg(DR_TAIL_V, take(kv_tail));
  Lo.emb = reg(DR_EMB, take((size_t)D.S * D.slots * D.d * 2));
  Lo.meta = reg(DR_META, take((size_t)D.S * sizeof(StreamMeta)));
  Lo.order = reg(DR_ORDER, take((size_t)D.S * D.slots * 4));
  Lo.slot_frame = reg(DR_SLOT_FRAME, take((size_t)D.S * D.slots * 4));
  Lo.slot_pos = reg(DR_SLOT_POS, take((size_t)D.S * D.slots * 8));
  Lo.evict_log = reg(DR_EVICT_LOG, take((size_t)D.S * (D.log_cap > 0 ? D.log_cap : 1) * 8));
  Lo.scores = reg(DR_SCORES, take((size_t)D.S * D.slots * 8));
  Lo.inv_freq = take((size_t)(D.D / 2) * 8);
  Lo.status = take(8 * 4);
  Lo.step_slot = reg(DR_STEP_SLOT, take((size_t)D.S * 4));
  Lo.chunk_slot = reg(DR_CHUNK_SLOT, take((size_t)VS_MAX_BATCH * 4));
  Lo.chunk_victim = reg(DR_CHUNK_VICTIM, take((size_t)VS_MAX_BATCH * 4));
  Lo.gemm_flags = reg(DR_GEMM_FLAGS, take((size_t)GEMM_XCHG_CTAS * 4));
  Lo.lm_keys = take((size_t)256 * 8);          // language-model head: per-row argmax keys and tickets, zero between calls
  Lo.lm_tickets = take((size_t)256 * 4);
  Lo.dbg_table = take(sizeof(DebugTable));
  Lo.persistent_end = off;
  Lo.scratch_begin = off;
  Lo.hbuf[0] = reg(DR_HBUF0, take((size_t)D.R_max * D.d * 2));
  Lo.hbuf[1] = reg(DR_HBUF1, take((size_t)D.R_max * D.d * 2));
  Lo.xn = reg(DR_XN, take((size_t)D.R_max * D.d * 2));
  Lo.row_ss = reg(DR_ROW_SS, take((size_t)2 * D.R_max * D.ss_parts * 4));
  Lo.act = reg(DR_ACT, take(D.d_ff > 0 ? (size_t)D.R_max * D.d_ff * 2 : 256));
  Lo.q = reg(DR_Q, take((size_t)D.R_max * D.Hq * D.D * 2));
  Lo.q_lo = reg(DR_Q_LO, take((size_t)D.R_max * D.Hq * D.D * 2));
  // the query in the attention kernel's operand layout: per batch entry ceil(rows / 16) row tiles, per tile and KV
  // head a block of [hi | lo][128][D]
  Lo.q_tiled = reg(DR_Q_TILED, take(((size_t)D.R_max / 16 + (size_t)VS_MAX_BATCH + 1) * D.Hkv * 2 * 128 * D.D * 2));
  Lo.kf = reg(DR_KF, take((size_t)D.R_max * D.Hkv * D.D * 2));
  Lo.vf = reg(DR_VF, take((size_t)D.R_max * D.Hkv * D.D * 2));
  Lo.rope = reg(DR_ROPE, take((size_t)D.R_max * (D.D / 2) * 8));
  Lo.obuf = reg(DR_OBUF, take((size_t)D.R_max * D.Hq * D.D * 4));
  Lo.emb_stage = reg(DR_EMB_STAGE, take((size_t)D.maxChunk * D.d * 2));
  Lo.chunk_scores = reg(DR_CHUNK_SCORES, take(D.maxChunk > 1 ? (size_t)D.maxChunk * (D.slots + D.maxChunk) * 8 : 8));
  Lo.gemm_xchg = reg(DR_GEMM_XCHG, take((size_t)GEMM_XCHG_CTAS * 256 * GEMM_BLOCK_M * 4));
  Lo.scratch_end = off;
  Lo.total = off;
}

}  // namespace

struct vs_stream {
  Dims dm;
  Layout lo;
  uint8_t* ws = nullptr;
  size_t ws_bytes = 0;
  int device = 0;
  int n_sms = 0;
  // chunked prefill: the chunk's bank updates run on a stream of their own beside the projection
  cudaStream_t side_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  std::vector<const bf16*> w, bias, gain;
  std::vector<const bf16*> gain2;                                  // full decoder block: post-attention RMSNorm gains
  std::vector<CUtensorMap> tm_wo, tm_gate, tm_up, tm_down;         // ... and its weight matrices
  std::vector<CUtensorMap> tm_w;
  CUtensorMap tm_lm;                         // language-model head: the vocabulary projection [vocab][d]
  const bf16* gain_f = nullptr;              // ... and the gain of the final RMSNorm (null: unit gain)
  // key/value tensor maps of the attention: the persistent ones span all layers, streams and KV heads
  CUtensorMap tm_prefix_k, tm_prefix_v, tm_bank_k, tm_bank_v, tm_tail_k, tm_tail_v;
  CUtensorMap tm_step_k, tm_step_v;          // the step's own rows [rows][Hkv * D]; re-encoded when `rows` changes
  int step_map_rows = -1;
  int attn_clusters[ATTN_MAX_SPLIT + 1] = {0};   // clusters of s attention CTAs that can be resident at once
#ifdef VS_TRACE
  unsigned long long* trace = nullptr;
  unsigned trace_seq = 0;
#endif
  std::vector<HostStream> hs;
  EncodeTiledFn encode = nullptr;
  cudaStream_t last_stream = nullptr;
  int last_rows = 0;
  // launch accounting: counts always, CUDA-event timing of every launch when enabled
  int64_t launches[VS_N_KERNEL_CLASSES] = {0};
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_ev;          // pairs (start, stop)
  std::vector<int> prof_class;               // class of pair i
  size_t prof_used = 0;                      // pairs in use

  template <typename T>
  T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

namespace {

int encode_2d(vs_stream* h, CUtensorMap* tm, const void* base, uint64_t inner, uint64_t rows, uint32_t box_rows) {
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {(cuuint32_t)GEMM_BLOCK_K, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = h->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? VS_OK : VS_ERR_CUDA;
}

// K or V rows for the attention kernel: dimensions {head_dim, rows, Z}, box {64, ATTN_KEY_BOX, 1}, 128-byte swizzle;
// rows (and Z) beyond the extents read as zeros.
int encode_kv(vs_stream* h, CUtensorMap* tm, const void* base, uint64_t head_dim, uint64_t rows, uint64_t row_stride_bytes,
              uint64_t nz, uint64_t z_stride_bytes) {
  cuuint64_t dims[3] = {head_dim, rows, nz};
  cuuint64_t strides[2] = {row_stride_bytes, z_stride_bytes};
  cuuint32_t box[3] = {64, (cuuint32_t)ATTN_KEY_BOX, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = h->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? VS_OK : VS_ERR_CUDA;
}

// the step's own K/V rows as the attention's last segment: extent = the step's rows, so that a box
// reaching past them reads zeros, not what an earlier step left in the scratch
int ensure_step_maps(vs_stream* h, int rows) {
  if (h->step_map_rows == rows) return VS_OK;
  const Dims& D = h->dm;
  const uint64_t rs = (uint64_t)D.Hkv * D.D * 2, zs = (uint64_t)D.D * 2;
  if (encode_kv(h, &h->tm_step_k, h->at<bf16>(h->lo.kf), D.D, rows, rs, D.Hkv, zs) != VS_OK) return VS_ERR_CUDA;
  if (encode_kv(h, &h->tm_step_v, h->at<bf16>(h->lo.vf), D.D, rows, rs, D.Hkv, zs) != VS_OK) return VS_ERR_CUDA;
  h->step_map_rows = rows;
  return VS_OK;
}

// CTAs to spread the key tiles of a row tile over (one cluster): every CTA of the attention kernel takes
// a whole SM, all clusters must be resident at once, and a split pays only while it shortens the longest
// CTA's run of key tiles.  key_len[i]: segment lengths of the longest key axis among the listed entries.
int attn_split(const vs_stream* h, const BatchParams& bp, const int* key_len, int n_len) {
  int padded = 0;
  for (int i = 0; i < n_len; ++i) padded += (key_len[i] + ATTN_KEY_BOX - 1) / ATTN_KEY_BOX * ATTN_KEY_BOX;
  const int key_tiles = (padded + 127) / 128;
  const long long row_ctas = (long long)((bp.rows_per_stream + 15) / 16) * h->dm.Hkv * bp.n_active;
  int best = 1;
  for (int s = 2; s <= ATTN_MAX_SPLIT; ++s) {
    if (s > key_tiles || row_ctas * s > h->n_sms || h->attn_clusters[s] < row_ctas) break;
    if ((key_tiles + s - 1) / s == (key_tiles + best - 1) / best) continue;
    best = s;
  }
  return best;
}

// segments of the attention's key axis
void seg_stored(AttnSegment& sg, const CUtensorMap& k, const CUtensorMap& v, int kind, int layer, const Dims& D) {
  sg.tk = k; sg.tv = v; sg.kind = kind; sg.rows_per_batch = 0;
  sg.z0 = layer * D.S * D.Hkv; sg.z_per_stream = D.Hkv;
}
void seg_step(AttnSegment& sg, const CUtensorMap& k, const CUtensorMap& v, int kind, int rows_per_batch) {
  sg.tk = k; sg.tv = v; sg.kind = kind; sg.rows_per_batch = rows_per_batch; sg.z0 = 0; sg.z_per_stream = 0;
}

// Token tiling of the projection.  Every CTA re-reads its weight rows and its token columns from
// L2, (rows_w + tile_n) * (d / ksplit) * 2 bytes, and that traffic bounds the main loop.  The
// choice minimises waves * ((rows_w + tile_n) / ksplit + the cost of summing a K split, about 40
// row-equivalents) over 128- or 256-row weight tiles, the number of token tiles and the K split.
// A K split needs the whole grid resident at once (its CTAs wait for one another), one CTA per SM.
void choose_tiles(int K, int E, int n_sms, int rows, int& tile_n, int& n_tiles, int& ksplit, int& m_sub) {
  const int total_kb = K / GEMM_BLOCK_K;
  const int resident = n_sms < GEMM_XCHG_CTAS ? n_sms : GEMM_XCHG_CTAS;
  const int nt_min = (rows + 255) / 256;
  long long best = -1;
  m_sub = 1; ksplit = 1; n_tiles = nt_min; tile_n = ((rows + nt_min - 1) / nt_min + 15) / 16 * 16;
  for (int sub = 1; sub <= 2; ++sub) {
    if (sub == 2 && E % (2 * GEMM_BLOCK_M) != 0) continue;
    const int mt = (E + GEMM_BLOCK_M * sub - 1) / (GEMM_BLOCK_M * sub);
    for (int nt = nt_min; nt <= nt_min + 32; ++nt) {
      const int tn = ((rows + nt - 1) / nt + 15) / 16 * 16;
      if ((long long)(nt - 1) * tn >= rows && nt > nt_min) continue;      // an empty last tile
      if (tn < 64 && nt > nt_min) break;
      for (int ks = 1; ks <= KSPLIT_MAX; ks *= 2) {
        if (ks > 1 && (sub != 1 || total_kb % ks != 0 || mt * nt * ks > resident)) continue;
        const long long waves = ((long long)mt * nt * ks + n_sms - 1) / n_sms;
        const long long cost = waves * ((GEMM_BLOCK_M * sub + tn) * 4 / ks + (ks > 1 ? 160 : 0));   // in quarter rows
        if (best < 0 || cost < best) { best = cost; m_sub = sub; n_tiles = nt; tile_n = tn; ksplit = ks; }
      }
    }
  }
}

int check_ids(vs_stream* h, const int32_t* ids, int32_t n) {
  if (h == nullptr || ids == nullptr || n < 1 || n > h->dm.S) return VS_ERR_INVALID_ARG;
  bool seen[VS_MAX_BATCH] = {false};
  for (int i = 0; i < n; ++i) {
    if (ids[i] < 0 || ids[i] >= h->dm.S || seen[ids[i]]) return VS_ERR_INVALID_ARG;
    seen[ids[i]] = true;
  }
  return VS_OK;
}

#if defined(VS_DEBUG_BOUNDS)
#define VS_BP_INIT(h, bp) do { std::memset(&(bp), 0, sizeof(bp)); (bp).dbg = (h)->at<DebugTable>((h)->lo.dbg_table); } while (0)
#define VS_TRACE_NEXT(h, bp)
#elif defined(VS_TRACE)
#define VS_BP_INIT(h, bp) do { std::memset(&(bp), 0, sizeof(bp)); (bp).trace = (h)->trace; (bp).trace_seq = (h)->trace_seq; } while (0)
#define VS_TRACE_NEXT(h, bp) do { (bp).trace_seq = ++(h)->trace_seq; } while (0)
#else
#define VS_BP_INIT(h, bp) std::memset(&(bp), 0, sizeof(bp))
#define VS_TRACE_NEXT(h, bp)
#endif

#define VS_CK(expr) do { if ((expr) != cudaSuccess) return VS_ERR_CUDA; } while (0)

enum KernelClass { KC_POOL = 0, KC_ROPE, KC_RMSNORM, KC_GEMM, KC_GEMV, KC_PREFILL_ATTN, KC_DECODE_ATTN,
                   KC_EVICT, KC_COMMIT, KC_OTHER };
static_assert(KC_OTHER + 1 == VS_N_KERNEL_CLASSES, "kernel class table");

// One launch: counted, and bracketed by CUDA events on the launching stream when profiling is on.
#define VS_LAUNCH(h, st, kc, expr)                                                          \
  do {                                                                                      \
    const bool vs_t_ = (h)->prof_on && (h)->prof_used * 2 + 1 < (h)->prof_ev.size();        \
    if (vs_t_) VS_CK(cudaEventRecord((h)->prof_ev[(h)->prof_used * 2], (st)));              \
    VS_CK(expr);                                                                            \
    if (vs_t_) {                                                                            \
      VS_CK(cudaEventRecord((h)->prof_ev[(h)->prof_used * 2 + 1], (st)));                   \
      (h)->prof_class[(h)->prof_used++] = (kc);                                             \
    }                                                                                       \
    (h)->launches[(kc)] += 1;                                                               \
  } while (0)

// QKV projection of `rows` token rows read from `src` ([rows][d] bf16) for layer l, finished
// rows written as `po` says.
int run_projection(vs_stream* h, int l, const bf16* src, int rows, const ProjectionOut& po, const BatchParams& bp,
                   cudaStream_t st) {
  const Dims& D = h->dm;
  if (po.rope == nullptr && qkv_gemv_supported(po, rows, D.d) && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    // a text step of a few rows: bound by reading W once, done on the CUDA cores
    VS_LAUNCH(h, st, KC_GEMV, launch_qkv_gemv(h->w[l], src, po, bp, rows, D.E_out, D.d, D.L > 1, st));
    return VS_OK;
  }
  GemmArgs g;
  choose_tiles(D.d, D.E_out, h->n_sms, rows, g.tile_n, g.n_tiles, g.ksplit, g.m_sub);
  g.xchg = h->at<float>(h->lo.gemm_xchg);
  g.flags = h->at<int>(h->lo.gemm_flags);
  g.n_sms = h->n_sms;
  g.tm_w = h->tm_w[l]; g.tm_w2 = h->tm_w[l];
  if (encode_2d(h, &g.tm_x, src, (uint64_t)D.d, (uint64_t)rows, (uint32_t)g.tile_n) != VS_OK) return VS_ERR_CUDA;
  g.out = po;
  g.rows = rows; g.E_out = D.E_out; g.d = D.d;
  g.status = h->at<int>(h->lo.status);
  VS_LAUNCH(h, st, KC_GEMM, launch_qkv_gemm(g, bp, st));
  return VS_OK;
}

// One linear layer of the rest of the decoder block on the tensor cores: rows x K times W[E][K]^T, finished as
// `po` says (mode 4: + residual; mode 5: SwiGLU of a gate / up pair, E = 2 * d_ff).
int run_linear(vs_stream* h, const CUtensorMap& tm_w, const CUtensorMap& tm_w2, const bf16* src, int rows, int K, int E,
               ProjectionOut po, const BatchParams& bp, cudaStream_t st) {
  GemmArgs g;
  choose_tiles(K, E, h->n_sms, rows, g.tile_n, g.n_tiles, g.ksplit, g.m_sub);
  g.xchg = h->at<float>(h->lo.gemm_xchg);
  g.flags = h->at<int>(h->lo.gemm_flags);
  g.n_sms = h->n_sms;
  g.tm_w = tm_w; g.tm_w2 = tm_w2;
  if (encode_2d(h, &g.tm_x, src, (uint64_t)K, (uint64_t)rows, (uint32_t)g.tile_n) != VS_OK) return VS_ERR_CUDA;
  po.rope = h->at<float2>(h->lo.rope);      // (not read: nothing is rotated; selects the kernel variant that takes a table)
  po.inv_freq = h->at<double>(h->lo.inv_freq);
  po.Hq = 0; po.Hkv = 0; po.D = 128; po.slots = 0; po.text_cap = 0; po.M = 0; po.norm_inline = 0;
  g.out = po;
  g.rows = rows; g.E_out = E; g.d = K;
  g.status = h->at<int>(h->lo.status);
  VS_LAUNCH(h, st, KC_GEMM, launch_qkv_gemm(g, bp, st));
  return VS_OK;
}

// The rest of decoder layer l (Section 4.1: Qwen2 backbone) after its attention: a_rows = the attention rows (bf16,
// [rows][d]), h_in = the layer's input.  h1 = h_in + A W_o^T -> hbuf[1]; act = SiLU(n W_gate^T) * (n W_up^T);
// h2 = h1 + act W_down^T -> hbuf[0] (and `final_out` on the last layer).  Each stored tensor leaves its RMSNorm
// statistics (and, with a gain vector, its gained copy) for the projection that reads it next.
int run_block_rest(vs_stream* h, int l, int rows, const bf16* h_in, const bf16* a_rows, void* final_out, const BatchParams& bp,
                   cudaStream_t st) {
  const Dims& D = h->dm;
  const Layout& lo = h->lo;
  bf16* h1 = h->at<bf16>(lo.hbuf[1]);
  bf16* h2 = h->at<bf16>(lo.hbuf[0]);
  float* ss1 = h->at<float>(lo.row_ss);
  float* ss2 = ss1 + (size_t)D.R_max * D.ss_parts;
  ProjectionOut po;
  std::memset(&po, 0, sizeof(po));
  // W_o
  po.mode = 4; po.lin_out = h1; po.lin_res = h_in; po.lin_out_region = DR_HBUF1;
  if (D.use_rmsnorm) { po.ss_out = ss2; po.ss_out_parts = D.ss_parts; po.next_gain = h->gain2[l]; po.xn_out = h->at<bf16>(lo.xn); }
  int rc = run_linear(h, h->tm_wo[l], h->tm_wo[l], a_rows, rows, D.d, D.d, po, bp, st);
  if (rc != VS_OK) return rc;
  // gate and up with the SwiGLU epilogue
  std::memset(&po, 0, sizeof(po));
  po.mode = 5; po.lin_out = h->at<bf16>(lo.act); po.lin_out_region = DR_ACT;
  if (D.use_rmsnorm) { po.row_ss = ss2; po.ss_parts = D.ss_parts; po.norm_eps = D.rms_eps; }
  const bf16* n_src = (D.use_rmsnorm && h->gain2[l] != nullptr) ? h->at<bf16>(lo.xn) : h1;
  rc = run_linear(h, h->tm_gate[l], h->tm_up[l], n_src, rows, D.d, 2 * D.d_ff, po, bp, st);
  if (rc != VS_OK) return rc;
  // W_down
  std::memset(&po, 0, sizeof(po));
  po.mode = 4; po.lin_out = h2; po.lin_res = h1; po.lin_out_region = DR_HBUF0;
  po.final_out = final_out; po.final_fp32 = D.out_fp32;
  if (D.use_rmsnorm && l + 1 < D.L) { po.ss_out = ss1; po.ss_out_parts = D.ss_parts; po.next_gain = h->gain[l + 1]; po.xn_out = h->at<bf16>(lo.xn); }
  return run_linear(h, h->tm_down[l], h->tm_down[l], h->at<bf16>(lo.act), rows, D.d_ff, D.d, po, bp, st);
}

size_t layer_stride_bank(const Dims& D) { return (size_t)D.S * D.Hkv * D.slots * D.D; }
size_t layer_stride_prefix(const Dims& D) { return (size_t)D.S * D.Hkv * D.maxP * D.D; }
size_t layer_stride_tail(const Dims& D) { return (size_t)D.S * D.Hkv * D.maxT * D.D; }

}  // namespace

extern "C" {

const char* vs_status_string(int status) {
  switch (status) {
    case VS_OK: return "ok";
    case VS_ERR_INVALID_ARG: return "invalid argument";
    case VS_ERR_STATE: return "call not legal in the stream's current phase";
    case VS_ERR_CAPACITY: return "capacity exceeded";
    case VS_ERR_CUDA: return "CUDA call failed";
    case VS_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case VS_ERR_UNSUPPORTED: return "unsupported shape";
    case VS_ERR_BOUNDS: return "store outside a workspace region (checked build)";
    default: return "unknown status";
  }
}

int vs_workspace_bytes(const vs_config* cfg, size_t* out_bytes) {
  if (out_bytes == nullptr) return VS_ERR_INVALID_ARG;
  Dims D;
  const int rc = fill_dims(cfg, D);
  if (rc != VS_OK) return rc;
  Layout lo;
  fill_layout(D, lo);
  *out_bytes = lo.total;
  return VS_OK;
}

int vs_create_stream(const vs_config* cfg, const vs_weights* weights, void* workspace, size_t workspace_bytes,
                     vs_stream** out) {
  if (out == nullptr) return VS_ERR_INVALID_ARG;
  *out = nullptr;
  if (weights == nullptr || weights->w_qkv == nullptr || workspace == nullptr) return VS_ERR_INVALID_ARG;
  Dims D;
  const int rc = fill_dims(cfg, D);
  if (rc != VS_OK) return rc;
  Layout lo;
  fill_layout(D, lo);
  if (workspace_bytes < lo.total) return VS_ERR_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return VS_ERR_INVALID_ARG;
  for (int l = 0; l < D.L; ++l) {
    if (weights->w_qkv[l] == nullptr) return VS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(weights->w_qkv[l]) & 15u) != 0) return VS_ERR_INVALID_ARG;
  }
  VS_CK(cudaSetDevice(cfg->device));
  vs_stream* h = new (std::nothrow) vs_stream();
  if (h == nullptr) return VS_ERR_INVALID_ARG;
  h->dm = D; h->lo = lo; h->ws = static_cast<uint8_t*>(workspace); h->ws_bytes = workspace_bytes;
  h->device = cfg->device;
  if (cudaDeviceGetAttribute(&h->n_sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess) { delete h; return VS_ERR_CUDA; }
  h->hs.assign(D.S, HostStream());
  for (int l = 0; l < D.L; ++l) {
    h->w.push_back(static_cast<const bf16*>(weights->w_qkv[l]));
    h->bias.push_back(weights->b_qkv ? static_cast<const bf16*>(weights->b_qkv[l]) : nullptr);
    h->gain.push_back(weights->norm_w ? static_cast<const bf16*>(weights->norm_w[l]) : nullptr);
  }
  auto fail = [&](int code) { delete h; return code; };
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr ||
      qres != cudaDriverEntryPointSuccess)
    return fail(VS_ERR_CUDA);
  h->encode = reinterpret_cast<EncodeTiledFn>(fn);
  h->tm_w.resize(D.L);
  for (int l = 0; l < D.L; ++l)
    if (encode_2d(h, &h->tm_w[l], h->w[l], (uint64_t)D.d, (uint64_t)D.E_out, GEMM_BLOCK_M) != VS_OK) return fail(VS_ERR_CUDA);
  {
    const uint64_t nz = (uint64_t)D.L * D.S * D.Hkv, rb = (uint64_t)D.D * 2;
    if (encode_kv(h, &h->tm_prefix_k, h->ws + lo.prefix_k, D.D, D.maxP, rb, nz, (uint64_t)D.maxP * rb) != VS_OK ||
        encode_kv(h, &h->tm_prefix_v, h->ws + lo.prefix_v, D.D, D.maxP, rb, nz, (uint64_t)D.maxP * rb) != VS_OK ||
        encode_kv(h, &h->tm_bank_k, h->ws + lo.bank_k, D.D, D.slots, rb, nz, (uint64_t)D.slots * rb) != VS_OK ||
        encode_kv(h, &h->tm_bank_v, h->ws + lo.bank_v, D.D, D.slots, rb, nz, (uint64_t)D.slots * rb) != VS_OK ||
        encode_kv(h, &h->tm_tail_k, h->ws + lo.tail_k, D.D, D.maxT, rb, nz, (uint64_t)D.maxT * rb) != VS_OK ||
        encode_kv(h, &h->tm_tail_v, h->ws + lo.tail_v, D.D, D.maxT, rb, nz, (uint64_t)D.maxT * rb) != VS_OK)
      return fail(VS_ERR_CUDA);
  }
  if (D.d_ff > 0) {
    if (weights->w_o == nullptr || weights->w_gate == nullptr || weights->w_up == nullptr || weights->w_down == nullptr) return fail(VS_ERR_INVALID_ARG);
    h->tm_wo.resize(D.L); h->tm_gate.resize(D.L); h->tm_up.resize(D.L); h->tm_down.resize(D.L);
    for (int l = 0; l < D.L; ++l) {
      const void* ptrs[4] = {weights->w_o[l], weights->w_gate[l], weights->w_up[l], weights->w_down[l]};
      for (const void* q : ptrs) if (q == nullptr || (reinterpret_cast<uintptr_t>(q) & 15u) != 0) return fail(VS_ERR_INVALID_ARG);
      h->gain2.push_back(weights->norm2_w ? static_cast<const bf16*>(weights->norm2_w[l]) : nullptr);
      if (encode_2d(h, &h->tm_wo[l], ptrs[0], (uint64_t)D.d, (uint64_t)D.d, GEMM_BLOCK_M) != VS_OK ||
          encode_2d(h, &h->tm_gate[l], ptrs[1], (uint64_t)D.d, (uint64_t)D.d_ff, GEMM_BLOCK_M / 2) != VS_OK ||
          encode_2d(h, &h->tm_up[l], ptrs[2], (uint64_t)D.d, (uint64_t)D.d_ff, GEMM_BLOCK_M / 2) != VS_OK ||
          encode_2d(h, &h->tm_down[l], ptrs[3], (uint64_t)D.d_ff, (uint64_t)D.d, GEMM_BLOCK_M) != VS_OK)
        return fail(VS_ERR_CUDA);
    }
  }
  if (D.vocab > 0) {
    if (weights->w_lm == nullptr || (reinterpret_cast<uintptr_t>(weights->w_lm) & 15u) != 0) return fail(VS_ERR_INVALID_ARG);
    h->gain_f = static_cast<const bf16*>(weights->norm_f_w);
    if (encode_2d(h, &h->tm_lm, weights->w_lm, (uint64_t)D.d, (uint64_t)D.vocab, GEMM_BLOCK_M) != VS_OK) return fail(VS_ERR_CUDA);
  }
  if (qkv_gemm_init() != cudaSuccess || qkv_gemv_init() != cudaSuccess || prefill_attention_tc_init() != cudaSuccess) return fail(VS_ERR_CUDA);
  for (int sp = 2; sp <= ATTN_MAX_SPLIT; ++sp) h->attn_clusters[sp] = prefill_attention_max_clusters(D.D, sp);
  // clear the whole workspace, then write the non-zero initial metadata
  if (cudaMemset(h->ws, 0, lo.total) != cudaSuccess) return fail(VS_ERR_CUDA);
  if (cudaMemset(h->ws + lo.slot_frame, 0xFF, (size_t)D.S * D.slots * 4) != cudaSuccess) return fail(VS_ERR_CUDA);
  std::vector<StreamMeta> metas(D.S);
  for (auto& m : metas) { std::memset(&m, 0, sizeof(m)); m.victim_logical = -1; m.last_victim_frame = -1; }
  if (cudaMemcpy(h->ws + lo.meta, metas.data(), metas.size() * sizeof(StreamMeta), cudaMemcpyHostToDevice) != cudaSuccess)
    return fail(VS_ERR_CUDA);
  std::vector<double> inv(D.D / 2);
  for (int k = 0; k < D.D / 2; ++k) inv[k] = std::pow((double)D.rope_theta, -2.0 * (double)k / (double)D.D);
  if (cudaMemcpy(h->ws + lo.inv_freq, inv.data(), inv.size() * 8, cudaMemcpyHostToDevice) != cudaSuccess)
    return fail(VS_ERR_CUDA);
#ifdef VS_DEBUG_BOUNDS
  {
    DebugTable t;
    std::memset(&t, 0, sizeof(t));
    for (int r = 0; r < DR_COUNT; ++r) {
      t.begin[r] = reinterpret_cast<unsigned long long>(h->ws + lo.region_begin[r]);
      t.end[r] = reinterpret_cast<unsigned long long>(h->ws + lo.region_end[r]);
      if (lo.region_end[r] > lo.region_begin[r] &&
          cudaMemset(h->ws + align_up(lo.region_end[r], 256), kGuardByte, kGuardBytes) != cudaSuccess) return fail(VS_ERR_CUDA);
    }
    t.bad_region = -1;
    if (cudaMemcpy(h->ws + lo.dbg_table, &t, sizeof(t), cudaMemcpyHostToDevice) != cudaSuccess) return fail(VS_ERR_CUDA);
  }
#endif
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(VS_ERR_CUDA);
  *out = h;
  return VS_OK;
}

int vs_destroy_stream(vs_stream* h) {
  if (h == nullptr) return VS_ERR_INVALID_ARG;
  for (cudaEvent_t e : h->prof_ev) cudaEventDestroy(e);
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  if (h->ev_join) cudaEventDestroy(h->ev_join);
  if (h->side_stream) cudaStreamDestroy(h->side_stream);
  delete h;
  return VS_OK;
}

int vs_frame_prefill(vs_stream* h, const int32_t* stream_ids, int32_t n_active, const void* hidden, int32_t N,
                     const void* carrier_override, void* out, void* cuda_stream) {
  int rc = check_ids(h, stream_ids, n_active);
  if (rc != VS_OK) return rc;
  if (hidden == nullptr || N < 1) return VS_ERR_INVALID_ARG;
  const Dims& D = h->dm;
  const Layout& lo = h->lo;
  if (N > D.maxN) return VS_ERR_CAPACITY;
  for (int i = 0; i < n_active; ++i)
    if (h->hs[stream_ids[i]].text_len != 0) return VS_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VS_CK(cudaSetDevice(h->device));

  BatchParams bp;
  VS_BP_INIT(h, bp);
  bp.n_active = n_active;
  bp.rows_per_stream = N + 1;
  VS_TRACE_NEXT(h, bp);
  bool any_full = false;
  for (int i = 0; i < n_active; ++i) {
    const HostStream& s = h->hs[stream_ids[i]];
    bp.stream_id[i] = stream_ids[i];
    bp.count[i] = (int32_t)(s.frames_seen < D.M ? s.frames_seen : D.M);
    bp.prefix_len[i] = (int32_t)s.prefix_len;
    bp.text_len[i] = 0;
    bp.pos_base[i] = s.next_pos;
    bp.frame_id[i] = s.frames_seen;
    if (D.M > 0 && bp.count[i] == D.M) any_full = true;
  }
  const int rows = n_active * (N + 1);
  StreamMeta* meta = h->at<StreamMeta>(lo.meta);

  BankUpdateArgs ba;
  ba.emb = h->at<bf16>(lo.emb); ba.meta = meta; ba.step_slot = h->at<int32_t>(lo.step_slot);
  ba.order = h->at<int32_t>(lo.order); ba.slot_frame = h->at<int32_t>(lo.slot_frame);
  ba.slot_pos = h->at<int64_t>(lo.slot_pos); ba.evict_log = h->at<int32_t>(lo.evict_log);
  ba.scores = h->at<double>(lo.scores);
  ba.d = D.d; ba.slots = D.slots; ba.M = D.M; ba.policy = D.evict_policy; ba.log_cap = D.log_cap;
  ba.incoming_emb = nullptr; ba.record_slot = nullptr; ba.record_victim = nullptr; ba.chunk_first_frame = 0; ba.chunk_l1 = 0;
  ba.pre_scores = nullptr; ba.pre_stride = 0;

  PoolArgs pa;
  pa.hidden = static_cast<const bf16*>(hidden);
  pa.carrier_override = static_cast<const bf16*>(carrier_override);
  pa.x = h->at<bf16>(lo.hbuf[0]);
  pa.emb = h->at<bf16>(lo.emb);
  pa.meta = meta;
  pa.step_slot = h->at<int32_t>(lo.step_slot);
  pa.emb_stage = nullptr;
  pa.inv_freq = h->at<double>(lo.inv_freq);
  pa.rope = h->at<float2>(lo.rope);
  pa.N = N; pa.d = D.d; pa.D = D.D; pa.slots = D.slots; pa.M = D.M; pa.agg_mode = D.agg_mode;
  VS_LAUNCH(h, st, KC_POOL, launch_pool(pa, bp, st));
  if (ensure_step_maps(h, rows) != VS_OK) return VS_ERR_CUDA;

  void* out_final = out ? out : h->at<void>(lo.obuf);
  int cur = 0;
  for (int l = 0; l < D.L; ++l) {
    if (l > 0) VS_TRACE_NEXT(h, bp);
    const bf16* h_in = h->at<bf16>(lo.hbuf[cur]);
    const bf16* src = h_in;
    if (D.use_rmsnorm) {
      // layer 0: a launch of its own; deeper layers: the attention kernel that stored h_in left the statistics
      if (l == 0) VS_LAUNCH(h, st, KC_RMSNORM, launch_rms_stats(h_in, h->gain[l], h->at<bf16>(lo.xn), h->at<float>(lo.row_ss),
                                                                D.ss_parts, rows, D.d, st));
      if (h->gain[l] != nullptr) src = h->at<bf16>(lo.xn);
    }
    ProjectionOut fa;
    fa.bias = h->bias[l];
    fa.row_ss = D.use_rmsnorm ? h->at<float>(lo.row_ss) : nullptr; fa.ss_parts = D.ss_parts; fa.norm_eps = D.rms_eps;
    fa.norm_inline = 0; fa.norm_gain = nullptr;
    fa.rope = h->at<float2>(lo.rope);
    fa.inv_freq = h->at<double>(lo.inv_freq);
    fa.q = h->at<bf16>(lo.q); fa.q_lo = h->at<bf16>(lo.q_lo); fa.kf = h->at<bf16>(lo.kf); fa.vf = h->at<bf16>(lo.vf);
    fa.q_tiled = h->at<bf16>(lo.q_tiled);
    fa.bank_k = h->at<bf16>(lo.bank_k) + (size_t)l * layer_stride_bank(D);
    fa.bank_v = h->at<bf16>(lo.bank_v) + (size_t)l * layer_stride_bank(D);
    fa.text_k = nullptr; fa.text_v = nullptr;
    fa.free_slot = h->at<int32_t>(lo.step_slot); fa.free_slot_stride = 1;
    fa.Hq = D.Hq; fa.Hkv = D.Hkv; fa.D = D.D; fa.slots = D.slots; fa.text_cap = 0; fa.mode = 0; fa.M = D.M;
    rc = run_projection(h, l, src, rows, fa, bp, st);
    if (rc != VS_OK) return rc;

    AttnArgs aa;
    std::memset(&aa, 0, sizeof(aa));
    aa.q = fa.q; aa.q_lo = fa.q_lo; aa.q_tiled = fa.q_tiled;
    seg_stored(aa.seg[0], h->tm_prefix_k, h->tm_prefix_v, 0, l, D);
    seg_stored(aa.seg[1], h->tm_bank_k, h->tm_bank_v, 1, l, D);
    seg_step(aa.seg[2], h->tm_step_k, h->tm_step_v, 3, N + 1);
    aa.n_seg = 3;
    const bool last = (l == D.L - 1);
    // a layer whose rows only feed the residual stream stores no output rows
    aa.out = last ? out_final : (D.residual ? nullptr : h->at<void>(lo.obuf));
    aa.out_fp32 = D.out_fp32;
    aa.h_in = D.residual ? h_in : nullptr;
    aa.h_out = D.residual ? h->at<bf16>(lo.hbuf[cur ^ 1]) : nullptr;
    aa.h_out_region = (cur ^ 1) ? DR_HBUF1 : DR_HBUF0;
    if (D.use_rmsnorm && l + 1 < D.L) { aa.ss_out = h->at<float>(lo.row_ss); aa.next_gain = h->gain[l + 1]; aa.xn_out = h->at<bf16>(lo.xn); }
    if (D.d_ff > 0) {
      // full decoder block: the attention rows (bf16) feed the output projection; the residual comes there
      aa.out = h->at<void>(lo.obuf); aa.out_fp32 = 0;
      aa.h_in = nullptr; aa.h_out = nullptr; aa.ss_out = nullptr; aa.next_gain = nullptr; aa.xn_out = nullptr;
    }
    aa.free_slot = h->at<int32_t>(lo.step_slot); aa.free_slot_stride = 1;
    {
      int kl[3] = {0, 0, N + 1};
      for (int i = 0; i < n_active; ++i) {
        const int bl = D.M == 0 ? 0 : (bp.count[i] == D.M ? D.M + 1 : bp.count[i]);
        if (bp.prefix_len[i] + bl > kl[0] + kl[1]) { kl[0] = bp.prefix_len[i]; kl[1] = bl; }
      }
      aa.nsplit = attn_split(h, bp, kl, 3);
    }
    // the bank update (Section 3.3, memory mechanism: evict if full, then append) rides in the last layer's launch
    if (last) { aa.bank = ba; aa.bank_blocks = any_full ? (D.M + 7) / 8 : 1; }
    aa.Hq = D.Hq; aa.Hkv = D.Hkv; aa.D = D.D; aa.slots = D.slots; aa.M = D.M;
    aa.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)D.D));
    VS_LAUNCH(h, st, KC_PREFILL_ATTN, launch_prefill_attention_tc(aa, bp, h->at<int>(lo.status), st));
    if (D.d_ff > 0) {
      // h2 lands in hbuf[0] again: the layer input of every layer is hbuf[0]
      rc = run_block_rest(h, l, rows, h_in, h->at<bf16>(lo.obuf), last ? out_final : nullptr, bp, st);
      if (rc != VS_OK) return rc;
    } else if (D.residual) cur ^= 1;
  }

  for (int i = 0; i < n_active; ++i) {
    HostStream& s = h->hs[stream_ids[i]];
    s.next_pos += N + 1;
    s.frames_seen += 1;
  }
  h->last_stream = st;
  h->last_rows = rows;
  return VS_OK;
}

int vs_frame_prefill_chunk(vs_stream* h, int32_t stream_id, const void* hidden, int32_t F, int32_t N, void* out,
                           void* cuda_stream) {
  int rc = check_ids(h, &stream_id, 1);
  if (rc != VS_OK) return rc;
  if (hidden == nullptr || N < 1 || F < 1) return VS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(hidden) & 15u) != 0) return VS_ERR_INVALID_ARG;
  const Dims& D = h->dm;
  const Layout& lo = h->lo;
  if (N > D.maxN || F > D.maxChunk) return VS_ERR_CAPACITY;
  HostStream& hs = h->hs[stream_id];
  if (hs.text_len != 0) return VS_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VS_CK(cudaSetDevice(h->device));

  // the F frames as F batch entries of the same stream, each with the bank count and the
  // positions it would find as a step of its own
  BatchParams bp;
  VS_BP_INIT(h, bp);
  bp.n_active = F;
  bp.rows_per_stream = N + 1;
  for (int j = 0; j < F; ++j) {
    const int64_t seen = hs.frames_seen + j;
    bp.stream_id[j] = stream_id;
    bp.count[j] = (int32_t)(seen < D.M ? seen : D.M);
    bp.prefix_len[j] = (int32_t)hs.prefix_len;
    bp.text_len[j] = 0;
    bp.pos_base[j] = hs.next_pos + (int64_t)j * (N + 1);
    bp.frame_id[j] = seen;
  }
  auto one_frame = [&](int j) {
    BatchParams b1;
    VS_BP_INIT(h, b1);
    b1.n_active = 1; b1.rows_per_stream = N + 1;
    b1.stream_id[0] = bp.stream_id[j]; b1.count[0] = bp.count[j]; b1.prefix_len[0] = bp.prefix_len[j];
    b1.pos_base[0] = bp.pos_base[j]; b1.frame_id[0] = bp.frame_id[j];
    return b1;
  };
  const int rows = F * (N + 1);
  StreamMeta* meta = h->at<StreamMeta>(lo.meta);
  int32_t* chunk_slot = h->at<int32_t>(lo.chunk_slot);
  int32_t* chunk_victim = h->at<int32_t>(lo.chunk_victim);
  // the bank as every frame of the chunk finds it on its key axis: the carriers that were there
  // before the chunk (all M + 1 slots once the bank is full)
  const int count0 = bp.count[0];
  const int l1 = (D.M > 0 && count0 == D.M) ? D.M + 1 : count0;
  // the attention launch's mask of hidden bank keys; refused on the bank's capacity, not on its fill, so that a
  // stream does not run into the limit only once its bank is full
  if ((D.M > 0 ? D.M + 1 : 0) + F > ATTN_EXCL_BITS) return VS_ERR_CAPACITY;

  // 1. carriers of all frames (Section 3.3: C = mean of the frame's tokens), parked until they have a slot
  PoolArgs pa;
  pa.hidden = static_cast<const bf16*>(hidden);
  pa.carrier_override = nullptr;
  pa.x = h->at<bf16>(lo.hbuf[0]);
  pa.emb = h->at<bf16>(lo.emb);
  pa.meta = meta;
  pa.step_slot = h->at<int32_t>(lo.step_slot);
  pa.emb_stage = h->at<bf16>(lo.emb_stage);
  pa.inv_freq = h->at<double>(lo.inv_freq);
  pa.rope = h->at<float2>(lo.rope);
  pa.N = N; pa.d = D.d; pa.D = D.D; pa.slots = D.slots; pa.M = D.M; pa.agg_mode = D.agg_mode;
  VS_LAUNCH(h, st, KC_POOL, launch_pool(pa, bp, st));

  // 2. the bank updates, frame by frame (Section 3.3, memory mechanism): they read embeddings only,
  //    so they can all run before any attention; each records the slot its carrier took.  The
  //    projection needs nothing of theirs, so they run beside it on a stream of the handle's own,
  //    forked here and joined ahead of the first attention launch.
  if (h->side_stream == nullptr) {
    // highest priority: its few small CTAs must not queue behind the projection's second wave
    int prio_low = 0, prio_high = 0;
    VS_CK(cudaDeviceGetStreamPriorityRange(&prio_low, &prio_high));
    VS_CK(cudaStreamCreateWithPriority(&h->side_stream, cudaStreamNonBlocking, prio_high));
    VS_CK(cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
    VS_CK(cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
  }
  const bool beside = !h->prof_on;           // the per-launch timing pass keeps everything on one stream
  cudaStream_t bst = beside ? h->side_stream : st;
  if (beside) {
    VS_CK(cudaEventRecord(h->ev_fork, st));
    VS_CK(cudaStreamWaitEvent(h->side_stream, h->ev_fork, 0));
  }
  {
    BankUpdateArgs ba;
    ba.emb = h->at<bf16>(lo.emb); ba.meta = meta; ba.step_slot = h->at<int32_t>(lo.step_slot);
    ba.order = h->at<int32_t>(lo.order); ba.slot_frame = h->at<int32_t>(lo.slot_frame);
    ba.slot_pos = h->at<int64_t>(lo.slot_pos); ba.evict_log = h->at<int32_t>(lo.evict_log);
    ba.scores = h->at<double>(lo.scores);
    ba.d = D.d; ba.slots = D.slots; ba.M = D.M; ba.policy = D.evict_policy; ba.log_cap = D.log_cap;
    ba.chunk_first_frame = bp.frame_id[0];
    ba.chunk_l1 = l1;
    ba.pre_scores = nullptr; ba.pre_stride = 0;
    const bool any_full = D.M > 0 && bp.count[F - 1] == D.M;
    if (D.evict_policy != 1 && F > 1) {
      // the updates score against their incoming carrier only (or not at all): every cosine of the
      // chunk in one launch, then all F updates in turn by one block
      ba.incoming_emb = h->at<bf16>(lo.emb_stage);
      ba.record_slot = chunk_slot;
      ba.record_victim = chunk_victim;
      ba.pre_scores = h->at<double>(lo.chunk_scores);
      ba.pre_stride = D.slots + D.maxChunk;
      if (any_full && D.evict_policy == 0)
        VS_LAUNCH(h, bst, KC_EVICT, launch_chunk_scores(ba, bp, h->at<bf16>(lo.emb_stage), h->at<double>(lo.chunk_scores), bst));
      VS_LAUNCH(h, bst, KC_COMMIT, launch_chunk_plan(ba, bp, bst));
    } else {
      // adjacent-pair scoring: which pairs are adjacent depends on the updates before, one launch per frame
      for (int j = 0; j < F; ++j) {
        ba.incoming_emb = h->at<bf16>(lo.emb_stage) + (size_t)j * D.d;
        ba.record_slot = chunk_slot + j;
        ba.record_victim = chunk_victim + j;
        const BatchParams b1 = one_frame(j);
        VS_LAUNCH(h, bst, KC_COMMIT, launch_bank_update(ba, b1, D.M > 0 && b1.count[0] == D.M, bst));
      }
    }
  }
  if (beside) VS_CK(cudaEventRecord(h->ev_join, h->side_stream));

  if (ensure_step_maps(h, rows) != VS_OK) return VS_ERR_CUDA;
  // the carrier rows of the chunk's frames (row N of every frame of the step's K/V) as a segment of their own
  CUtensorMap tm_carr_k, tm_carr_v;
  {
    const uint64_t rs = (uint64_t)(N + 1) * D.Hkv * D.D * 2, zs = (uint64_t)D.D * 2;
    if (encode_kv(h, &tm_carr_k, h->at<bf16>(lo.kf) + (size_t)N * D.Hkv * D.D, D.D, F, rs, D.Hkv, zs) != VS_OK ||
        encode_kv(h, &tm_carr_v, h->at<bf16>(lo.vf) + (size_t)N * D.Hkv * D.D, D.D, F, rs, D.Hkv, zs) != VS_OK)
      return VS_ERR_CUDA;
  }
  // 3. layer by layer: one projection over all F * (N + 1) rows, one attention launch over all
  //    frames, then the K/V rows of the chunk's surviving carriers go into their bank slots
  char* out_bytes = static_cast<char*>(out ? out : h->at<void>(lo.obuf));
  int cur = 0;
  for (int l = 0; l < D.L; ++l) {
    const bf16* h_in = h->at<bf16>(lo.hbuf[cur]);
    const bf16* src = h_in;
    if (D.use_rmsnorm) {
      // layer 0: a launch of its own; deeper layers: the attention kernel that stored h_in left the statistics
      if (l == 0) VS_LAUNCH(h, st, KC_RMSNORM, launch_rms_stats(h_in, h->gain[l], h->at<bf16>(lo.xn), h->at<float>(lo.row_ss),
                                                                D.ss_parts, rows, D.d, st));
      if (h->gain[l] != nullptr) src = h->at<bf16>(lo.xn);
    }
    ProjectionOut fa;
    std::memset(&fa, 0, sizeof(fa));
    fa.bias = h->bias[l];
    fa.row_ss = D.use_rmsnorm ? h->at<float>(lo.row_ss) : nullptr; fa.ss_parts = D.ss_parts; fa.norm_eps = D.rms_eps;
    fa.rope = h->at<float2>(lo.rope);
    fa.inv_freq = h->at<double>(lo.inv_freq);
    fa.q = h->at<bf16>(lo.q); fa.q_lo = h->at<bf16>(lo.q_lo); fa.kf = h->at<bf16>(lo.kf); fa.vf = h->at<bf16>(lo.vf);
    fa.q_tiled = h->at<bf16>(lo.q_tiled);
    fa.bank_k = h->at<bf16>(lo.bank_k) + (size_t)l * layer_stride_bank(D);
    fa.bank_v = h->at<bf16>(lo.bank_v) + (size_t)l * layer_stride_bank(D);
    fa.free_slot = chunk_slot; fa.free_slot_stride = 0;
    fa.Hq = D.Hq; fa.Hkv = D.Hkv; fa.D = D.D; fa.slots = D.slots; fa.text_cap = 0; fa.mode = 3; fa.M = D.M;
    rc = run_projection(h, l, src, rows, fa, bp, st);
    if (rc != VS_OK) return rc;

    const bool last = (l == D.L - 1);
    char* layer_out = last ? out_bytes : static_cast<char*>(h->at<void>(lo.obuf));
    if (l == 0 && beside) VS_CK(cudaStreamWaitEvent(st, h->ev_join, 0));
    {
      // every frame is a batch entry; frame b sees the bank of before the chunk minus what the
      // updates of frames 0 .. b-1 evicted, plus the carriers of those frames (from the step's K/V)
      AttnArgs aa;
      std::memset(&aa, 0, sizeof(aa));
      aa.q = fa.q; aa.q_lo = fa.q_lo; aa.q_tiled = fa.q_tiled;
      seg_stored(aa.seg[0], h->tm_prefix_k, h->tm_prefix_v, 0, l, D);
      seg_stored(aa.seg[1], h->tm_bank_k, h->tm_bank_v, 1, l, D);
      seg_step(aa.seg[2], tm_carr_k, tm_carr_v, 4, 0);
      seg_step(aa.seg[3], h->tm_step_k, h->tm_step_v, 3, N + 1);
      aa.n_seg = 4;
      aa.out = (last || !D.residual) ? layer_out : nullptr;
      aa.out_fp32 = D.out_fp32;
      aa.h_in = D.residual ? h_in : nullptr;
      aa.h_out = D.residual ? h->at<bf16>(lo.hbuf[cur ^ 1]) : nullptr;
    aa.h_out_region = (cur ^ 1) ? DR_HBUF1 : DR_HBUF0;
    if (D.use_rmsnorm && l + 1 < D.L) { aa.ss_out = h->at<float>(lo.row_ss); aa.next_gain = h->gain[l + 1]; aa.xn_out = h->at<bf16>(lo.xn); }
      if (D.d_ff > 0) {
        // full decoder block: the attention rows (bf16) feed the output projection; the residual comes there
        aa.out = h->at<void>(lo.obuf); aa.out_fp32 = 0;
        aa.h_in = nullptr; aa.h_out = nullptr; aa.ss_out = nullptr; aa.next_gain = nullptr; aa.xn_out = nullptr;
      }
      aa.free_slot = chunk_slot; aa.free_slot_stride = 0;
      aa.chunk_mode = 1; aa.chunk_count0 = count0; aa.chunk_victim = chunk_victim;
      {
        const int kl[4] = {bp.prefix_len[0], D.M == 0 ? 0 : l1, D.M == 0 ? 0 : F - 1, N + 1};
        aa.nsplit = attn_split(h, bp, kl, 4);
      }
      aa.Hq = D.Hq; aa.Hkv = D.Hkv; aa.D = D.D; aa.slots = D.slots; aa.M = D.M;
      aa.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)D.D));
      VS_LAUNCH(h, st, KC_PREFILL_ATTN, launch_prefill_attention_tc(aa, bp, h->at<int>(lo.status), st));
      if (D.M > 0) {
        ChunkKvCommitArgs ca;
        ca.kf = fa.kf; ca.vf = fa.vf; ca.bank_k = fa.bank_k; ca.bank_v = fa.bank_v;
        ca.chunk_slot = chunk_slot; ca.chunk_victim = chunk_victim;
        ca.F = F; ca.N = N; ca.Hkv = D.Hkv; ca.D = D.D; ca.slots = D.slots; ca.sid = stream_id; ca.l1 = l1;
        VS_LAUNCH(h, st, KC_OTHER, launch_chunk_kv_commit(ca, st));
      }
    }
    if (D.d_ff > 0) {
      // h2 lands in hbuf[0] again: the layer input of every layer is hbuf[0]
      rc = run_block_rest(h, l, rows, h_in, h->at<bf16>(lo.obuf), (last && out != nullptr) ? out : nullptr, bp, st);
      if (rc != VS_OK) return rc;
    } else if (D.residual) cur ^= 1;
  }

  hs.next_pos += (int64_t)F * (N + 1);
  hs.frames_seen += F;
  h->last_stream = st;
  h->last_rows = rows;
  return VS_OK;
}

int vs_bank_forward(vs_stream* h, int32_t stream_id, void* out, void* cuda_stream) {
  int rc = check_ids(h, &stream_id, 1);
  if (rc != VS_OK) return rc;
  const Dims& D = h->dm;
  const Layout& lo = h->lo;
  if ((D.d & 7) != 0) return VS_ERR_UNSUPPORTED;
  const HostStream& hs = h->hs[stream_id];
  const int count = (int)(hs.frames_seen < D.M ? hs.frames_seen : D.M);
  if (count == 0) return VS_OK;
  if (out == nullptr) return VS_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VS_CK(cudaSetDevice(h->device));

  // one text-like step of `count` rows right after the prompt; nothing is kept
  BatchParams bp;
  VS_BP_INIT(h, bp);
  bp.n_active = 1;
  bp.rows_per_stream = count;
  bp.stream_id[0] = stream_id;
  bp.prefix_len[0] = (int32_t)hs.prefix_len;
  bp.pos_base[0] = hs.prefix_len;
  const int rows = count;
  VS_LAUNCH(h, st, KC_OTHER, launch_gather_carriers(h->at<bf16>(lo.emb), h->at<int32_t>(lo.order), h->at<bf16>(lo.hbuf[0]),
                                                    stream_id, D.slots, D.d, count, st));
  RopeArgs ra;
  ra.inv_freq = h->at<double>(lo.inv_freq); ra.rope = h->at<float2>(lo.rope); ra.D = D.D;
  VS_LAUNCH(h, st, KC_ROPE, launch_rope_table(ra, bp, st));
  if (ensure_step_maps(h, rows) != VS_OK) return VS_ERR_CUDA;

  int cur = 0;
  for (int l = 0; l < D.L; ++l) {
    const bf16* h_in = h->at<bf16>(lo.hbuf[cur]);
    const bf16* src = h_in;
    if (D.use_rmsnorm) {
      // layer 0: a launch of its own; deeper layers: the attention kernel that stored h_in left the statistics
      if (l == 0) VS_LAUNCH(h, st, KC_RMSNORM, launch_rms_stats(h_in, h->gain[l], h->at<bf16>(lo.xn), h->at<float>(lo.row_ss),
                                                                D.ss_parts, rows, D.d, st));
      if (h->gain[l] != nullptr) src = h->at<bf16>(lo.xn);
    }
    ProjectionOut fa;
    std::memset(&fa, 0, sizeof(fa));
    fa.bias = h->bias[l];
    fa.row_ss = D.use_rmsnorm ? h->at<float>(lo.row_ss) : nullptr; fa.ss_parts = D.ss_parts; fa.norm_eps = D.rms_eps;
    fa.rope = h->at<float2>(lo.rope);
    fa.inv_freq = h->at<double>(lo.inv_freq);
    fa.q = h->at<bf16>(lo.q); fa.q_lo = h->at<bf16>(lo.q_lo); fa.kf = h->at<bf16>(lo.kf); fa.vf = h->at<bf16>(lo.vf);
    fa.q_tiled = h->at<bf16>(lo.q_tiled);
    fa.free_slot = h->at<int32_t>(lo.step_slot); fa.free_slot_stride = 0;
    fa.Hq = D.Hq; fa.Hkv = D.Hkv; fa.D = D.D; fa.slots = D.slots; fa.text_cap = 0; fa.mode = 3; fa.M = D.M;
    rc = run_projection(h, l, src, rows, fa, bp, st);
    if (rc != VS_OK) return rc;

    AttnArgs aa;
    std::memset(&aa, 0, sizeof(aa));
    aa.q = fa.q; aa.q_lo = fa.q_lo; aa.q_tiled = fa.q_tiled;
    seg_stored(aa.seg[0], h->tm_prefix_k, h->tm_prefix_v, 0, l, D);
    seg_step(aa.seg[1], h->tm_step_k, h->tm_step_v, 3, rows);
    aa.n_seg = 2;
    aa.out = (l == D.L - 1) ? out : (D.residual ? nullptr : h->at<void>(lo.obuf));
    aa.out_fp32 = D.out_fp32;
    aa.h_in = D.residual ? h_in : nullptr;
    aa.h_out = D.residual ? h->at<bf16>(lo.hbuf[cur ^ 1]) : nullptr;
    aa.h_out_region = (cur ^ 1) ? DR_HBUF1 : DR_HBUF0;
    if (D.use_rmsnorm && l + 1 < D.L) { aa.ss_out = h->at<float>(lo.row_ss); aa.next_gain = h->gain[l + 1]; aa.xn_out = h->at<bf16>(lo.xn); }
    if (D.d_ff > 0) {
      aa.out = h->at<void>(lo.obuf); aa.out_fp32 = 0;
      aa.h_in = nullptr; aa.h_out = nullptr; aa.ss_out = nullptr; aa.next_gain = nullptr; aa.xn_out = nullptr;
    }
    aa.free_slot = h->at<int32_t>(lo.step_slot); aa.free_slot_stride = 0;
    aa.Hq = D.Hq; aa.Hkv = D.Hkv; aa.D = D.D; aa.slots = D.slots; aa.M = 0;      // no bank segment on this key axis
    {
      const int kl[2] = {bp.prefix_len[0], rows};
      aa.nsplit = attn_split(h, bp, kl, 2);
    }
    aa.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)D.D));
    VS_LAUNCH(h, st, KC_PREFILL_ATTN, launch_prefill_attention_tc(aa, bp, h->at<int>(lo.status), st));
    if (D.d_ff > 0) {
      rc = run_block_rest(h, l, rows, h_in, h->at<bf16>(lo.obuf), (l == D.L - 1) ? out : nullptr, bp, st);
      if (rc != VS_OK) return rc;
    } else if (D.residual) cur ^= 1;
  }
  h->last_stream = st;
  h->last_rows = rows;
  return VS_OK;
}

int vs_decode_step(vs_stream* h, const int32_t* stream_ids, int32_t n_active, const void* hidden, int32_t T,
                   void* out, void* cuda_stream) {
  int rc = check_ids(h, stream_ids, n_active);
  if (rc != VS_OK) return rc;
  if (hidden == nullptr || out == nullptr || T < 1) return VS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(hidden) & 15u) != 0) return VS_ERR_INVALID_ARG;
  const Dims& D = h->dm;
  const Layout& lo = h->lo;
  if (T > D.maxStepT) return VS_ERR_CAPACITY;
  const bool to_prefix = h->hs[stream_ids[0]].frames_seen == 0;
  for (int i = 0; i < n_active; ++i) {
    const HostStream& s = h->hs[stream_ids[i]];
    if ((s.frames_seen == 0) != to_prefix) return VS_ERR_STATE;
    if (to_prefix ? (s.prefix_len + T > D.capP) : (s.text_len + T > D.capT)) return VS_ERR_CAPACITY;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VS_CK(cudaSetDevice(h->device));

  BatchParams bp;
  VS_BP_INIT(h, bp);
  bp.n_active = n_active;
  bp.rows_per_stream = T;
  VS_TRACE_NEXT(h, bp);
  int max_keys = 0;
  for (int i = 0; i < n_active; ++i) {
    const HostStream& s = h->hs[stream_ids[i]];
    bp.stream_id[i] = stream_ids[i];
    bp.count[i] = (int32_t)(s.frames_seen < D.M ? s.frames_seen : D.M);
    bp.prefix_len[i] = (int32_t)s.prefix_len;
    bp.text_len[i] = (int32_t)s.text_len;
    bp.pos_base[i] = to_prefix ? s.next_pos : s.next_pos + s.text_len;
    bp.frame_id[i] = s.frames_seen;
    const int keys = (int)s.prefix_len + bp.count[i] + 1 + (int)s.text_len + T;
    if (keys > max_keys) max_keys = keys;
  }
  const int rows = n_active * T;
  StreamMeta* meta = h->at<StreamMeta>(lo.meta);

  // a step of up to 16 rows needs no table: the projection works the rotation out itself
  const bool rope_inline = rows <= 16;
  if (!rope_inline) {
    RopeArgs ra;
    ra.inv_freq = h->at<double>(lo.inv_freq); ra.rope = h->at<float2>(lo.rope); ra.D = D.D;
    VS_LAUNCH(h, st, KC_ROPE, launch_rope_table(ra, bp, st));
  }

  if (T > 1 && ensure_step_maps(h, rows) != VS_OK) return VS_ERR_CUDA;
  const bf16* h_in = static_cast<const bf16*>(hidden);
  int next_buf = 0;
  for (int l = 0; l < D.L; ++l) {
    if (l > 0) VS_TRACE_NEXT(h, bp);
    const bf16* src = h_in;
    // a step the matrix-vector kernel takes needs no statistics launch: that kernel normalises itself
    ProjectionOut probe;
    std::memset(&probe, 0, sizeof(probe));
    probe.mode = 1; probe.D = D.D;
    const bool by_gemv = rope_inline && qkv_gemv_supported(probe, rows, D.d) && (reinterpret_cast<uintptr_t>(h_in) & 15u) == 0;
    if (D.use_rmsnorm && !by_gemv) {
      // layer 0, and every layer of a single-token step (its attention kernel leaves no statistics): a launch of
      // its own; else the tensor-core attention that stored h_in left them
      if (l == 0 || (T == 1 && D.d_ff == 0)) VS_LAUNCH(h, st, KC_RMSNORM, launch_rms_stats(h_in, h->gain[l], h->at<bf16>(lo.xn), h->at<float>(lo.row_ss),
                                                                          D.ss_parts, rows, D.d, st));
      if (h->gain[l] != nullptr) src = h->at<bf16>(lo.xn);
    }
    bf16* pk = h->at<bf16>(lo.prefix_k) + (size_t)l * layer_stride_prefix(D);
    bf16* pv = h->at<bf16>(lo.prefix_v) + (size_t)l * layer_stride_prefix(D);
    bf16* tk = h->at<bf16>(lo.tail_k) + (size_t)l * layer_stride_tail(D);
    bf16* tv = h->at<bf16>(lo.tail_v) + (size_t)l * layer_stride_tail(D);
    bf16* bk = h->at<bf16>(lo.bank_k) + (size_t)l * layer_stride_bank(D);
    bf16* bv = h->at<bf16>(lo.bank_v) + (size_t)l * layer_stride_bank(D);

    ProjectionOut fa;
    fa.bias = h->bias[l];
    fa.row_ss = (D.use_rmsnorm && !by_gemv) ? h->at<float>(lo.row_ss) : nullptr; fa.ss_parts = D.ss_parts;
    fa.norm_inline = (D.use_rmsnorm && by_gemv) ? 1 : 0; fa.norm_gain = h->gain[l]; fa.norm_eps = D.rms_eps;
    fa.rope = rope_inline ? nullptr : h->at<float2>(lo.rope);
    fa.inv_freq = h->at<double>(lo.inv_freq);
    fa.q = h->at<bf16>(lo.q); fa.q_lo = h->at<bf16>(lo.q_lo); fa.kf = h->at<bf16>(lo.kf); fa.vf = h->at<bf16>(lo.vf);
    // a step of several rows goes to the tensor-core attention: its GEMM leaves the query in that kernel's layout
    fa.q_tiled = (T > 1 && !by_gemv) ? h->at<bf16>(lo.q_tiled) : nullptr;
    fa.bank_k = bk; fa.bank_v = bv;
    fa.text_k = to_prefix ? pk : tk; fa.text_v = to_prefix ? pv : tv;
    fa.free_slot = &meta->free_slot; fa.free_slot_stride = (int)(sizeof(StreamMeta) / sizeof(int32_t));
    fa.Hq = D.Hq; fa.Hkv = D.Hkv; fa.D = D.D; fa.slots = D.slots;
    fa.text_cap = to_prefix ? D.maxP : D.maxT; fa.mode = to_prefix ? 1 : 2; fa.M = D.M;
    rc = run_projection(h, l, src, rows, fa, bp, st);
    if (rc != VS_OK) return rc;

    bf16* h_out = D.residual ? h->at<bf16>(lo.hbuf[next_buf]) : nullptr;
    const int h_out_region = next_buf ? DR_HBUF1 : DR_HBUF0;
    const float scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)D.D));
    if (T == 1) {
      DecodeArgs da;
      da.q = fa.q; da.q_lo = fa.q_lo;
      da.prefix_k = pk; da.prefix_v = pv; da.bank_k = bk; da.bank_v = bv; da.tail_k = tk; da.tail_v = tv;
      da.out = (l == D.L - 1) ? out : h->at<void>(lo.obuf);
      da.out_fp32 = D.out_fp32;
      da.h_in = D.residual ? h_in : nullptr; da.h_out = h_out; da.h_out_region = h_out_region;
      if (D.d_ff > 0) { da.out = h->at<void>(lo.obuf); da.out_fp32 = 0; da.h_in = nullptr; da.h_out = nullptr; }
      da.meta = meta;
      da.Hq = D.Hq; da.Hkv = D.Hkv; da.D = D.D; da.slots = D.slots; da.M = D.M; da.maxP = D.maxP; da.maxT = D.maxT;
      // short contexts: one CTA per (stream, query head) writes the row directly; longer ones are
      // split over a cluster of 2, 4 or 8 CTAs (a CTA then walks about 64 to 128 keys), fewer
      // when many streams already fill the GPU
      int ns = (max_keys <= 96) ? 1 : (max_keys <= 192 ? 2 : (max_keys <= 448 ? 4 : 8));
      while (ns > 1 && (long long)ns * D.Hq * n_active > 4LL * h->n_sms) ns >>= 1;
      da.nsplit = ns;
      da.to_prefix = to_prefix ? 1 : 0;
      da.scale_log2e = scale_log2e;
      VS_LAUNCH(h, st, KC_DECODE_ATTN, launch_decode_attention(da, bp, st));
    } else {
      AttnArgs aa;
      std::memset(&aa, 0, sizeof(aa));
      aa.q = fa.q; aa.q_lo = fa.q_lo; aa.q_tiled = fa.q_tiled;
      int ns = 0;
      seg_stored(aa.seg[ns++], h->tm_prefix_k, h->tm_prefix_v, 0, l, D);
      if (!to_prefix) {
        seg_stored(aa.seg[ns++], h->tm_bank_k, h->tm_bank_v, 1, l, D);
        seg_stored(aa.seg[ns++], h->tm_tail_k, h->tm_tail_v, 2, l, D);
      }
      seg_step(aa.seg[ns++], h->tm_step_k, h->tm_step_v, 3, T);
      aa.n_seg = ns;
      {
        int kl[4] = {0, 0, 0, T};
        for (int i = 0; i < n_active; ++i) {
          const int bl = (to_prefix || D.M == 0) ? 0 : (bp.count[i] == D.M ? D.M + 1 : bp.count[i]);
          const int tl = to_prefix ? 0 : bp.text_len[i];
          if (bp.prefix_len[i] + bl + tl > kl[0] + kl[1] + kl[2]) { kl[0] = bp.prefix_len[i]; kl[1] = bl; kl[2] = tl; }
        }
        aa.nsplit = attn_split(h, bp, kl, 4);
      }
      aa.out = (l == D.L - 1) ? out : (D.residual ? nullptr : h->at<void>(lo.obuf));
      aa.out_fp32 = D.out_fp32;
      aa.h_in = D.residual ? h_in : nullptr;
      aa.h_out = h_out; aa.h_out_region = h_out_region;
      if (D.use_rmsnorm && l + 1 < D.L && !by_gemv) { aa.ss_out = h->at<float>(lo.row_ss); aa.next_gain = h->gain[l + 1]; aa.xn_out = h->at<bf16>(lo.xn); }
      aa.free_slot = &meta->free_slot; aa.free_slot_stride = (int)(sizeof(StreamMeta) / sizeof(int32_t));
      aa.Hq = D.Hq; aa.Hkv = D.Hkv; aa.D = D.D; aa.slots = D.slots; aa.M = D.M;
      aa.scale_log2e = scale_log2e;
      if (D.d_ff > 0) {
        aa.out = h->at<void>(lo.obuf); aa.out_fp32 = 0;
        aa.h_in = nullptr; aa.h_out = nullptr; aa.ss_out = nullptr; aa.next_gain = nullptr; aa.xn_out = nullptr;
      }
      VS_LAUNCH(h, st, KC_PREFILL_ATTN, launch_prefill_attention_tc(aa, bp, h->at<int>(lo.status), st));
    }
    if (D.d_ff > 0) {
      rc = run_block_rest(h, l, rows, h_in, h->at<bf16>(lo.obuf), (l == D.L - 1) ? out : nullptr, bp, st);
      if (rc != VS_OK) return rc;
      h_in = h->at<bf16>(lo.hbuf[0]);
    } else if (D.residual) { h_in = h_out; next_buf ^= 1; }
  }

  for (int i = 0; i < n_active; ++i) {
    HostStream& s = h->hs[stream_ids[i]];
    if (to_prefix) { s.prefix_len += T; s.next_pos += T; }
    else s.text_len += T;
  }
  h->last_stream = st;
  h->last_rows = rows;
  return VS_OK;
}

int vs_reset_stream(vs_stream* h, const int32_t* stream_ids, int32_t n_active, void* cuda_stream) {
  const int rc = check_ids(h, stream_ids, n_active);
  if (rc != VS_OK) return rc;
  const Dims& D = h->dm;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VS_CK(cudaSetDevice(h->device));
  BatchParams bp;
  VS_BP_INIT(h, bp);
  bp.n_active = n_active;
  for (int i = 0; i < n_active; ++i) bp.stream_id[i] = stream_ids[i];
  VS_LAUNCH(h, st, KC_OTHER, launch_reset(h->at<StreamMeta>(h->lo.meta), h->at<int32_t>(h->lo.slot_frame), D.slots, bp, st));
  for (int i = 0; i < n_active; ++i) h->hs[stream_ids[i]] = HostStream();
  h->last_stream = st;
  return VS_OK;
}

int vs_profile_enable(vs_stream* h, int32_t on, int32_t max_launches) {
  if (h == nullptr || max_launches < 0) return VS_ERR_INVALID_ARG;
  VS_CK(cudaSetDevice(h->device));
  if (on) {
    while (h->prof_ev.size() < (size_t)max_launches * 2) {
      cudaEvent_t e;
      VS_CK(cudaEventCreate(&e));
      h->prof_ev.push_back(e);
    }
    h->prof_class.resize(h->prof_ev.size() / 2);
  }
  h->prof_on = on != 0;
  h->prof_used = 0;
  return VS_OK;
}

int vs_profile_read(vs_stream* h, double* ms, int64_t* timed, int64_t* launches) {
  if (h == nullptr) return VS_ERR_INVALID_ARG;
  VS_CK(cudaSetDevice(h->device));
  VS_CK(cudaStreamSynchronize(h->last_stream));
  for (int k = 0; k < VS_N_KERNEL_CLASSES; ++k) {
    if (ms) ms[k] = 0.0;
    if (timed) timed[k] = 0;
    if (launches) { launches[k] = h->launches[k]; }
    h->launches[k] = 0;
  }
  for (size_t i = 0; i < h->prof_used; ++i) {
    float t = 0.f;
    VS_CK(cudaEventElapsedTime(&t, h->prof_ev[2 * i], h->prof_ev[2 * i + 1]));
    if (ms) ms[h->prof_class[i]] += (double)t;
    if (timed) timed[h->prof_class[i]] += 1;
  }
  h->prof_used = 0;
  return VS_OK;
}

const char* vs_kernel_class_name(int32_t k) {
  static const char* names[VS_N_KERNEL_CLASSES] = {"pool", "rope_table", "rmsnorm", "qkv_gemm", "qkv_gemv",
                                                   "prefill_attention", "decode_attention", "chunk_scores",
                                                   "bank_update", "other"};
  return (k >= 0 && k < VS_N_KERNEL_CLASSES) ? names[k] : "?";
}

int vs_lm_head(vs_stream* h, const void* hidden, int32_t rows, void* logits, int32_t* next_token, void* cuda_stream) {
  if (h == nullptr || hidden == nullptr || logits == nullptr) return VS_ERR_INVALID_ARG;
  const Dims& D = h->dm;
  const Layout& lo = h->lo;
  if (D.vocab == 0) return VS_ERR_UNSUPPORTED;
  if (rows < 1) return VS_ERR_INVALID_ARG;
  if (rows > D.R_max || rows > 256) return VS_ERR_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(hidden) & 7u) != 0 || (reinterpret_cast<uintptr_t>(logits) & 15u) != 0) return VS_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VS_CK(cudaSetDevice(h->device));
  BatchParams bp;
  VS_BP_INIT(h, bp);
  bp.n_active = 1;
  bp.rows_per_stream = rows;
  VS_TRACE_NEXT(h, bp);
  bf16* xn = h->at<bf16>(lo.xn);
  float* ss = h->at<float>(lo.row_ss);
  VS_LAUNCH(h, st, KC_RMSNORM, launch_lm_norm(hidden, D.out_fp32, D.use_rmsnorm ? h->gain_f : nullptr, xn, ss, D.ss_parts, rows, D.d, st));
  ProjectionOut po;
  std::memset(&po, 0, sizeof(po));
  po.mode = 6; po.final_out = logits; po.final_fp32 = 1;
  if (D.use_rmsnorm) { po.row_ss = ss; po.ss_parts = D.ss_parts; po.norm_eps = D.rms_eps; }
  int rc = run_linear(h, h->tm_lm, h->tm_lm, xn, rows, D.d, D.vocab, po, bp, st);
  if (rc != VS_OK) return rc;
  if (next_token != nullptr) VS_LAUNCH(h, st, KC_OTHER, launch_argmax_rows(static_cast<const float*>(logits), next_token, h->at<unsigned long long>(lo.lm_keys),
                                                                    h->at<int>(lo.lm_tickets), rows, D.vocab, st));
  return VS_OK;
}

int vs_end_turn(vs_stream* h, const int32_t* stream_ids, int32_t n_active) {
  const int rc = check_ids(h, stream_ids, n_active);
  if (rc != VS_OK) return rc;
  for (int i = 0; i < n_active; ++i) h->hs[stream_ids[i]].text_len = 0;
  return VS_OK;
}

int vs_bank_state(vs_stream* h, int32_t stream_id, vs_bank_info* info, int32_t* frame_ids, int64_t* positions,
                  int32_t* slots, int32_t* evict_log, int32_t evict_log_cap, int32_t* evict_log_n, void* emb_out,
                  int32_t layer, void* k_out, void* v_out) {
  if (h == nullptr || stream_id < 0 || stream_id >= h->dm.S) return VS_ERR_INVALID_ARG;
  const Dims& D = h->dm;
  const Layout& lo = h->lo;
  if ((k_out != nullptr || v_out != nullptr) && (layer < 0 || layer >= D.L)) return VS_ERR_INVALID_ARG;
  VS_CK(cudaSetDevice(h->device));
  VS_CK(cudaStreamSynchronize(h->last_stream));
  StreamMeta m;
  VS_CK(cudaMemcpy(&m, h->ws + lo.meta + (size_t)stream_id * sizeof(StreamMeta), sizeof(m), cudaMemcpyDeviceToHost));
  int status[8];
  VS_CK(cudaMemcpy(status, h->ws + lo.status, sizeof(status), cudaMemcpyDeviceToHost));
  std::vector<int32_t> order(D.slots), sframe(D.slots);
  std::vector<int64_t> spos(D.slots);
  VS_CK(cudaMemcpy(order.data(), h->ws + lo.order + (size_t)stream_id * D.slots * 4, (size_t)D.slots * 4, cudaMemcpyDeviceToHost));
  VS_CK(cudaMemcpy(sframe.data(), h->ws + lo.slot_frame + (size_t)stream_id * D.slots * 4, (size_t)D.slots * 4, cudaMemcpyDeviceToHost));
  VS_CK(cudaMemcpy(spos.data(), h->ws + lo.slot_pos + (size_t)stream_id * D.slots * 8, (size_t)D.slots * 8, cudaMemcpyDeviceToHost));
#ifdef VS_DEBUG_BOUNDS
  {
    // a refused store, or guard bytes behind a region that no longer hold their pattern
    DebugTable t;
    VS_CK(cudaMemcpy(&t, h->ws + lo.dbg_table, sizeof(t), cudaMemcpyDeviceToHost));
    bool bad = t.bad_region != -1;
    unsigned char guard[256];
    for (int r = 0; r < DR_COUNT && !bad; ++r) {
      if (lo.region_end[r] <= lo.region_begin[r]) continue;
      VS_CK(cudaMemcpy(guard, h->ws + align_up(lo.region_end[r], 256), kGuardBytes, cudaMemcpyDeviceToHost));
      for (size_t i = 0; i < kGuardBytes; ++i) if (guard[i] != kGuardByte) { bad = true; std::fprintf(stderr, "videoscan: guard bytes behind workspace region %d overwritten\n", r); break; }
    }
    if (t.bad_region != -1) std::fprintf(stderr, "videoscan: store outside workspace region %d refused (offset %lld)\n", t.bad_region, t.bad_offset);
    if (bad && status[0] == 0) status[0] = VS_ERR_BOUNDS;
  }
#endif
  const HostStream& s = h->hs[stream_id];
  if (info != nullptr) {
    info->count = m.count; info->capacity = D.M;
    info->frames_seen = m.frames_seen; info->evictions = m.evictions;
    info->next_pos = s.next_pos; info->prefix_len = s.prefix_len; info->text_len = s.text_len;
    info->last_victim_frame = m.last_victim_frame;
    info->device_status = status[0];
    info->persistent_bytes = lo.persistent_end;
    info->workspace_bytes = lo.total;
  }
  for (int j = 0; j < m.count; ++j) {
    const int sl = order[j];
    if (frame_ids) frame_ids[j] = sframe[sl];
    if (positions) positions[j] = spos[sl];
    if (slots) slots[j] = sl;
  }
  if (evict_log != nullptr && evict_log_cap > 0 && D.log_cap > 0) {
    std::vector<int32_t> ring((size_t)D.log_cap * 2);
    VS_CK(cudaMemcpy(ring.data(), h->ws + lo.evict_log + (size_t)stream_id * D.log_cap * 8, ring.size() * 4, cudaMemcpyDeviceToHost));
    int kept = m.log_count < D.log_cap ? m.log_count : D.log_cap;
    if (kept > evict_log_cap) kept = evict_log_cap;
    for (int i = 0; i < kept; ++i) {
      const int src = (m.log_count - kept + i) % D.log_cap;
      evict_log[2 * i] = ring[2 * src]; evict_log[2 * i + 1] = ring[2 * src + 1];
    }
    if (evict_log_n) *evict_log_n = kept;
  } else if (evict_log_n) {
    *evict_log_n = 0;
  }
  if (emb_out != nullptr) {
    for (int j = 0; j < m.count; ++j)
      VS_CK(cudaMemcpy(static_cast<uint8_t*>(emb_out) + (size_t)j * D.d * 2,
                       h->ws + lo.emb + ((size_t)stream_id * D.slots + order[j]) * D.d * 2, (size_t)D.d * 2, cudaMemcpyDeviceToHost));
  }
  for (int which = 0; which < 2; ++which) {
    uint8_t* dst = static_cast<uint8_t*>(which == 0 ? k_out : v_out);
    if (dst == nullptr) continue;
    const size_t base = (which == 0 ? lo.bank_k : lo.bank_v) + (size_t)layer * layer_stride_bank(D) * 2;
    for (int j = 0; j < m.count; ++j)
      for (int hk = 0; hk < D.Hkv; ++hk)
        VS_CK(cudaMemcpy(dst + ((size_t)j * D.Hkv + hk) * D.D * 2,
                         h->ws + base + ((((size_t)stream_id * D.Hkv + hk) * D.slots) + order[j]) * D.D * 2,
                         (size_t)D.D * 2, cudaMemcpyDeviceToHost));
  }
  return status[0] == 0 ? VS_OK : status[0];
}

int vs_last_step_kv(vs_stream* h, void* k_out, void* v_out, int32_t rows) {
  if (h == nullptr || rows < 1 || rows > h->last_rows) return VS_ERR_INVALID_ARG;
  VS_CK(cudaSetDevice(h->device));
  VS_CK(cudaStreamSynchronize(h->last_stream));
  const size_t bytes = (size_t)rows * h->dm.Hkv * h->dm.D * 2;
  if (k_out) VS_CK(cudaMemcpy(k_out, h->ws + h->lo.kf, bytes, cudaMemcpyDeviceToHost));
  if (v_out) VS_CK(cudaMemcpy(v_out, h->ws + h->lo.vf, bytes, cudaMemcpyDeviceToHost));
  return VS_OK;
}

#ifdef VS_TRACE
// -DVS_TRACE build only: `log` = DEVICE buffer of VS_TRACE_WORDS 64-bit words, zeroed by the caller, or NULL to stop
int vs_trace_set(vs_stream* h, void* log) {
  if (h == nullptr) return VS_ERR_INVALID_ARG;
  h->trace = static_cast<unsigned long long*>(log);
  return VS_OK;
}
#endif

int vs_poison_scratch(vs_stream* h, void* cuda_stream) {
  if (h == nullptr) return VS_ERR_INVALID_ARG;
  VS_CK(cudaSetDevice(h->device));
  VS_LAUNCH(h, static_cast<cudaStream_t>(cuda_stream), KC_OTHER,
            launch_poison(h->ws + h->lo.scratch_begin, h->lo.scratch_end - h->lo.scratch_begin,
                          static_cast<cudaStream_t>(cuda_stream)));
#ifdef VS_DEBUG_BOUNDS
  for (int r = 0; r < DR_COUNT; ++r)
    if (h->lo.region_end[r] > h->lo.region_begin[r] && h->lo.region_begin[r] >= h->lo.scratch_begin)
      VS_CK(cudaMemsetAsync(h->ws + align_up(h->lo.region_end[r], 256), kGuardByte, kGuardBytes, static_cast<cudaStream_t>(cuda_stream)));
#endif
  h->last_stream = static_cast<cudaStream_t>(cuda_stream);
  return VS_OK;
}

}  // extern "C"
