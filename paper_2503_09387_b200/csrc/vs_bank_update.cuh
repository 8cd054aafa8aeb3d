// Bank update (Section 3.3, memory mechanism): evict-if-full, then append, as a device function
// run by spare CTAs of a frame step's last attention launch (it needs the carrier embeddings,
// not the attention's result, so it runs beside it instead of after it).
#pragma once

#include "vs_common.cuh"

namespace vs {

__device__ __forceinline__ double warp_tree_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// cos(va, vb) over d elements by one warp: lane p sums elements k = p (mod 32) in ascending k in
// fp64, then a butterfly 16, 8, 4, 2, 1; the result is the same in every lane
__device__ __forceinline__ double warp_cosine(const bf16* va, const bf16* vb, int d, int lane) {
  double dot = 0.0, na = 0.0, nb = 0.0;
  for (int k = lane; k < d; k += 32) {
    const double x = (double)__bfloat162float(va[k]);
    const double y = (double)__bfloat162float(vb[k]);
    dot = __dadd_rn(dot, __dmul_rn(x, y));
    na = __dadd_rn(na, __dmul_rn(x, x));
    nb = __dadd_rn(nb, __dmul_rn(y, y));
  }
  dot = warp_tree_sum(dot); na = warp_tree_sum(na); nb = warp_tree_sum(nb);
  double s = 0.0;
  if (na != 0.0 && nb != 0.0) s = __ddiv_rn(dot, __dmul_rn(__dsqrt_rn(na), __dsqrt_rn(nb)));
  // a vector holding Inf or NaN has no cosine: counted as 0, like a zero vector
  if (!(s >= -2.0 && s <= 2.0)) s = 0.0;
  return s;
}

// Block `block` of `n_blocks` (as the host sized them: one if no listed stream's bank is full,
// else ceil(M / 8)) working on listed stream b.  Called by every thread of the CTA; threads
// beyond the first 256 only keep the barriers company.
// Bank not full: block 0 appends; the other blocks return.
// Bank full: one warp per temporal index j scores cos(e_j, e_other) -- e_other is the incoming
// carrier (policy 0) or the next carrier in temporal order (policy 1).  Dot products are
// accumulated in fp64 in a fixed order -- lane p sums elements k = p (mod 32) in ascending k,
// then a butterfly 16, 8, 4, 2, 1 -- so that the score, and with it the argmax, is
// reproducible bit for bit; products of two bf16 values are exact in fp64, so fused and
// unfused accumulation agree.  The last block of a stream to finish picks the victim (largest
// score, oldest on ties), closes the gap in the temporal order and appends.
__device__ __forceinline__ void bank_update_block(const BankUpdateArgs& a, const BatchParams& bp, int b, int block) {
  constexpr int NT = 256;
  const int tid = threadIdx.x;
  const bool on = tid < NT;
  const int sid = bp.stream_id[b];
  StreamMeta* meta = a.meta + sid;
  if (a.M == 0) {
    if (block == 0 && tid == 0) { meta->frames_seen += 1; meta->last_victim_frame = -1; }
    return;
  }
  int32_t* order = a.order + (size_t)sid * a.slots;
  int32_t* slot_frame = a.slot_frame + (size_t)sid * a.slots;
  int64_t* slot_pos = a.slot_pos + (size_t)sid * a.slots;
  const int count = bp.count[b];
  const int incoming = (a.incoming_emb != nullptr) ? meta->free_slot : a.step_slot[sid];
  // chunked prefill: the incoming embedding is read from where it is parked and moved into its slot
  // by whoever commits
  const bf16* emb_in = (a.incoming_emb != nullptr) ? a.incoming_emb + (size_t)b * a.d
                                                   : a.emb + ((size_t)sid * a.slots + incoming) * a.d;
  auto adopt = [&]() {      // all threads of the committing block
    if (a.incoming_emb != nullptr) {
      bf16* dst = const_cast<bf16*>(a.emb) + ((size_t)sid * a.slots + incoming) * a.d;
      for (int k = tid; k < a.d; k += blockDim.x) if (VS_STORE_OK(bp, DR_EMB, dst + k, 2)) dst[k] = emb_in[k];
      if (tid == 0) { a.record_slot[b] = incoming; a.record_victim[b] = -1; }
    }
  };
  const int64_t carrier_pos = bp.pos_base[b] + bp.rows_per_stream - 1;
  if (count < a.M) {
    if (block == 0) adopt();
    if (block == 0 && tid == 0) {
      if (VS_STORE_OK(bp, DR_ORDER, order + count, 4)) order[count] = incoming;
      if (VS_STORE_OK(bp, DR_SLOT_FRAME, slot_frame + incoming, 4)) slot_frame[incoming] = (int32_t)bp.frame_id[b];
      if (VS_STORE_OK(bp, DR_SLOT_POS, slot_pos + incoming, 8)) slot_pos[incoming] = carrier_pos;
      meta->count = count + 1;
      meta->free_slot = count + 1;          // slots fill in order until the bank is full
      meta->last_victim_frame = -1;
      meta->frames_seen += 1;
    }
    return;
  }
  // ---- bank full: score, then the last block commits --------------------------------------
  double* scores = a.scores + (size_t)sid * a.slots;
  const int lane = tid & 31;
  const int n_score_blocks = (a.M + 7) / 8;
  const bool planned = a.pre_scores != nullptr;      // one block, scores already there: no ticket
  if (!planned) {
  if (block >= n_score_blocks) return;
  const int j = block * 8 + (tid >> 5);
  if (on && j < count && a.policy != 2) {
    const int sa = order[j];
    const int sb = (a.policy == 1 && j + 1 < count) ? order[j + 1] : incoming;
    const bf16* va = a.emb + ((size_t)sid * a.slots + sa) * a.d;
    const bf16* vb = (sb == incoming) ? emb_in : a.emb + ((size_t)sid * a.slots + sb) * a.d;
    const double s = warp_cosine(va, vb, a.d, lane);
    if (lane == 0 && VS_STORE_OK(bp, DR_SCORES, scores + j, 8)) scores[j] = s;
  }
  __shared__ int is_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = (atomicAdd(&meta->score_ticket, 1) == n_score_blocks - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  }
  __shared__ double best_s[NT];
  __shared__ int best_j[NT];
  double bs = -4.0; int bj = 0x7fffffff;   // every score lies in [-2, 2], so some thread takes an index < count
  if (on && a.policy != 2) {
    for (int i = tid; i < count; i += NT) {
      double s;
      if (planned) {
        // the carrier at temporal index i, as an index on the chunk's bank axis
        const int slot_i = order[i];
        const long long fr = slot_frame[slot_i];
        const int c = (fr >= a.chunk_first_frame) ? a.chunk_l1 + (int)(fr - a.chunk_first_frame) : slot_i;
        s = a.pre_scores[(size_t)b * a.pre_stride + c];
      } else {
        s = __ldcg(scores + i);
      }
      if (s > bs) { bs = s; bj = i; }                 // ascending i: first maximum kept
    }
  }
  if (on) { best_s[tid] = bs; best_j[tid] = bj; }
  __syncthreads();
  for (int o = NT / 2; o > 0; o >>= 1) {
    if (tid < o) {
      const double s2 = best_s[tid + o]; const int j2 = best_j[tid + o];
      if (s2 > best_s[tid] || (s2 == best_s[tid] && j2 < best_j[tid])) {
        best_s[tid] = s2; best_j[tid] = j2;
      }
    }
    __syncthreads();
  }
  adopt();
  // the index stays inside the bank whatever the scores were
  const int v = (a.policy == 2 || (unsigned)best_j[0] >= (unsigned)count) ? 0 : best_j[0];
  const int victim_slot = order[v];
  const int victim_frame = slot_frame[victim_slot];
  __syncthreads();
  // close the gap in the temporal order, one chunk of NT at a time in ascending order: a chunk
  // reads [base+1, base+NT] before anything at or above base is written
  for (int base = v; base < count - 1; base += NT) {
    const int jj = base + tid;
    const int32_t next = (on && jj < count - 1) ? order[jj + 1] : 0;
    __syncthreads();
    if (on && jj < count - 1 && VS_STORE_OK(bp, DR_ORDER, order + jj, 4)) order[jj] = next;
    __syncthreads();
  }
  if (tid == 0) {
    if (VS_STORE_OK(bp, DR_ORDER, order + count - 1, 4)) order[count - 1] = incoming;
    if (VS_STORE_OK(bp, DR_SLOT_FRAME, slot_frame + victim_slot, 4)) slot_frame[victim_slot] = -1;
    if (VS_STORE_OK(bp, DR_SLOT_FRAME, slot_frame + incoming, 4)) slot_frame[incoming] = (int32_t)bp.frame_id[b];
    if (VS_STORE_OK(bp, DR_SLOT_POS, slot_pos + incoming, 8)) slot_pos[incoming] = carrier_pos;
    if (a.log_cap > 0) {
      int32_t* e = a.evict_log + ((size_t)sid * a.log_cap + (meta->log_count % a.log_cap)) * 2;
      if (VS_STORE_OK(bp, DR_EVICT_LOG, e, 8)) { e[0] = (int32_t)bp.frame_id[b]; e[1] = victim_frame; }
    }
    meta->log_count += 1;
    meta->evictions += 1;
    meta->last_victim_frame = victim_frame;
    if (a.incoming_emb != nullptr)
      a.record_victim[b] = (victim_frame >= a.chunk_first_frame) ? a.chunk_l1 + (int)(victim_frame - a.chunk_first_frame)
                                                                 : victim_slot;
    meta->free_slot = victim_slot;
    meta->victim_logical = -1;
    meta->frames_seen += 1;
    if (!planned) meta->score_ticket = 0;
  }
}

}  // namespace vs
