// Memory-bound and bookkeeping kernels of the frame / text step:
//   carrier aggregation (Section 3.3: C = (1/N) sum_i E_i), RoPE table, RMSNorm, eviction
//   scoring and bank commit (Section 3.3, memory mechanism).
#include "vs_common.cuh"
#include "vs_bank_update.cuh"

namespace vs {

// fp64 -> bf16, round to nearest even, with no intermediate rounding: first to fp32 with
// round-to-odd (keeps a sticky bit), then fp32 -> bf16 RNE; 24 bits >= 8 + 2 makes the
// second rounding see exactly the information of the original value.
__device__ __forceinline__ bf16 f64_to_bf16_rne(double x) {
  float f = __double2float_rz(x);
  if ((double)f != x) f = __uint_as_float(__float_as_uint(f) | 1u);
  return __float2bfloat16_rn(f);
}

// ------------------------------------------------------------------------------------------
// Carrier aggregation + layer-0 input assembly + RoPE table.
// grid = (pool_blocks + rope_blocks, n_active).  A pool block owns 64 channels of every row:
// 256 threads = 32 row groups x 8 lanes of 16 bytes (8 channels).  Every thread issues all of
// its <= 8 row loads before using any of them, so the whole frame (1.2 MB) is in flight at
// once.  The sum of <= 256 bf16 values in fp64 is exact, hence independent of the order.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pool_kernel(PoolArgs a, BatchParams bp, int pool_blocks) {
  // what depends on the parameters alone comes before the wait on the stream's earlier kernels
  const int b = blockIdx.y;
  const int sid = bp.stream_id[b];
  const int N = a.N, d = a.d;
  const long long pos0 = bp.pos_base[b];
  VS_STAMP(bp, 0, 0);
  if ((int)blockIdx.x >= pool_blocks) {
    pdl_wait();
    pdl_launch_dependents();
    // RoPE table of this step's N + 1 positions: angle = pos * theta^(-2k/D), in fp64
    const int half = a.D / 2;
    const int idx = (blockIdx.x - pool_blocks) * blockDim.x + threadIdx.x;
    if (idx < (N + 1) * half) {
      const int r = idx / half, k = idx - r * half;
      const double ang = (double)(pos0 + r) * a.inv_freq[k];
      double s, c;
      sincos(ang, &s, &c);
      float2* rp = a.rope + ((size_t)b * (N + 1) + r) * half + k;
      if (VS_STORE_OK(bp, DR_ROPE, rp, 8)) *rp = make_float2((float)c, (float)s);
    }
    return;
  }
  constexpr int RG = 32;                    // row groups
  constexpr int MAXR = 8;                   // rows per thread (N <= 255)
  __shared__ double red[RG][64];
  const int cl = threadIdx.x & 7, grp = threadIdx.x >> 3;
  const int ch = blockIdx.x * 64 + cl * 8;  // d is a multiple of 64
  const bf16* src = a.hidden + (size_t)b * N * d + ch;
  bf16* dst = a.x + (size_t)b * (N + 1) * d + ch;
  pdl_wait();
  pdl_launch_dependents();
  VS_STAMP(bp, 0, 1);
  uint4 v[MAXR];
#pragma unroll
  for (int i = 0; i < MAXR; ++i) {
    const int r = grp + i * RG;
    v[i] = (r < N) ? *reinterpret_cast<const uint4*>(src + (size_t)r * d) : make_uint4(0, 0, 0, 0);
  }
  double acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.0;
#pragma unroll
  for (int i = 0; i < MAXR; ++i) {
    const int r = grp + i * RG;
    if (r < N) {
      if (VS_STORE_OK(bp, DR_HBUF0, dst + (size_t)r * d, 16)) *reinterpret_cast<uint4*>(dst + (size_t)r * d) = v[i];
      const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v[i]);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[2 * j] += (double)__bfloat162float(h2[j].x);
        acc[2 * j + 1] += (double)__bfloat162float(h2[j].y);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) red[grp][cl * 8 + j] = acc[j];
  __syncthreads();
  if (threadIdx.x < 64) {
    const int c = blockIdx.x * 64 + threadIdx.x;
    bf16 cv;
    if (a.carrier_override != nullptr) {
      cv = a.carrier_override[(size_t)b * d + c];
    } else if (a.agg_mode == 1) {
      cv = a.hidden[(size_t)b * N * d + (size_t)(N - 1) * d + c];
    } else {
      double t = 0.0;
#pragma unroll
      for (int g = 0; g < RG; ++g) t += red[g][threadIdx.x];
      cv = f64_to_bf16_rne(t / (double)N);
    }
    bf16* xc = a.x + (size_t)b * (N + 1) * d + (size_t)N * d + c;
    if (VS_STORE_OK(bp, DR_HBUF0, xc, 2)) *xc = cv;   // carrier = last token of the frame
    if (a.emb_stage != nullptr) {
      if (VS_STORE_OK(bp, DR_EMB_STAGE, a.emb_stage + (size_t)b * d + c, 2)) a.emb_stage[(size_t)b * d + c] = cv;          // chunk of frames: the slot is not known yet
    } else if (a.M > 0) {
      const int slot = a.meta[sid].free_slot;
      bf16* ep = a.emb + ((size_t)sid * a.slots + slot) * d + c;
      if (VS_STORE_OK(bp, DR_EMB, ep, 2)) *ep = cv;
      // the step's other kernels take the slot from this copy: the bank update, which moves
      // meta.free_slot on, runs beside the last attention kernel
      if (blockIdx.x == 0 && threadIdx.x == 0) a.step_slot[sid] = slot;
    }
  }
  VS_STAMP(bp, 0, 15);
}

cudaError_t launch_pool(const PoolArgs& a, const BatchParams& bp, cudaStream_t st) {
  const int pool_blocks = a.d / 64;
  const int rope_blocks = ((a.N + 1) * (a.D / 2) + 255) / 256;
  dim3 grid(pool_blocks + rope_blocks, bp.n_active);
  return launch_pdl(pool_kernel, grid, dim3(256), 0, st, a, bp, pool_blocks);
}

__global__ void __launch_bounds__(256) rope_table_kernel(RopeArgs a, BatchParams bp) {
  pdl_wait();
  pdl_launch_dependents();
  const int b = blockIdx.y;
  const int half = a.D / 2, T = bp.rows_per_stream;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * half) return;
  const int r = idx / half, k = idx - r * half;
  const double ang = (double)(bp.pos_base[b] + r) * a.inv_freq[k];
  double s, c;
  sincos(ang, &s, &c);
  a.rope[((size_t)b * T + r) * half + k] = make_float2((float)c, (float)s);
}

cudaError_t launch_rope_table(const RopeArgs& a, const BatchParams& bp, cudaStream_t st) {
  dim3 grid((bp.rows_per_stream * (a.D / 2) + 255) / 256, bp.n_active);
  return launch_pdl(rope_table_kernel, grid, dim3(256), 0, st, a, bp);
}

// ------------------------------------------------------------------------------------------
// RMSNorm statistics of a layer input that no kernel of this library produced (layer 0; deeper
// layers get theirs from the attention kernel that stores the residual rows).
// xn = h * r * gain with r = 1 / sqrt(mean(h^2) + eps).  The row scale r commutes with the
// projection, so the projection applies it in fp32 in its epilogue and reads the bf16 residual
// stream itself: no rounded copy of the normalised activations exists (with a gain vector,
// bf16(h * gain) is written and read instead).  This kernel leaves the row's sum of squares in
// part 0 of row_ss[row][parts].  One block per row.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rms_stats_kernel(const bf16* __restrict__ h, const bf16* __restrict__ gain,
                                                        bf16* __restrict__ hg, float* __restrict__ row_ss,
                                                        int parts, int d) {
  pdl_wait();
  pdl_launch_dependents();
  const size_t row = blockIdx.x;
  const bf16* src = h + row * d;
  float ss = 0.f;
  for (int c = threadIdx.x * 2; c < d; c += 512) {
    const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(src + c));
    ss += v.x * v.x + v.y * v.y;
    if (gain != nullptr) {
      const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(gain + c));
      *reinterpret_cast<__nv_bfloat162*>(hg + row * d + c) = __floats2bfloat162_rn(v.x * g.x, v.y * g.y);
    }
  }
  __shared__ float red[8];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += red[i];
    row_ss[row * parts] = tot;
    for (int i = 1; i < parts; ++i) row_ss[row * parts + i] = 0.f;
  }
}

cudaError_t launch_rms_stats(const bf16* h, const bf16* gain, bf16* hg, float* row_ss, int parts, int rows, int d,
                             cudaStream_t st) {
  return launch_pdl(rms_stats_kernel, dim3(rows), dim3(256), 0, st, h, gain, hg, row_ss, parts, d);
}

// ------------------------------------------------------------------------------------------
// Language-model head (Section 3.3, decoding phase: the next token comes from the output at the last
// position; the Qwen2 backbone of Section 4.1 ends in an RMSNorm and a vocabulary projection).
// lm_norm_kernel: the hidden rows enter as a stored (bf16) tensor whatever type they arrive in; the
// projection reads xn and applies the row scale from the sum of squares left here.  One block per row.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) lm_norm_kernel(const void* __restrict__ h, int h_fp32, const bf16* __restrict__ gain,
                                                      bf16* __restrict__ xn, float* __restrict__ row_ss, int parts, int d) {
  pdl_wait();
  pdl_launch_dependents();
  const size_t row = blockIdx.x;
  float ss = 0.f;
  for (int c = threadIdx.x * 2; c < d; c += 512) {
    __nv_bfloat162 hv;
    if (h_fp32) {
      const float2 f = *reinterpret_cast<const float2*>(static_cast<const float*>(h) + row * d + c);
      hv = __floats2bfloat162_rn(f.x, f.y);
    } else {
      hv = *reinterpret_cast<const __nv_bfloat162*>(static_cast<const bf16*>(h) + row * d + c);
    }
    const float2 v = __bfloat1622float2(hv);
    ss += v.x * v.x + v.y * v.y;
    if (gain != nullptr) {
      const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(gain + c));
      hv = __floats2bfloat162_rn(v.x * g.x, v.y * g.y);
    }
    *reinterpret_cast<__nv_bfloat162*>(xn + row * d + c) = hv;
  }
  __shared__ float red[8];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += red[i];
    row_ss[row * parts] = tot;
    for (int i = 1; i < parts; ++i) row_ss[row * parts + i] = 0.f;
  }
}

cudaError_t launch_lm_norm(const void* h, int h_fp32, const bf16* gain, bf16* xn, float* row_ss, int parts, int rows, int d,
                           cudaStream_t st) {
  return launch_pdl(lm_norm_kernel, dim3(rows), dim3(256), 0, st, h, h_fp32, gain, xn, row_ss, parts, d);
}

// Greedy choice.  (value, index) pairs are compared as "larger value, else equal value and lower
// index"; a NaN is never larger, so it loses to every number, and a row without any number above
// -inf gives token 0.  grid = (slices, rows): every block reduces its slice of the row and offers
// the result to the row's 64-bit key by atomicMax -- the key orders like the pair: the value's
// bits mapped monotonically to an unsigned word on top, the complemented index below -- and the
// block that arrives last (a ticket per row) turns the key back into the token and clears key and
// ticket for the next call.
__device__ __forceinline__ unsigned long long argmax_key(float v, int i) {
  const uint32_t b = __float_as_uint(v);
  const uint32_t ordered = (b & 0x80000000u) ? ~b : (b | 0x80000000u);     // ascending with v (no NaN gets here)
  return ((unsigned long long)ordered << 32) | (uint32_t)(0x7fffffff - i);
}

__global__ void __launch_bounds__(256) argmax_rows_kernel(const float* __restrict__ logits, int32_t* __restrict__ token,
                                                          unsigned long long* __restrict__ keys, int* __restrict__ tickets, int vocab) {
  pdl_wait();
  pdl_launch_dependents();
  const int row = blockIdx.y;
  const float* src = logits + (size_t)row * vocab;
  const int per = (vocab + (int)gridDim.x - 1) / (int)gridDim.x;
  const int i0 = (int)blockIdx.x * per, i1 = min(vocab, i0 + per);
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int i = i0 + (int)threadIdx.x; i < i1; i += 256) {
    const float v = src[i];
    if (v > bv) { bv = v; bi = i; }          // ascending i per thread: the first of equals stays
  }
  auto better = [](float v1, int i1_, float v2, int i2_) { return v1 > v2 || (v1 == v2 && i1_ < i2_); };
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
  }
  __shared__ float sv[8];
  __shared__ int si[8];
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w)
      if (better(sv[w], si[w], bv, bi)) { bv = sv[w]; bi = si[w]; }
    if (bi != 0x7fffffff) atomicMax(keys + row, argmax_key(bv, bi));      // a slice without a number offers nothing
    __threadfence();
    if (atomicAdd(tickets + row, 1) == (int)gridDim.x - 1) {
      __threadfence();
      const unsigned long long k = atomicExch(keys + row, 0ull);
      token[row] = (k == 0ull) ? 0 : 0x7fffffff - (int)(uint32_t)(k & 0xffffffffull);
      tickets[row] = 0;
    }
  }
}

cudaError_t launch_argmax_rows(const float* logits, int32_t* token, unsigned long long* keys, int* tickets, int rows, int vocab,
                               cudaStream_t st) {
  int slices = (vocab + 4095) / 4096;
  if (slices > 64) slices = 64;
  return launch_pdl(argmax_rows_kernel, dim3(slices, rows), dim3(256), 0, st, logits, token, keys, tickets, vocab);
}

// The bank update of one frame as a launch of its own (chunked prefill).
__global__ void __launch_bounds__(256, 8) bank_update_kernel(BankUpdateArgs a, BatchParams bp) {   // <= 32 registers: fits beside a projection CTA
  pdl_wait();
  pdl_launch_dependents();
  bank_update_block(a, bp, (int)blockIdx.y, (int)blockIdx.x);
}

cudaError_t launch_bank_update(const BankUpdateArgs& a, const BatchParams& bp, bool full, cudaStream_t st) {
  dim3 grid(full ? (a.M + 7) / 8 : 1, bp.n_active);
  return launch_pdl(bank_update_kernel, grid, dim3(256), 0, st, a, bp);
}

// All cosines a chunk's bank updates can need when every update scores against its incoming carrier
// (policy 0): frame b's carrier against bank slots 0 .. l1-1 as they were before the chunk and against
// the chunk's carriers 0 .. b-1.  grid = (ceil((l1 + F) / 8), F), one warp per pair.
__global__ void __launch_bounds__(256, 8) chunk_scores_kernel(BankUpdateArgs a, BatchParams bp, const bf16* emb_stage,
                                                              double* out) {
  pdl_wait();                       // the pooled carriers are in place
  pdl_launch_dependents();
  const int b = blockIdx.y, lane = threadIdx.x & 31;
  const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (c >= a.chunk_l1 + b) return;                                 // uniform over the warp
  const int sid = bp.stream_id[b];
  const bf16* va = (c < a.chunk_l1) ? a.emb + ((size_t)sid * a.slots + c) * a.d : emb_stage + (size_t)(c - a.chunk_l1) * a.d;
  const double s = warp_cosine(va, emb_stage + (size_t)b * a.d, a.d, lane);
  if (lane == 0) out[(size_t)b * a.pre_stride + c] = s;
}

cudaError_t launch_chunk_scores(const BankUpdateArgs& a, const BatchParams& bp, const bf16* emb_stage, double* out, cudaStream_t st) {
  dim3 grid((a.chunk_l1 + bp.n_active + 7) / 8, bp.n_active);
  return launch_pdl(chunk_scores_kernel, grid, dim3(256), 0, st, a, bp, emb_stage, out);
}

// The chunk's bank updates in turn by one block (the scores are looked up, the rest is the streaming
// update): frame b finds the bank as frame b-1 left it.
__global__ void __launch_bounds__(256, 8) chunk_plan_kernel(BankUpdateArgs a, BatchParams bp) {
  pdl_wait();
  pdl_launch_dependents();
  for (int b = 0; b < bp.n_active; ++b) {
    bank_update_block(a, bp, b, 0);
    __threadfence_block();
    __syncthreads();
  }
}

cudaError_t launch_chunk_plan(const BankUpdateArgs& a, const BatchParams& bp, cudaStream_t st) {
  return launch_pdl(chunk_plan_kernel, dim3(1), dim3(256), 0, st, a, bp);
}

// grid = F CTAs of 128 threads: CTA i copies the carrier row of the chunk's frame i unless a later
// update of the chunk evicted that carrier (its slot then belongs to someone else).
__global__ void __launch_bounds__(128) chunk_kv_commit_kernel(ChunkKvCommitArgs a) {
  pdl_wait();                       // the attention launch has finished reading the bank
  pdl_launch_dependents();
  const int i = blockIdx.x;
  for (int u = i + 1; u < a.F; ++u)
    if (a.chunk_victim[u] == a.l1 + i) return;
  const int slot = a.chunk_slot[i];
  const int per_head = a.D / 8;                                       // 16-byte chunks of one head's row
  const size_t src = ((size_t)i * (a.N + 1) + a.N) * a.Hkv * a.D;
  for (int c = threadIdx.x; c < a.Hkv * per_head; c += blockDim.x) {
    const int hk = c / per_head, cc = c - hk * per_head;
    const size_t dst = (((size_t)a.sid * a.Hkv + hk) * a.slots + slot) * a.D + cc * 8;
    *reinterpret_cast<uint4*>(a.bank_k + dst) = *reinterpret_cast<const uint4*>(a.kf + src + hk * a.D + cc * 8);
    *reinterpret_cast<uint4*>(a.bank_v + dst) = *reinterpret_cast<const uint4*>(a.vf + src + hk * a.D + cc * 8);
  }
}

cudaError_t launch_chunk_kv_commit(const ChunkKvCommitArgs& a, cudaStream_t st) {
  return launch_pdl(chunk_kv_commit_kernel, dim3(a.F), dim3(128), 0, st, a);
}

__global__ void __launch_bounds__(256) gather_carriers_kernel(const bf16* __restrict__ emb, const int32_t* __restrict__ order,
                                                             bf16* __restrict__ x, int sid, int slots, int d) {
  pdl_wait();
  pdl_launch_dependents();
  const int i = blockIdx.x;
  const uint4* src = reinterpret_cast<const uint4*>(emb + ((size_t)sid * slots + order[(size_t)sid * slots + i]) * d);
  uint4* dst = reinterpret_cast<uint4*>(x + (size_t)i * d);
  for (int c = threadIdx.x; c < d / 8; c += blockDim.x) dst[c] = src[c];
}

cudaError_t launch_gather_carriers(const bf16* emb, const int32_t* order, bf16* x, int sid, int slots, int d, int count,
                                   cudaStream_t st) {
  return launch_pdl(gather_carriers_kernel, dim3(count), dim3(256), 0, st, emb, order, x, sid, slots, d);
}

__global__ void poison_kernel(uint32_t* p, size_t n) {
  pdl_wait();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    p[i] = 0xFFFFFFFFu;
}

cudaError_t launch_poison(void* p, size_t bytes, cudaStream_t st) {
  poison_kernel<<<592, 256, 0, st>>>(reinterpret_cast<uint32_t*>(p), bytes / 4);
  return cudaGetLastError();
}

// a stream starts over (new video): empty bank, no history; K/V payloads need no clearing
// because nothing reads a slot that the metadata does not list
__global__ void reset_kernel(StreamMeta* meta, int32_t* slot_frame, int slots, BatchParams bp) {
  pdl_wait();
  const int sid = bp.stream_id[blockIdx.x];
  for (int i = threadIdx.x; i < slots; i += blockDim.x) slot_frame[(size_t)sid * slots + i] = -1;
  if (threadIdx.x == 0) {
    StreamMeta m;
    m.count = 0; m.free_slot = 0; m.victim_logical = -1; m.last_victim_frame = -1;
    m.frames_seen = 0; m.evictions = 0; m.log_count = 0; m.score_ticket = 0;
    m.pad[0] = m.pad[1] = m.pad[2] = m.pad[3] = 0;
    meta[sid] = m;
  }
}

cudaError_t launch_reset(StreamMeta* meta, int32_t* slot_frame, int slots, const BatchParams& bp, cudaStream_t st) {
  reset_kernel<<<bp.n_active, 256, 0, st>>>(meta, slot_frame, slots, bp);
  return cudaGetLastError();
}

}  // namespace vs
