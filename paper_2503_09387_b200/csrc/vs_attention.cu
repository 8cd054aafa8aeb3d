// Attention kernels (Eq. 1: Y = Softmax(Q K^T / sqrt(d_k)) V, per head, grouped KV heads).
//
// prefill_attn_kernel -- the frame step (Section 3.3, prefilling) and multi-token text
//   steps: query rows of one step attend to [prompt prefix | carrier bank | earlier tokens
//   of the turn | the step's own rows, causal].  The carrier is the last row of its frame,
//   so the causal rule alone lets it see every visual token while no visual token sees it
//   (Section 3.2).  One CTA = 16 query rows x one KV head; warp g owns query head
//   hkv*G + g, so the G query heads of a group share every K/V tile staged in shared
//   memory.  QK^T and PV run on tensor cores (mma.sync m16n8k16, bf16 in, fp32 out) with
//   the online softmax kept in registers and row statistics reduced by warp shuffles.
//
// decode_attn_kernel -- the decoding phase (Section 3.3): one query token per stream over
//   [prefix | bank | tail]; the key range is split over CTAs, each thread streams K/V
//   with 128-bit loads, and the last CTA of a (stream, KV head) to finish combines the
//   partial (m, l, o) triples.  No CTA waits for another.
#include "vs_common.cuh"

namespace vs {

namespace {

constexpr int kChunk = 64;   // keys per shared-memory tile

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk `c` of key row `r` inside a [kChunk][D] bf16 tile; the XOR
// spreads the 8 rows an ldmatrix touches over all banks
template <int D>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return (uint32_t)(r * (D * 2) + ((c ^ (r & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(256) prefill_attn_kernel(AttnArgs a, BatchParams bp) {
  extern __shared__ __align__(128) uint8_t smem[];
  constexpr int kTileBytes = kChunk * D * 2;
  constexpr int CPR = D / 8;                 // 16-byte chunks per key row
  const int b = blockIdx.z, hkv = blockIdx.y;
  const int r0 = blockIdx.x * 16;
  const int rps = bp.rows_per_stream;
  const int sid = bp.stream_id[b];
  const int G = a.Hq / a.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qhead = hkv * G + warp;
  const int nthreads = blockDim.x;
  const int count = bp.count[b];
  const bool bank_full = (a.M > 0 && count == a.M);
  const int free_slot = bank_full ? a.meta[sid].free_slot : -1;

  // segment lengths and base pointers for this (stream, KV head)
  int seg_len[4];
  const bf16* seg_k[4];
  const bf16* seg_v[4];
  long long seg_stride[4];
  int seg_kind[4];
  int n_chunks_total = 0;
  int seg_chunk0[5];
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    seg_len[s] = 0; seg_k[s] = nullptr; seg_v[s] = nullptr; seg_stride[s] = 0; seg_kind[s] = 0;
    seg_chunk0[s] = n_chunks_total;
    if (s < a.n_seg) {
      const AttnSegment sg = a.seg[s];
      int len = 0;
      if (sg.kind == 0) len = bp.prefix_len[b];
      else if (sg.kind == 1) len = (a.M == 0) ? 0 : (bank_full ? a.M + 1 : count);
      else if (sg.kind == 2) len = bp.text_len[b];
      else len = min(rps, r0 + 16);          // causal: keys beyond the tile's last row are never visible
      const long long off = (long long)(sg.by_batch ? b : sid) * sg.stream_stride + (long long)hkv * sg.head_stride;
      seg_len[s] = len; seg_k[s] = sg.k + off; seg_v[s] = sg.v + off;
      seg_stride[s] = sg.row_stride; seg_kind[s] = sg.kind;
      n_chunks_total += (len + kChunk - 1) / kChunk;
    }
  }
  seg_chunk0[4] = n_chunks_total;

  auto locate = [&](int ci, int& s, int& start) {
    s = 0;
#pragma unroll
    for (int t = 1; t < 4; ++t) if (ci >= seg_chunk0[t]) s = t;
    start = (ci - seg_chunk0[s]) * kChunk;
  };
  auto load_chunk = [&](int ci, int buf) {
    int s, start;
    locate(ci, s, start);
    const bf16* kp = seg_k[s]; const bf16* vp = seg_v[s];
    const long long stride = seg_stride[s];
    const int len = seg_len[s];
    const uint32_t kdst = smem_u32(smem) + (uint32_t)buf * 2u * kTileBytes;
    const uint32_t vdst = kdst + kTileBytes;
    for (int idx = threadIdx.x; idx < kChunk * CPR; idx += nthreads) {
      const int r = idx / CPR, c = idx - r * CPR;
      const bool valid = (start + r) < len;
      const long long goff = valid ? ((long long)(start + r) * stride + c * 8) : 0;
      cp_async16(kdst + tile_off<D>(r, c), kp + goff, valid);
      cp_async16(vdst + tile_off<D>(r, c), vp + goff, valid);
    }
  };

  // Q fragments (A operand): rows r0 + lane/4 and + 8, all D/16 k-steps
  // (hi and lo halves: Q = qf + ql carries 16 mantissa bits into the scores)
  uint32_t qf[D / 16][4], ql[D / 16][4];
  {
    const int ra = r0 + (lane >> 2), rb = ra + 8;
    const size_t oa = ((size_t)b * rps + ra) * a.Hq * D + (size_t)qhead * D + 2 * (lane & 3);
    const size_t ob = ((size_t)b * rps + rb) * a.Hq * D + (size_t)qhead * D + 2 * (lane & 3);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      qf[ks][0] = (ra < rps) ? *reinterpret_cast<const uint32_t*>(a.q + oa + ks * 16) : 0u;
      qf[ks][1] = (rb < rps) ? *reinterpret_cast<const uint32_t*>(a.q + ob + ks * 16) : 0u;
      qf[ks][2] = (ra < rps) ? *reinterpret_cast<const uint32_t*>(a.q + oa + ks * 16 + 8) : 0u;
      qf[ks][3] = (rb < rps) ? *reinterpret_cast<const uint32_t*>(a.q + ob + ks * 16 + 8) : 0u;
      ql[ks][0] = (ra < rps) ? *reinterpret_cast<const uint32_t*>(a.q_lo + oa + ks * 16) : 0u;
      ql[ks][1] = (rb < rps) ? *reinterpret_cast<const uint32_t*>(a.q_lo + ob + ks * 16) : 0u;
      ql[ks][2] = (ra < rps) ? *reinterpret_cast<const uint32_t*>(a.q_lo + oa + ks * 16 + 8) : 0u;
      ql[ks][3] = (rb < rps) ? *reinterpret_cast<const uint32_t*>(a.q_lo + ob + ks * 16 + 8) : 0u;
    }
  }

  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
  const int qrow[2] = {r0 + (lane >> 2), r0 + (lane >> 2) + 8};

  if (n_chunks_total > 0) { load_chunk(0, 0); }
  cp_async_commit();

  for (int ci = 0; ci < n_chunks_total; ++ci) {
    const int buf = ci & 1;
    if (ci + 1 < n_chunks_total) load_chunk(ci + 1, buf ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();

    int s_idx, start;
    locate(ci, s_idx, start);
    const int len = seg_len[s_idx];
    const int kind = seg_kind[s_idx];
    const uint32_t kbase = smem_u32(smem) + (uint32_t)buf * 2u * kTileBytes;
    const uint32_t vbase = kbase + kTileBytes;

    // S = Q K^T for 64 keys
    float sc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        const int key = jp * 16 + ((lane >> 4) << 3) + (lane & 7);
        const int chunk = 2 * ks + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(kbase + tile_off<D>(key, chunk), b0, b1, b2, b3);
        mma_bf16(sc[2 * jp], qf[ks], b0, b1);
        mma_bf16(sc[2 * jp + 1], qf[ks], b2, b3);
        mma_bf16(sc[2 * jp], ql[ks], b0, b1);
        mma_bf16(sc[2 * jp + 1], ql[ks], b2, b3);
      }
    }
    // mask, scale (log2 domain), running max
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = start + j * 8 + 2 * (lane & 3) + (e & 1);
        const int row = qrow[e >> 1];
        bool vis = key < len;
        if (kind == 1) vis = vis && (key != free_slot);
        if (kind == 3) vis = vis && (key <= row);
        const float v = vis ? sc[j][e] * a.scale_log2e : -INFINITY;
        sc[j][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float alpha[2], m_use[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      const float m_new = fmaxf(m_run[h], mx[h]);
      m_use[h] = (m_new == -INFINITY) ? 0.f : m_new;
      alpha[h] = (m_run[h] == -INFINITY) ? 0.f : exp2f(m_run[h] - m_use[h]);
      m_run[h] = m_new;
    }
    float rs[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float p = exp2f(sc[j][e] - m_use[e >> 1]);
        sc[j][e] = p;
        rs[e >> 1] += p;
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      rs[h] += __shfl_xor_sync(0xffffffffu, rs[h], 1);
      rs[h] += __shfl_xor_sync(0xffffffffu, rs[h], 2);
      l_run[h] = l_run[h] * alpha[h] + rs[h];
    }
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
      o[i][0] *= alpha[0]; o[i][1] *= alpha[0]; o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t pa[4];
      pa[0] = pack_bf16(sc[2 * kk][0], sc[2 * kk][1]);
      pa[1] = pack_bf16(sc[2 * kk][2], sc[2 * kk][3]);
      pa[2] = pack_bf16(sc[2 * kk + 1][0], sc[2 * kk + 1][1]);
      pa[3] = pack_bf16(sc[2 * kk + 1][2], sc[2 * kk + 1][3]);
#pragma unroll
      for (int ndp = 0; ndp < D / 16; ++ndp) {
        const int key = kk * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
        const int chunk = 2 * ndp + (lane >> 4);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(vbase + tile_off<D>(key, chunk), b0, b1, b2, b3);
        mma_bf16(o[2 * ndp], pa, b0, b1);
        mma_bf16(o[2 * ndp + 1], pa, b2, b3);
      }
    }
    __syncthreads();   // everyone is done with `buf` before the next iteration refills it
  }
  cp_async_wait<0>();

  // normalise and store; optionally add onto the residual stream
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = qrow[h];
    if (row >= rps) continue;
    const float inv = (l_run[h] > 0.f) ? 1.f / l_run[h] : 0.f;
    const size_t grow = (size_t)b * rps + row;
    const size_t obase = grow * a.Hq * D + (size_t)qhead * D + 2 * (lane & 3);
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
      const float v0 = o[i][2 * h] * inv, v1 = o[i][2 * h + 1] * inv;
      if (a.out_fp32) *reinterpret_cast<float2*>(static_cast<float*>(a.out) + obase + i * 8) = make_float2(v0, v1);
      else *reinterpret_cast<__nv_bfloat162*>(static_cast<bf16*>(a.out) + obase + i * 8) = __floats2bfloat162_rn(v0, v1);
      if (a.h_out != nullptr) {
        const size_t hoff = grow * a.Hq * D + (size_t)qhead * D + 2 * (lane & 3) + i * 8;
        const float2 hv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(a.h_in + hoff));
        *reinterpret_cast<__nv_bfloat162*>(a.h_out + hoff) = __floats2bfloat162_rn(hv.x + v0, hv.y + v1);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// split-KV decode
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(128) decode_attn_kernel(DecodeArgs a, BatchParams bp) {
  constexpr int LPK = D / 8;            // lanes that share one key row (16 bytes each)
  constexpr int KPW = 32 / LPK;         // keys a warp handles per iteration
  constexpr int NSTATE = 4 * KPW;
  constexpr int GMAX = 8;
  __shared__ float st_m[NSTATE][GMAX];
  __shared__ float st_l[NSTATE][GMAX];
  __shared__ float st_o[NSTATE][GMAX][D];
  __shared__ int is_last;

  const int split = blockIdx.x, hkv = blockIdx.y, b = blockIdx.z;
  const int sid = bp.stream_id[b];
  const int G = a.Hq / a.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPK, li = lane % LPK;
  const int count = bp.count[b];
  const bool bank_full = (a.M > 0 && count == a.M);
  const int free_slot = bank_full ? a.meta[sid].free_slot : -1;

  int P, NB, TL;
  if (a.to_prefix) { P = bp.prefix_len[b] + 1; NB = 0; TL = 0; }
  else { P = bp.prefix_len[b]; NB = (a.M == 0) ? 0 : (bank_full ? a.M + 1 : count); TL = bp.text_len[b] + 1; }
  const int Lv = P + NB + TL;
  const int begin = (int)(((long long)Lv * split) / a.nsplit);
  const int end = (int)(((long long)Lv * (split + 1)) / a.nsplit);

  const bf16* pk = a.prefix_k + ((size_t)sid * a.Hkv + hkv) * a.maxP * D;
  const bf16* pv = a.prefix_v + ((size_t)sid * a.Hkv + hkv) * a.maxP * D;
  const bf16* bk = a.bank_k + ((size_t)sid * a.Hkv + hkv) * a.slots * D;
  const bf16* bv = a.bank_v + ((size_t)sid * a.Hkv + hkv) * a.slots * D;
  const bf16* tk = a.tail_k + ((size_t)sid * a.Hkv + hkv) * a.maxT * D;
  const bf16* tv = a.tail_v + ((size_t)sid * a.Hkv + hkv) * a.maxT * D;

  float q[GMAX][8];
#pragma unroll
  for (int g = 0; g < GMAX; ++g) {
    if (g < G) {
      const size_t qo = (size_t)b * a.Hq * D + (size_t)(hkv * G + g) * D + li * 8;
      const uint4 raw = *reinterpret_cast<const uint4*>(a.q + qo);
      const uint4 raw_lo = *reinterpret_cast<const uint4*>(a.q_lo + qo);
      const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
      const __nv_bfloat162* l2 = reinterpret_cast<const __nv_bfloat162*>(&raw_lo);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h2[i]);
        const float2 fl = __bfloat1622float2(l2[i]);
        q[g][2 * i] = (f.x + fl.x) * a.scale_log2e; q[g][2 * i + 1] = (f.y + fl.y) * a.scale_log2e;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) q[g][i] = 0.f;
    }
  }
  float m[GMAX], l[GMAX], o[GMAX][8];
#pragma unroll
  for (int g = 0; g < GMAX; ++g) {
    m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
  }

  for (int base = begin + warp * KPW; base < end; base += 4 * KPW) {
    const int v = base + sub;
    bool active = v < end;
    const bf16* kp = pk; const bf16* vp = pv;
    if (active) {
      if (v < P) { kp = pk + (size_t)v * D; vp = pv + (size_t)v * D; }
      else if (v < P + NB) {
        const int slot = v - P;
        if (slot == free_slot) active = false;
        kp = bk + (size_t)slot * D; vp = bv + (size_t)slot * D;
      } else { const int t = v - P - NB; kp = tk + (size_t)t * D; vp = tv + (size_t)t * D; }
    }
    float kf[8], vf[8];
    if (active) {
      const uint4 kr = *reinterpret_cast<const uint4*>(kp + li * 8);
      const uint4 vr = *reinterpret_cast<const uint4*>(vp + li * 8);
      const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kr);
      const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vr);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 fk = __bfloat1622float2(k2[i]); kf[2 * i] = fk.x; kf[2 * i + 1] = fk.y;
        const float2 fv = __bfloat1622float2(v2[i]); vf[2 * i] = fv.x; vf[2 * i + 1] = fv.y;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) { kf[i] = 0.f; vf[i] = 0.f; }
    }
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
      if (g < G) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) s += q[g][i] * kf[i];
#pragma unroll
        for (int off = LPK / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (active) {
          if (s > m[g]) {
            const float sc = exp2f(m[g] - s);      // exp2f(-inf) = 0 on the first key
            l[g] *= sc;
#pragma unroll
            for (int i = 0; i < 8; ++i) o[g][i] *= sc;
            m[g] = s;
          }
          const float p = exp2f(s - m[g]);
          l[g] += p;
#pragma unroll
          for (int i = 0; i < 8; ++i) o[g][i] += p * vf[i];
        }
      }
    }
  }
  // merge the NSTATE running states of this CTA
  const int state = warp * KPW + sub;
#pragma unroll
  for (int g = 0; g < GMAX; ++g) {
    if (g < G) {
      if (li == 0) { st_m[state][g] = m[g]; st_l[state][g] = l[g]; }
#pragma unroll
      for (int i = 0; i < 8; ++i) st_o[state][g][li * 8 + i] = o[g][i];
    }
  }
  __syncthreads();
  float* part = a.partials + (((size_t)split * bp.n_active + b) * a.Hq + (size_t)hkv * G) * (D + 2);
  for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
    const int g = idx / D, c = idx - g * D;
    float M = -INFINITY;
#pragma unroll
    for (int s = 0; s < NSTATE; ++s) M = fmaxf(M, st_m[s][g]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int s = 0; s < NSTATE; ++s) {
      const float w = (st_m[s][g] == -INFINITY) ? 0.f : exp2f(st_m[s][g] - M);
      L += st_l[s][g] * w;
      O += st_o[s][g][c] * w;
    }
    part[(size_t)g * (D + 2) + c] = O;
    if (c == 0) { part[(size_t)g * (D + 2) + D] = M; part[(size_t)g * (D + 2) + D + 1] = L; }
  }
  // last CTA of this (stream, KV head) combines the splits
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int done = atomicAdd(a.tickets + sid * a.Hkv + hkv, 1);
    is_last = (done == a.nsplit - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
    const int g = idx / D, c = idx - g * D;
    const int qh = hkv * G + g;
    float M = -INFINITY;
    for (int s = 0; s < a.nsplit; ++s)
      M = fmaxf(M, __ldcg(a.partials + (((size_t)s * bp.n_active + b) * a.Hq + qh) * (D + 2) + D));
    float L = 0.f, O = 0.f;
    for (int s = 0; s < a.nsplit; ++s) {
      const float* pp = a.partials + (((size_t)s * bp.n_active + b) * a.Hq + qh) * (D + 2);
      const float ms = __ldcg(pp + D);
      const float w = (ms == -INFINITY) ? 0.f : exp2f(ms - M);
      L += __ldcg(pp + D + 1) * w;
      O += __ldcg(pp + c) * w;
    }
    const float val = (L > 0.f) ? O / L : 0.f;
    const size_t off = (size_t)b * a.Hq * D + (size_t)qh * D + c;
    if (a.out_fp32) static_cast<float*>(a.out)[off] = val;
    else static_cast<bf16*>(a.out)[off] = __float2bfloat16_rn(val);
    if (a.h_out != nullptr) a.h_out[off] = __float2bfloat16_rn(__bfloat162float(a.h_in[off]) + val);
  }
  if (threadIdx.x == 0) a.tickets[sid * a.Hkv + hkv] = 0;
}

}  // namespace

cudaError_t prefill_attention_init() {
  cudaError_t e = cudaFuncSetAttribute(prefill_attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       4 * kChunk * 128 * 2);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(prefill_attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              4 * kChunk * 64 * 2);
}

cudaError_t launch_prefill_attention(const AttnArgs& a, const BatchParams& bp, cudaStream_t st) {
  const int G = a.Hq / a.Hkv;
  dim3 grid((bp.rows_per_stream + 15) / 16, a.Hkv, bp.n_active);
  dim3 block(32 * G);
  if (a.D == 128) {
    prefill_attn_kernel<128><<<grid, block, 4 * kChunk * 128 * 2, st>>>(a, bp);
  } else if (a.D == 64) {
    prefill_attn_kernel<64><<<grid, block, 4 * kChunk * 64 * 2, st>>>(a, bp);
  } else {
    return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_decode_attention(const DecodeArgs& a, const BatchParams& bp, cudaStream_t st) {
  dim3 grid(a.nsplit, a.Hkv, bp.n_active);
  if (a.D == 128) decode_attn_kernel<128><<<grid, 128, 0, st>>>(a, bp);
  else if (a.D == 64) decode_attn_kernel<64><<<grid, 128, 0, st>>>(a, bp);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace vs
