// Decode attention (Section 3.3, decoding phase; Eq. 1 per head with grouped KV heads): one
// query token per stream attends over [prompt prefix | carrier bank | text of the turn].  No
// visual-token K/V exists at this point -- only carriers.
//
// grid = (key splits, KV heads, streams), 256 threads.  A group of D/8 lanes owns one key row
// and reads it with 128-bit loads; every lane issues the K and V loads of four keys before it
// uses any of them, so a warp has 8 key rows (4 KB) in flight.  The G query heads of the group
// are kept in registers and share each key.  Warps merge their running (m, l, o) through
// shared memory; with several key splits the last CTA of a (stream, KV head) to finish
// combines the partial triples -- no CTA ever waits for another.
#include "vs_common.cuh"

namespace vs {

namespace {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int GMAX = 8;
constexpr int kBatch = 4;     // keys a lane group loads before computing

template <int D>
__global__ void __launch_bounds__(kDecThreads) decode_attn_kernel(DecodeArgs a, BatchParams bp) {
  constexpr int LPK = D / 8;            // lanes that share one key row (16 bytes each)
  constexpr int KPW = 32 / LPK;         // lane groups (keys in parallel) per warp
  __shared__ float st_m[kDecWarps][GMAX];
  __shared__ float st_l[kDecWarps][GMAX];
  __shared__ float st_o[kDecWarps][GMAX][D];
  __shared__ float sp_w[DEC_SPLIT_MAX][GMAX];
  __shared__ int is_last;

  pdl_wait();
  pdl_launch_dependents();
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

  const size_t hoff = (size_t)sid * a.Hkv + hkv;
  const bf16* pk = a.prefix_k + hoff * a.maxP * D + li * 8;
  const bf16* pv = a.prefix_v + hoff * a.maxP * D + li * 8;
  const bf16* bk = a.bank_k + hoff * a.slots * D + li * 8;
  const bf16* bv = a.bank_v + hoff * a.slots * D + li * 8;
  const bf16* tk = a.tail_k + hoff * a.maxT * D + li * 8;
  const bf16* tv = a.tail_v + hoff * a.maxT * D + li * 8;

  // query (bf16 hi + lo pair) of the G heads, pre-scaled into the log2 domain
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

  // keys of this CTA are dealt to (warp, lane group) round-robin, kBatch at a time
  constexpr int kStride = kDecWarps * KPW;
  for (int wbase = begin + warp * KPW; wbase < end; wbase += kBatch * kStride) {   // uniform over the warp
    const int base = wbase + sub;
    uint4 kr[kBatch], vr[kBatch];
    bool act[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int v = base + u * kStride;
      act[u] = v < end;
      const bf16* kp = pk; const bf16* vp = pv;
      if (act[u]) {
        if (v < P) { kp = pk + (size_t)v * D; vp = pv + (size_t)v * D; }
        else if (v < P + NB) {
          const int slot = v - P;
          act[u] = slot != free_slot;                    // the slot being refilled holds no carrier
          kp = bk + (size_t)slot * D; vp = bv + (size_t)slot * D;
        } else { kp = tk + (size_t)(v - P - NB) * D; vp = tv + (size_t)(v - P - NB) * D; }
      }
      kr[u] = act[u] ? *reinterpret_cast<const uint4*>(kp) : make_uint4(0, 0, 0, 0);
      vr[u] = act[u] ? *reinterpret_cast<const uint4*>(vp) : make_uint4(0, 0, 0, 0);
    }
    float s[kBatch][GMAX];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      float kf[8];
      const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kr[u]);
#pragma unroll
      for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(k2[i]); kf[2 * i] = f.x; kf[2 * i + 1] = f.y; }
#pragma unroll
      for (int g = 0; g < GMAX; ++g) {
        float d = 0.f;
        if (g < G) {
#pragma unroll
          for (int i = 0; i < 8; ++i) d = fmaf(q[g][i], kf[i], d);
#pragma unroll
          for (int off = LPK / 2; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
        }
        s[u][g] = act[u] ? d : -INFINITY;
      }
    }
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
      if (g < G) {
        float mx = m[g];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) mx = fmaxf(mx, s[u][g]);
        if (mx > -INFINITY) {
          const float sc = exp2f(m[g] - mx);             // exp2f(-inf) = 0 on the first keys
          l[g] *= sc;
#pragma unroll
          for (int i = 0; i < 8; ++i) o[g][i] *= sc;
          m[g] = mx;
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const float p = exp2f(s[u][g] - mx);
            l[g] += p;
            const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vr[u]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 f = __bfloat1622float2(v2[i]);
              o[g][2 * i] = fmaf(p, f.x, o[g][2 * i]);
              o[g][2 * i + 1] = fmaf(p, f.y, o[g][2 * i + 1]);
            }
          }
        }
      }
    }
  }

  // lane groups of a warp merge by shuffles (they own the same dims of different keys)
#pragma unroll
  for (int off = LPK; off < 32; off <<= 1) {
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
      if (g < G) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m[g], off);
        const float l2 = __shfl_xor_sync(0xffffffffu, l[g], off);
        const float mn = fmaxf(m[g], m2);
        const float w1 = (m[g] == -INFINITY) ? 0.f : exp2f(m[g] - mn);
        const float w2 = (m2 == -INFINITY) ? 0.f : exp2f(m2 - mn);
        l[g] = l[g] * w1 + l2 * w2;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float o2 = __shfl_xor_sync(0xffffffffu, o[g][i], off);
          o[g][i] = o[g][i] * w1 + o2 * w2;
        }
        m[g] = mn;
      }
    }
  }
  if (sub == 0) {
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
      if (g < G) {
        if (li == 0) { st_m[warp][g] = m[g]; st_l[warp][g] = l[g]; }
#pragma unroll
        for (int i = 0; i < 8; ++i) st_o[warp][g][li * 8 + i] = o[g][i];
      }
    }
  }
  __syncthreads();

  // warps -> CTA
  const bool direct = a.nsplit == 1;
  float* part = a.partials + (((size_t)split * bp.n_active + b) * a.Hq + (size_t)hkv * G) * (D + 2);
  for (int idx = threadIdx.x; idx < G * D; idx += kDecThreads) {
    const int g = idx / D, c = idx - g * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, st_m[w][g]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float wt = (st_m[w][g] == -INFINITY) ? 0.f : exp2f(st_m[w][g] - M);
      L += st_l[w][g] * wt;
      O += st_o[w][g][c] * wt;
    }
    if (direct) {
      const float val = (L > 0.f) ? O / L : 0.f;
      const size_t off = (size_t)b * a.Hq * D + (size_t)(hkv * G + g) * D + c;
      if (a.out_fp32) static_cast<float*>(a.out)[off] = val;
      else static_cast<bf16*>(a.out)[off] = __float2bfloat16_rn(val);
      if (a.h_out != nullptr) a.h_out[off] = __float2bfloat16_rn(__bfloat162float(a.h_in[off]) + val);
    } else {
      part[(size_t)g * (D + 2) + c] = O;
      if (c == 0) { part[(size_t)g * (D + 2) + D] = M; part[(size_t)g * (D + 2) + D + 1] = L; }
    }
  }
  if (direct) return;

  // last CTA of this (stream, KV head) combines the splits
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(a.tickets + sid * a.Hkv + hkv, 1) == a.nsplit - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // weights of the splits per head, then every output element with all its loads in flight
  if (threadIdx.x < G) {
    const int g = threadIdx.x, qh = hkv * G + g;
    float ms[DEC_SPLIT_MAX], ls[DEC_SPLIT_MAX];
    float M = -INFINITY;
#pragma unroll
    for (int s = 0; s < DEC_SPLIT_MAX; ++s) {
      if (s < a.nsplit) {
        const float* pp = a.partials + (((size_t)s * bp.n_active + b) * a.Hq + qh) * (D + 2);
        ms[s] = __ldcg(pp + D); ls[s] = __ldcg(pp + D + 1);
        M = fmaxf(M, ms[s]);
      }
    }
    float L = 0.f;
#pragma unroll
    for (int s = 0; s < DEC_SPLIT_MAX; ++s) {
      if (s < a.nsplit) {
        const float wt = (ms[s] == -INFINITY) ? 0.f : exp2f(ms[s] - M);
        L += ls[s] * wt;
        sp_w[s][g] = wt;
      }
    }
    const float inv = (L > 0.f) ? 1.f / L : 0.f;
#pragma unroll
    for (int s = 0; s < DEC_SPLIT_MAX; ++s) if (s < a.nsplit) sp_w[s][g] *= inv;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < G * D; idx += kDecThreads) {
    const int g = idx / D, c = idx - g * D;
    const int qh = hkv * G + g;
    float v[DEC_SPLIT_MAX];
#pragma unroll
    for (int s = 0; s < DEC_SPLIT_MAX; ++s)
      v[s] = (s < a.nsplit) ? __ldcg(a.partials + (((size_t)s * bp.n_active + b) * a.Hq + qh) * (D + 2) + c) : 0.f;
    float val = 0.f;
#pragma unroll
    for (int s = 0; s < DEC_SPLIT_MAX; ++s) if (s < a.nsplit) val = fmaf(v[s], sp_w[s][g], val);
    const size_t off = (size_t)b * a.Hq * D + (size_t)qh * D + c;
    if (a.out_fp32) static_cast<float*>(a.out)[off] = val;
    else static_cast<bf16*>(a.out)[off] = __float2bfloat16_rn(val);
    if (a.h_out != nullptr) a.h_out[off] = __float2bfloat16_rn(__bfloat162float(a.h_in[off]) + val);
  }
  if (threadIdx.x == 0) a.tickets[sid * a.Hkv + hkv] = 0;
}

}  // namespace

cudaError_t launch_decode_attention(const DecodeArgs& a, const BatchParams& bp, cudaStream_t st) {
  if (a.nsplit < 1 || a.nsplit > DEC_SPLIT_MAX || a.Hq / a.Hkv > GMAX) return cudaErrorInvalidValue;
  dim3 grid(a.nsplit, a.Hkv, bp.n_active);
  if (a.D == 128) return launch_pdl(decode_attn_kernel<128>, grid, dim3(kDecThreads), 0, st, a, bp);
  if (a.D == 64) return launch_pdl(decode_attn_kernel<64>, grid, dim3(kDecThreads), 0, st, a, bp);
  return cudaErrorInvalidValue;
}

}  // namespace vs
