// Decode attention (Section 3.3, decoding phase; Eq. 1 per head with grouped KV heads): one
// query token per stream attends over [prompt prefix | carrier bank | text of the turn].  No
// visual-token K/V exists at this point -- only carriers.
//
// grid = (key splits, query heads, streams), 256 threads.  A group of D/8 lanes owns one key
// row and reads it with 128-bit loads; every lane issues the K and V loads of eight keys before
// it uses any of them, so a warp has 16 key rows (8 KB) in flight.  Warps merge their running
// (m, l, o) by shuffles and through shared memory.  The key splits of one (stream, query head)
// form a thread-block cluster (1, 2, 4 or 8 CTAs): every CTA writes its partial triple into rank 0's
// shared memory (distributed shared memory) and arrives at the cluster's hardware barrier; rank 0
// alone waits there, combines and writes the row -- no global scratch, no atomics, no polling; the
// co-scheduled cluster is what guarantees that the barrier completes.
#include "vs_common.cuh"

namespace vs {

namespace {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kBatch = 8;     // keys a lane group loads before computing
constexpr int kMaxCluster = 8;  // portable cluster size: most key splits of one (stream, query head)

__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_shared_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_shared_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// One CTA = one query head x one key split x one stream.  The heads of a KV group read the
// same K/V rows from L2; spreading them over CTAs keeps every SM's instruction stream short,
// which is what bounds this kernel (a few hundred keys of 256 bytes each).
template <int D>
__global__ void __launch_bounds__(kDecThreads, 2) decode_attn_kernel(DecodeArgs a, BatchParams bp) {
  constexpr int LPK = D / 8;            // lanes that share one key row (16 bytes each)
  constexpr int KPW = 32 / LPK;         // lane groups (keys in parallel) per warp
  __shared__ float st_m[kDecWarps];
  __shared__ float st_l[kDecWarps];
  __shared__ float st_o[kDecWarps][D];
  __shared__ float peer_o[kMaxCluster][D];     // rank 0 only: the partial triples its peers (and itself) leave here
  __shared__ float peer_ml[kMaxCluster][2];

  // what follows from the parameters alone comes before the wait on the stream's earlier kernels
  const int split = blockIdx.x, qh = blockIdx.y, b = blockIdx.z;
  const int sid = bp.stream_id[b];
  const int hkv = qh / (a.Hq / a.Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPK, li = lane % LPK;
  const int count = bp.count[b];
  const bool bank_full = (a.M > 0 && count == a.M);
  // first phase of the cluster's barrier: "this CTA runs", so that nobody writes into the shared memory of a
  // CTA that has not started; everyone arrives here and waits only just before its one remote write
  if (a.nsplit > 1) cluster_arrive_relaxed();

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

  // Only the step's own token (the last key) was written by the kernel just before this one; every
  // other key, and the bank's metadata, date from earlier steps, whose kernels had completed before
  // that kernel let this one start.  So the first pass of K/V rows is fetched before the wait.
  // The slot being refilled holds no carrier: its key is fetched like any other (the row exists)
  // and masked when the scores are formed.
  const int hole = bank_full ? P + a.meta[sid].free_slot : -1;
  const int own_v = Lv - 1;
  constexpr int kStride = kDecWarps * KPW;
  // late == false: every key of the pass but the step's own; late == true: the step's own only
  auto load_pass = [&](int wbase, uint4 (&kr)[kBatch], uint4 (&vr)[kBatch], bool late) {
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int v = wbase + sub + u * kStride;
      if (v < end && ((v == own_v) == late)) {
        const bf16* kp; const bf16* vp;
        if (v < P) { kp = pk + (size_t)v * D; vp = pv + (size_t)v * D; }
        else if (v < P + NB) { kp = bk + (size_t)(v - P) * D; vp = bv + (size_t)(v - P) * D; }
        else { kp = tk + (size_t)(v - P - NB) * D; vp = tv + (size_t)(v - P - NB) * D; }
        kr[u] = *reinterpret_cast<const uint4*>(kp);
        vr[u] = *reinterpret_cast<const uint4*>(vp);
      } else if (!late) {
        kr[u] = make_uint4(0, 0, 0, 0); vr[u] = make_uint4(0, 0, 0, 0);
      }
    }
  };
  const int wbase0 = begin + warp * KPW;                 // keys are dealt to (warp, lane group) round-robin
  uint4 kr0[kBatch], vr0[kBatch];
  load_pass(wbase0, kr0, vr0, false);

  VS_STAMP(bp, 5, 0);
  pdl_wait();
  pdl_launch_dependents();
  VS_STAMP(bp, 5, 1);
  // the step's own key and the query are both fresh: their loads go out together
  if (wbase0 < end) load_pass(wbase0, kr0, vr0, true);

  // this lane's 8 dims of the query (bf16 hi + lo pair), pre-scaled into the log2 domain
  float q[8];
  {
    const size_t qo = (size_t)b * a.Hq * D + (size_t)qh * D + li * 8;
    const uint4 raw = *reinterpret_cast<const uint4*>(a.q + qo);
    const uint4 raw_lo = *reinterpret_cast<const uint4*>(a.q_lo + qo);
    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
    const __nv_bfloat162* l2 = reinterpret_cast<const __nv_bfloat162*>(&raw_lo);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(h2[i]);
      const float2 fl = __bfloat1622float2(l2[i]);
      q[2 * i] = (f.x + fl.x) * a.scale_log2e; q[2 * i + 1] = (f.y + fl.y) * a.scale_log2e;
    }
  }
  float m = -INFINITY, l = 0.f, o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i] = 0.f;

  auto compute_pass = [&](int wbase, const uint4 (&kr)[kBatch], const uint4 (&vr)[kBatch]) {
    float s[kBatch];
    float mx = m;
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int v = wbase + sub + u * kStride;
      const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kr[u]);
      float d = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(k2[i]);
        d = fmaf(q[2 * i], f.x, d); d = fmaf(q[2 * i + 1], f.y, d);
      }
#pragma unroll
      for (int off = LPK / 2; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
      s[u] = (v < end && v != hole) ? d : -INFINITY;
      mx = fmaxf(mx, s[u]);
    }
    if (mx > -INFINITY) {
      const float sc = exp2f(m - mx);                    // exp2f(-inf) = 0 on the first keys
      l *= sc;
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] *= sc;
      m = mx;
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const float p = exp2f(s[u] - mx);
        l += p;
        const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vr[u]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(v2[i]);
          o[2 * i] = fmaf(p, f.x, o[2 * i]);
          o[2 * i + 1] = fmaf(p, f.y, o[2 * i + 1]);
        }
      }
    }
  };
  if (wbase0 < end) compute_pass(wbase0, kr0, vr0);      // uniform over the warp
  for (int wbase = wbase0 + kBatch * kStride; wbase < end; wbase += kBatch * kStride) {
    uint4 kr[kBatch], vr[kBatch];
    load_pass(wbase, kr, vr, false);
    load_pass(wbase, kr, vr, true);
    compute_pass(wbase, kr, vr);
  }

  // lane groups of a warp merge by shuffles (they own the same dims of different keys)
#pragma unroll
  for (int off = LPK; off < 32; off <<= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
    const float l2 = __shfl_xor_sync(0xffffffffu, l, off);
    const float mn = fmaxf(m, m2);
    const float w1 = (m == -INFINITY) ? 0.f : exp2f(m - mn);
    const float w2 = (m2 == -INFINITY) ? 0.f : exp2f(m2 - mn);
    l = l * w1 + l2 * w2;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float o2 = __shfl_xor_sync(0xffffffffu, o[i], off);
      o[i] = o[i] * w1 + o2 * w2;
    }
    m = mn;
  }
  if (sub == 0) {
    if (li == 0) { st_m[warp] = m; st_l[warp] = l; }
#pragma unroll
    for (int i = 0; i < 8; ++i) st_o[warp][li * 8 + i] = o[i];
  }
  __syncthreads();

  // warps -> CTA
  const bool direct = a.nsplit == 1;
  const size_t out_off = (size_t)b * a.Hq * D + (size_t)qh * D;
  // the residual input is needed by whoever writes the row: fetched ahead of the cluster barrier
  float h_res = 0.f;
  if (a.h_out != nullptr && split == 0 && threadIdx.x < D) h_res = __bfloat162float(a.h_in[out_off + threadIdx.x]);
  float M_cta = -INFINITY, L_cta = 0.f, O_cta = 0.f;      // this CTA's partial triple (threads below D)
  if (threadIdx.x < D) {
    const int c = threadIdx.x;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, st_m[w]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float wt = (st_m[w] == -INFINITY) ? 0.f : exp2f(st_m[w] - M);
      L += st_l[w] * wt;
      O += st_o[w][c] * wt;
    }
    if (direct) {
      const float val = (L > 0.f) ? O / L : 0.f;
      if (a.out_fp32) static_cast<float*>(a.out)[out_off + c] = val;
      else static_cast<bf16*>(a.out)[out_off + c] = __float2bfloat16_rn(val);
      if (a.h_out != nullptr && VS_STORE_OK(bp, a.h_out_region, a.h_out + out_off + c, 2)) a.h_out[out_off + c] = __float2bfloat16_rn(h_res + val);
    } else {
      M_cta = M; L_cta = L; O_cta = O;
    }
  }
  if (direct) { VS_STAMP(bp, 5, 15); return; }

  // Every CTA of the cluster (the key splits of this stream and query head) leaves its partial triple in rank 0's
  // shared memory and arrives at the cluster's barrier; only rank 0 waits there, then combines what it was given.
  // The other CTAs are done: nothing of theirs is read after they exit.
  VS_STAMP(bp, 5, 4);
  cluster_wait_acquire();                           // phase 1 (every CTA of the cluster has started) -- long since complete
  if (threadIdx.x < D) {
    const int c = threadIdx.x;
    st_shared_cluster_f32(map_shared_rank(static_cast<uint32_t>(__cvta_generic_to_shared(&peer_o[split][c])), 0u), O_cta);
    if (c == 0) {
      const uint32_t ml = map_shared_rank(static_cast<uint32_t>(__cvta_generic_to_shared(&peer_ml[split][0])), 0u);
      st_shared_cluster_f32(ml, M_cta);
      st_shared_cluster_f32(ml + 4, L_cta);
    }
  }
  cluster_arrive_release();                         // phase 2: "my triple is in place"
  if (split != 0) { VS_STAMP(bp, 5, 15); return; }
  cluster_wait_acquire();
  VS_STAMP(bp, 5, 5);
  if (threadIdx.x < D) {
    const int c = threadIdx.x;
    float M = -INFINITY;
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r) if (r < a.nsplit) M = fmaxf(M, peer_ml[r][0]);
    float L = 0.f, val = 0.f;
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r) {
      if (r < a.nsplit) {
        const float wt = (peer_ml[r][0] == -INFINITY) ? 0.f : exp2f(peer_ml[r][0] - M);
        L = fmaf(peer_ml[r][1], wt, L);
        val = fmaf(peer_o[r][c], wt, val);
      }
    }
    val = (L > 0.f) ? val / L : 0.f;
    if (a.out_fp32) static_cast<float*>(a.out)[out_off + c] = val;
    else static_cast<bf16*>(a.out)[out_off + c] = __float2bfloat16_rn(val);
    if (a.h_out != nullptr && VS_STORE_OK(bp, a.h_out_region, a.h_out + out_off + c, 2)) a.h_out[out_off + c] = __float2bfloat16_rn(h_res + val);
  }
  VS_STAMP(bp, 5, 15);
}

}  // namespace

cudaError_t launch_decode_attention(const DecodeArgs& a, const BatchParams& bp, cudaStream_t st) {
  if (a.nsplit != 1 && a.nsplit != 2 && a.nsplit != 4 && a.nsplit != 8) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.nsplit, a.Hq, bp.n_active);
  cfg.blockDim = dim3(kDecThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;            // the key splits of a row are one cluster
  attr[1].val.clusterDim.x = a.nsplit; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (a.D == 128) return cudaLaunchKernelEx(&cfg, decode_attn_kernel<128>, a, bp);
  if (a.D == 64) return cudaLaunchKernelEx(&cfg, decode_attn_kernel<64>, a, bp);
  return cudaErrorInvalidValue;
}

}  // namespace vs
