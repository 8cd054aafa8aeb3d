// QKV projection of a text step of one to four token rows (Eq. 1 with a handful of rows:
// decode, Section 3.3's answer tokens).  With so few rows the projection is a matrix-vector
// product bound by reading W once, not a tensor-core contraction.  Every CTA owns 32 rows of
// W ([E_out, d] bf16, row-major) and streams them through a ring of shared-memory stages filled
// by 16-byte asynchronous copies (a stage = 256 elements of all 32 rows, 16 KiB; eight stages,
// so up to 112 KiB per SM are in flight whatever the registers hold).  The products are formed by
// the warp-level tensor-core instruction (mma.sync m16n8k16, bf16 x bf16 -> fp32) with the token rows
// as its 8-column operand: not for its arithmetic rate but for its instruction count -- unpacking
// bf16 pairs and multiply-adding them one by one on the CUDA cores cost some 95 instructions per warp
// and stage and made the loop issue-bound; this way it is ten.
//
// A CTA's 32 rows are 16 rotation pairs (k, k + D/2) of one head, so the epilogue has both
// elements of a pair at hand: RMSNorm row scale, bias, RoPE (the angle in fp64 from the token's
// position, as the table kernel computes it), bf16 rounding, the query's hi + lo pair, and the
// write of K/V rows to the prefix or to the turn's tail.  RMSNorm is done here too (every CTA
// holds the token rows, so each works out the row scale and, with a gain vector, bf16(h * gain)
// itself): such a step launches no statistics kernel.
//
// W never changes while the stream handle lives, so the ring is filled and the rotation angles
// are worked out before the wait on the stream's earlier kernels; the token rows are read after
// it.
#include "vs_common.cuh"

namespace vs {

namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerCta = 32;     // 16 rotation pairs
constexpr int kStageElems = 256;    // K elements of every row in one stage
constexpr int kStageBytes = kRowsPerCta * kStageElems * 2;   // 16 KiB
constexpr int kStages = 8;

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int R>   // token rows held (1, 2 or 4)
__global__ void __launch_bounds__(kThreads, 2) qkv_gemv_kernel(const bf16* __restrict__ W, const bf16* __restrict__ x,
                                                            ProjectionOut o, BatchParams bp, int rows, int d, int l2_ahead) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  // carve: ring [kStages][32 rows][512 B] | token rows [R][d] bf16 | partial results [4][R][32] | row scales [R] | partial sums [R][8]
  uint4* xs = reinterpret_cast<uint4*>(smem_raw + kStages * kStageBytes);
  float* ysp = reinterpret_cast<float*>(smem_raw + kStages * kStageBytes + (size_t)R * d * 2);   // [4 K quarters][R][32]
  float* rs = ysp + 4 * R * kRowsPerCta;
  float* red = rs + R;
  const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem_raw));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int D = o.D, half = D >> 1;
  const int blocks_per_head = half / 16;
  const int hs = (int)blockIdx.x / blocks_per_head;                     // head slot: Q heads, K heads, V heads
  const int pb = (int)blockIdx.x - hs * blocks_per_head;
  const int n_stage_total = d / kStageElems;
  const int chunks_per_row = d >> 3;

  // copies of a stage: thread t moves the 16-byte chunks t, t + 256, ... of the stage's 1024;
  // chunk index -> (local row lr = idx / 32, column idx % 32); lr -> pair lr & 15, second element
  // of the pair if lr >= 16
  const bf16* csrc[4];
  uint32_t cdst[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int idx = tid + kThreads * q;
    const int lr = idx >> 5, c = idx & 31;
    const int f = hs * D + pb * 16 + (lr & 15) + (lr >> 4) * half;
    csrc[q] = W + (size_t)f * d + c * 8;
    // rows 2j and 2j + 1 are read side by side by a quarter warp: bit 2 of the chunk index is flipped in odd
    // rows so that the two rows' 64-byte pieces fall into different banks
    cdst[q] = (uint32_t)(lr * (kStageElems * 2) + ((c ^ ((lr & 1) << 2)) * 16));
  }
  auto issue_stage = [&](int i) {
    if (i < n_stage_total) {
      const uint32_t slot = ring + (uint32_t)(i % kStages) * kStageBytes;
#pragma unroll
      for (int q = 0; q < 4; ++q) cp_async16(slot + cdst[q], csrc[q] + (size_t)i * kStageElems);
    }
    cp_async_commit();                                                  // one group per stage, empty or not
  };
  for (int i = 0; i < kStages - 1; ++i) issue_stage(i);                 // W is constant: no need to wait for it
  // what the ring cannot hold yet of this CTA's 32 rows (a contiguous piece of each row) is asked
  // into L2 now, so that all of the layer's matrix is on its way from HBM while the kernel ahead
  // of this one -- the attention of the layer before -- still runs
  if (l2_ahead && tid < kRowsPerCta && n_stage_total > kStages - 1) {
    const int f = hs * D + pb * 16 + (tid & 15) + (tid >> 4) * half;
    prefetch_l2_bulk(W + (size_t)f * d + (size_t)(kStages - 1) * kStageElems,
                     (uint32_t)(n_stage_total - (kStages - 1)) * kStageElems * 2);
  }

  // finishing threads: (token row r, pair p); the rotation depends on the parameters alone
  const int fr = tid >> 4, fp = tid & 15;
  const int k0 = pb * 16 + fp;                                          // index inside the half head
  const bool finisher = fr < R && fr < rows;
  const bool rotate = hs < o.Hq + o.Hkv;
  float rc = 1.f, rsn = 0.f;
  int fb = 0, ftt = 0;
  if (finisher) {
    fb = fr / bp.rows_per_stream; ftt = fr - fb * bp.rows_per_stream;
    if (rotate) {
      double sn, cs;
      sincos((double)(bp.pos_base[fb] + ftt) * o.inv_freq[k0], &sn, &cs);
      rc = (float)cs; rsn = (float)sn;
    }
  }

  VS_STAMP(bp, 4, 0);
  pdl_wait();                       // earlier kernels of the stream have completed
  pdl_launch_dependents();
  VS_STAMP(bp, 4, 1);

  // token rows -> shared memory; with RMSNorm: sum of squares of the raw row, and the row times
  // the gain vector (rounded to bf16, as the statistics kernel stores it) in place of the row
  {
    float ss[R];
#pragma unroll
    for (int r = 0; r < R; ++r) ss[r] = 0.f;
    for (int c = tid; c < chunks_per_row; c += kThreads) {
      uint4 g4 = make_uint4(0u, 0u, 0u, 0u);
      if (o.norm_inline && o.norm_gain != nullptr) g4 = reinterpret_cast<const uint4*>(o.norm_gain)[c];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        uint4 v = (r < rows) ? reinterpret_cast<const uint4*>(x)[r * chunks_per_row + c] : make_uint4(0u, 0u, 0u, 0u);
        if (o.norm_inline) {
          const uint32_t* vw = reinterpret_cast<const uint32_t*>(&v);
          const uint32_t* gw = reinterpret_cast<const uint32_t*>(&g4);
          uint32_t ow[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float a0 = bf_lo(vw[k]), a1 = bf_hi(vw[k]);
            ss[r] += a0 * a0 + a1 * a1;
            const __nv_bfloat162 p = __floats2bfloat162_rn(a0 * bf_lo(gw[k]), a1 * bf_hi(gw[k]));
            ow[k] = *reinterpret_cast<const uint32_t*>(&p);
          }
          if (o.norm_gain != nullptr) v = make_uint4(ow[0], ow[1], ow[2], ow[3]);
        }
        xs[r * chunks_per_row + c] = v;
      }
    }
    if (o.norm_inline) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float v = ss[r];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0) red[r * 8 + warp] = v;
      }
    }
  }
  __syncthreads();
  if (o.norm_inline && tid < R) {
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += red[tid * 8 + i];
    rs[tid] = rsqrtf(tot / (float)d + o.norm_eps);
  }

  // Warp w owns the 16-row tile w & 1 (first or second elements of the CTA's rotation pairs) and the two 32-element
  // K blocks 2 * (w >> 1), + 1 of every stage.  Inside a block, lane (g, t) = (lane / 4, lane % 4) reads the 16 bytes
  // k = 8t .. 8t + 7 of weight rows g and g + 8 and of token row g: the first 8 bytes feed one MMA, the last 8 the
  // next -- a permutation of K that the weights and the tokens share, which a dot product does not see.
  const int mt = warp & 1, kg = warp >> 1;
  const int g = lane >> 2, t4 = lane & 3;
  const uint32_t ring_u = ring;
  const uint32_t a_row0 = (uint32_t)((mt * 16 + g) * (kStageElems * 2)), a_row1 = a_row0 + 8u * (kStageElems * 2);
  const uint32_t sw0 = (uint32_t)(((mt * 16 + g) & 1) << 2);                // rows g and g + 8 have the same parity
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int i = 0; i < n_stage_total; ++i) {
    cp_async_wait<kStages - 2>();   // this thread's copies of stage i have landed
    __syncthreads();                // everyone's have, and everyone is done with stage i - 1
    issue_stage(i + kStages - 1);   // into the slot stage i - 1 occupied
    const uint32_t slot = ring_u + (uint32_t)(i % kStages) * kStageBytes;
#pragma unroll
    for (int kb2 = 0; kb2 < 2; ++kb2) {
      const int kb = kg * 2 + kb2;                                          // 32-element block inside the stage
      const uint32_t chunk = (uint32_t)(kb * 4 + t4);
      uint32_t a0[4], a1[4];
      asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(a0[0]), "=r"(a0[1]), "=r"(a0[2]), "=r"(a0[3])
                   : "r"(slot + a_row0 + ((chunk ^ sw0) << 4)));
      asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(a1[0]), "=r"(a1[1]), "=r"(a1[2]), "=r"(a1[3])
                   : "r"(slot + a_row1 + ((chunk ^ sw0) << 4)));
      uint4 xv = make_uint4(0u, 0u, 0u, 0u);
      if (g < R) xv = xs[g * chunks_per_row + i * 32 + (int)chunk];
      asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                   : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3])
                   : "r"(a0[0]), "r"(a1[0]), "r"(a0[1]), "r"(a1[1]), "r"(xv.x), "r"(xv.y));
      asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                   : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3])
                   : "r"(a0[2]), "r"(a1[2]), "r"(a0[3]), "r"(a1[3]), "r"(xv.z), "r"(xv.w));
    }
  }
  cp_async_wait<0>();
  // accumulator: acc[0], acc[1] = (row g, tokens 2t, 2t + 1), acc[2], acc[3] = (row g + 8, same tokens);
  // the four warps that share a row tile leave their parts side by side, the finishing threads add them
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int tok = 2 * t4 + j;
    if (tok < R) {
      ysp[(kg * R + tok) * kRowsPerCta + mt * 16 + g] = acc[j];
      ysp[(kg * R + tok) * kRowsPerCta + mt * 16 + g + 8] = acc[2 + j];
    }
  }
  __syncthreads();

  if (finisher) {
    const int row = fr;
    float x1 = 0.f, x2 = 0.f;
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {                       // the K quarters of the stage, in a fixed order
      x1 += ysp[(k4 * R + row) * kRowsPerCta + fp];
      x2 += ysp[(k4 * R + row) * kRowsPerCta + 16 + fp];
    }
    const int f1 = hs * D + k0, f2 = f1 + half;
    // RMSNorm's row scale commutes with the projection
    float rsc = 1.f;
    if (o.norm_inline) rsc = rs[row];
    else if (o.row_ss != nullptr) {
      float tot = 0.f;
      for (int i = 0; i < o.ss_parts; ++i) tot += o.row_ss[(size_t)row * o.ss_parts + i];
      rsc = rsqrtf(tot / (float)d + o.norm_eps);
    }
    const float b1 = (o.bias != nullptr) ? __bfloat162float(o.bias[f1]) : 0.f;
    const float b2 = (o.bias != nullptr) ? __bfloat162float(o.bias[f2]) : 0.f;
    x1 = fmaf(x1, rsc, b1); x2 = fmaf(x2, rsc, b2);
    if (rotate) {
      const float y1 = x1 * rc - x2 * rsn;
      const float y2 = x2 * rc + x1 * rsn;
      x1 = y1; x2 = y2;
    }
    const bf16 o1 = __float2bfloat16_rn(x1), o2 = __float2bfloat16_rn(x2);
    if (hs < o.Hq) {
      // the query stays inside the step: kept as a bf16 pair (hi + lo)
      const size_t qo = (size_t)row * o.Hq * D + (size_t)hs * D + k0;
      if (VS_STORE_OK(bp, DR_Q, o.q + qo, 2) && VS_STORE_OK(bp, DR_Q, o.q + qo + half, 2) &&
          VS_STORE_OK(bp, DR_Q_LO, o.q_lo + qo, 2) && VS_STORE_OK(bp, DR_Q_LO, o.q_lo + qo + half, 2)) {
        o.q[qo] = o1; o.q[qo + half] = o2;
        o.q_lo[qo] = __float2bfloat16_rn(x1 - __bfloat162float(o1));
        o.q_lo[qo + half] = __float2bfloat16_rn(x2 - __bfloat162float(o2));
      }
    } else {
      const bool is_k = hs < o.Hq + o.Hkv;
      const int hkv = is_k ? hs - o.Hq : hs - o.Hq - o.Hkv;
      bf16* f = (is_k ? o.kf : o.vf) + (size_t)row * o.Hkv * D + (size_t)hkv * D + k0;
      if (VS_STORE_OK(bp, is_k ? DR_KF : DR_VF, f, 2) && VS_STORE_OK(bp, is_k ? DR_KF : DR_VF, f + half, 2)) { f[0] = o1; f[half] = o2; }
      const int sid = bp.stream_id[fb];
      const int tb = (o.mode == 1) ? bp.prefix_len[fb] : bp.text_len[fb];
      bf16* dst = (is_k ? o.text_k : o.text_v) + (((size_t)sid * o.Hkv + hkv) * o.text_cap + tb + ftt) * D + k0;
      const int dreg = (o.mode == 1) ? (is_k ? DR_PREFIX_K : DR_PREFIX_V) : (is_k ? DR_TAIL_K : DR_TAIL_V);
      if (VS_STORE_OK(bp, dreg, dst, 2) && VS_STORE_OK(bp, dreg, dst + half, 2)) { dst[0] = o1; dst[half] = o2; }
    }
  }
  VS_STAMP(bp, 4, 15);
}

}  // namespace

static size_t gemv_smem_bytes(int R, int d) {
  return (size_t)kStages * kStageBytes + (size_t)R * d * 2 + (size_t)4 * R * kRowsPerCta * 4 + (size_t)R * 4 + (size_t)R * 8 * 4;
}

bool qkv_gemv_supported(const ProjectionOut& o, int rows, int d) {
  if (rows < 1 || rows > 4 || (o.mode != 1 && o.mode != 2)) return false;   // text steps only
  if ((d & 255) != 0 || (o.D != 64 && o.D != 128)) return false;
  return gemv_smem_bytes(4, d) <= 200 * 1024;
}

cudaError_t qkv_gemv_init() {
  cudaError_t e = cudaFuncSetAttribute(qkv_gemv_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(qkv_gemv_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(qkv_gemv_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  return e;
}

cudaError_t launch_qkv_gemv(const bf16* W, const bf16* x, const ProjectionOut& o, const BatchParams& bp, int rows, int E_out,
                            int d, bool l2_ahead, cudaStream_t st) {
  if (!qkv_gemv_supported(o, rows, d) || o.inv_freq == nullptr) return cudaErrorInvalidValue;
  const dim3 grid((E_out / o.D) * ((o.D / 2) / 16));
  const int R = rows == 1 ? 1 : (rows == 2 ? 2 : 4);
  const size_t smem = gemv_smem_bytes(R, d);
  const int ahead = l2_ahead ? 1 : 0;
  if (R == 1) return launch_pdl(qkv_gemv_kernel<1>, grid, dim3(kThreads), smem, st, W, x, o, bp, rows, d, ahead);
  if (R == 2) return launch_pdl(qkv_gemv_kernel<2>, grid, dim3(kThreads), smem, st, W, x, o, bp, rows, d, ahead);
  return launch_pdl(qkv_gemv_kernel<4>, grid, dim3(kThreads), smem, st, W, x, o, bp, rows, d, ahead);
}

}  // namespace vs
