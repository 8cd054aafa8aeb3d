// QKV projection of a text step of one to four token rows (Eq. 1 with a handful of rows:
// decode, Section 3.3's answer tokens).  With so few rows the projection is a matrix-vector
// product bound by reading W once, not a tensor-core contraction: every CTA streams 32 rows of
// W ([E_out, d] bf16, row-major) with 16-byte loads, each warp owning four rows and each lane a
// 16-byte column of them, fp32 accumulation, a shuffle reduction per row.
//
// A CTA's 32 rows are 16 rotation pairs (k, k + D/2) of one head, so the epilogue has both
// elements of a pair at hand: RMSNorm row scale, bias, RoPE (the angle in fp64 from the token's
// position, as the table kernel computes it), bf16 rounding, the query's hi + lo pair, and the
// write of K/V rows to the prefix or to the turn's tail.
//
// W never changes while the stream handle lives, so the first batch of W loads and the rotation
// angles are issued before the wait on the stream's earlier kernels; the token rows are read
// after it.
#include "vs_common.cuh"

namespace vs {

namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerCta = 32;     // 16 rotation pairs
constexpr int kU = 2;               // 16-byte chunks per W row in one batch of loads (two batches in flight)

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float dot8(const uint4& w, const uint4& x, float acc) {
  acc = fmaf(bf_lo(w.x), bf_lo(x.x), acc); acc = fmaf(bf_hi(w.x), bf_hi(x.x), acc);
  acc = fmaf(bf_lo(w.y), bf_lo(x.y), acc); acc = fmaf(bf_hi(w.y), bf_hi(x.y), acc);
  acc = fmaf(bf_lo(w.z), bf_lo(x.z), acc); acc = fmaf(bf_hi(w.z), bf_hi(x.z), acc);
  acc = fmaf(bf_lo(w.w), bf_lo(x.w), acc); acc = fmaf(bf_hi(w.w), bf_hi(x.w), acc);
  return acc;
}

template <int R>   // token rows held (1, 2 or 4)
__global__ void __launch_bounds__(kThreads, 2) qkv_gemv_kernel(const bf16* __restrict__ W, const bf16* __restrict__ x,
                                                            ProjectionOut o, BatchParams bp, int rows, int d) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  uint4* xs = reinterpret_cast<uint4*>(smem_raw);                       // [R][d / 8]
  float* ys = reinterpret_cast<float*>(smem_raw + (size_t)R * d * 2);   // [R][32]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int D = o.D, half = D >> 1;
  const int blocks_per_head = half / 16;
  const int hs = (int)blockIdx.x / blocks_per_head;                     // head slot: Q heads, K heads, V heads
  const int pb = (int)blockIdx.x - hs * blocks_per_head;
  const int n_chunks = d >> 8;                                          // 16-byte chunks per lane and row
  const int chunks_per_row = d >> 3;

  // the warp's four rows of W: local row lr -> pair lr & 15, second element of the pair if lr >= 16
  const uint4* wrow[4];
#pragma unroll
  for (int rr = 0; rr < 4; ++rr) {
    const int lr = warp * 4 + rr;
    const int f = hs * D + pb * 16 + (lr & 15) + (lr >> 4) * half;
    wrow[rr] = reinterpret_cast<const uint4*>(W + (size_t)f * d) + lane;
  }
  auto load_batch = [&](uint4 (&buf)[4][kU], int i0) {
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int i = i0 + u;
#pragma unroll
      for (int rr = 0; rr < 4; ++rr)
        buf[rr][u] = (i < n_chunks) ? __ldg(wrow[rr] + i * 32) : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  uint4 bufA[4][kU], bufB[4][kU];
  load_batch(bufA, 0);                                                  // W is constant: no need to wait for it

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

  pdl_wait();                       // earlier kernels of the stream have completed
  pdl_launch_dependents();

  for (int idx = tid; idx < R * chunks_per_row; idx += kThreads) {
    const int r = idx / chunks_per_row;
    xs[idx] = (r < rows) ? reinterpret_cast<const uint4*>(x)[idx] : make_uint4(0u, 0u, 0u, 0u);
  }
  __syncthreads();

  float acc[4][R];
#pragma unroll
  for (int rr = 0; rr < 4; ++rr)
#pragma unroll
    for (int r = 0; r < R; ++r) acc[rr][r] = 0.f;
  auto consume = [&](const uint4 (&buf)[4][kU], int i0) {
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int i = i0 + u;
      if (i < n_chunks) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const uint4 xv = xs[r * chunks_per_row + i * 32 + lane];
#pragma unroll
          for (int rr = 0; rr < 4; ++rr) acc[rr][r] = dot8(buf[rr][u], xv, acc[rr][r]);
        }
      }
    }
  };
  for (int i0 = 0; i0 < n_chunks; i0 += 2 * kU) {
    load_batch(bufB, i0 + kU);
    consume(bufA, i0);
    load_batch(bufA, i0 + 2 * kU);
    consume(bufB, i0 + kU);
  }
#pragma unroll
  for (int rr = 0; rr < 4; ++rr)
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float v = acc[rr][r];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (lane == 0) ys[r * kRowsPerCta + warp * 4 + rr] = v;
    }
  __syncthreads();

  if (finisher) {
    const int row = fr;
    float x1 = ys[row * kRowsPerCta + fp], x2 = ys[row * kRowsPerCta + 16 + fp];
    const int f1 = hs * D + k0, f2 = f1 + half;
    const float rsc = (o.row_scale != nullptr) ? o.row_scale[row] : 1.f;   // RMSNorm's row scale commutes with the projection
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
      o.q[qo] = o1; o.q[qo + half] = o2;
      o.q_lo[qo] = __float2bfloat16_rn(x1 - __bfloat162float(o1));
      o.q_lo[qo + half] = __float2bfloat16_rn(x2 - __bfloat162float(o2));
    } else {
      const bool is_k = hs < o.Hq + o.Hkv;
      const int hkv = is_k ? hs - o.Hq : hs - o.Hq - o.Hkv;
      bf16* f = (is_k ? o.kf : o.vf) + (size_t)row * o.Hkv * D + (size_t)hkv * D + k0;
      f[0] = o1; f[half] = o2;
      const int sid = bp.stream_id[fb];
      const int tb = (o.mode == 1) ? bp.prefix_len[fb] : bp.text_len[fb];
      bf16* dst = (is_k ? o.text_k : o.text_v) + (((size_t)sid * o.Hkv + hkv) * o.text_cap + tb + ftt) * D + k0;
      dst[0] = o1; dst[half] = o2;
    }
  }
}

}  // namespace

bool qkv_gemv_supported(const ProjectionOut& o, int rows, int d) {
  if (rows < 1 || rows > 4 || o.mode == 0) return false;                // text steps only
  if ((d & 255) != 0 || (o.D != 64 && o.D != 128)) return false;
  return (size_t)4 * d * 2 + 4 * kRowsPerCta * 4 <= 48 * 1024;          // fits the default dynamic shared memory
}

cudaError_t launch_qkv_gemv(const bf16* W, const bf16* x, const ProjectionOut& o, const BatchParams& bp, int rows, int E_out,
                            int d, cudaStream_t st) {
  if (!qkv_gemv_supported(o, rows, d) || o.inv_freq == nullptr) return cudaErrorInvalidValue;
  const dim3 grid((E_out / o.D) * ((o.D / 2) / 16));
  const int R = rows == 1 ? 1 : (rows == 2 ? 2 : 4);
  const size_t smem = (size_t)R * d * 2 + (size_t)R * kRowsPerCta * 4;
  if (R == 1) return launch_pdl(qkv_gemv_kernel<1>, grid, dim3(kThreads), smem, st, W, x, o, bp, rows, d);
  if (R == 2) return launch_pdl(qkv_gemv_kernel<2>, grid, dim3(kThreads), smem, st, W, x, o, bp, rows, d);
  return launch_pdl(qkv_gemv_kernel<4>, grid, dim3(kThreads), smem, st, W, x, o, bp, rows, d);
}

}  // namespace vs
