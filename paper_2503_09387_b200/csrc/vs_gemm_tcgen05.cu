// QKV projection (Eq. 1: Q = X W_Q, K = X W_K, V = X W_V) on the 5th-generation tensor
// cores: tcgen05.mma with the accumulator in tensor memory, operands staged in shared
// memory by TMA, one elected thread issuing the MMAs.
//
// Orientation.  A frame brings only N + 1 (<= 256) token rows but E_out = (Hq + 2 Hkv) D
// output features (4608 at the Qwen2-7B shape), so the *features* take the MMA's M axis
// (128 weight rows per accumulator, read K-major straight from the caller's [E_out, d] matrix)
// and the *tokens* take the MMA's N axis (any multiple of 16 up to 256: 170 tokens cost 176
// columns, 3.5 % padding instead of 33 % with 128-row token tiles).
//
// Few rows (a frame, a short text step): the reduction dimension d is split over `ksplit` CTAs
// so that m_tiles * n_tiles * ksplit fills the 148 SMs.  The tile's tokens are cut into ksplit
// slices and CTA r finishes slice r: every CTA stores the other slices of its fp32 partial
// accumulator to an exchange buffer in global memory (it stays in L2), counts itself in on the
// owners' flags, and the owner of a slice, once its flag shows ksplit - 1 arrivals, adds the
// peers' partials to its own.  All CTAs of the grid are resident at once (the launch checks
// it), so the wait on the flag ends; it is bounded like every other wait.
// Many rows (a chunk of frames, a batch of streams): no K split; a CTA may hold two 128-row
// weight sub-tiles (two accumulators, 256 x tile_n outputs), which halves the token columns it
// re-reads from L2 per output.
//
// The epilogue adds the bias, applies RoPE (a 128-row tile holds whole heads, so both elements
// of a rotation pair are at hand), writes Q as a bf16 hi + lo pair and K, V as bf16, and
// persists what the method keeps: the carrier row's K/V goes straight into the bank's free slot
// (Section 3.2: only the carrier keeps its K/V), text rows are appended to the prefix or to the
// turn's tail.
//
// Per CTA: 6 or 18 warps.  Warp 0 lane 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer
// (lane 0), warps 2.. = epilogue, 4 or 16 of them (tcgen05.ld of the 32-lane quarter that
// warp % 4 allows; with 16, four warps per quarter take every fourth block of 16 columns).
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, records
// VS_ERR_DEVICE_TIMEOUT, lets in-flight copies land, frees its tensor memory and exits.
#include "vs_common.cuh"

namespace vs {

namespace {

constexpr int kMaxEpiWarps = 16;                 // 4 per scheduler: the epilogue is bound by instruction latency
constexpr int kMaxThreads = 64 + 32 * kMaxEpiWarps;
constexpr int kStageABytes = GEMM_BLOCK_M * GEMM_BLOCK_K * 2;   // 16 KiB
constexpr unsigned long long kWaitLimitNs = 400ull * 1000ull * 1000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: spins on try_wait (which itself blocks for a short hardware-defined time) and
// consults the clock only every 1024 failed polls.  Returns false if the wait expired or
// another role already aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  uint32_t spins = 0;
  unsigned long long t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 1023u) == 0u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows of 128 bytes,
// 8-row groups 1024 bytes apart (stride byte offset), descriptor version 1, layout 2.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024u >> 4) << 32;                 // stride byte offset
  d |= (uint64_t)1 << 46;                            // descriptor version (Blackwell)
  d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
  return d;
}
// Instruction descriptor, kind::f16: D = fp32, A = B = bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t make_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(GEMM_BLOCK_M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}

struct KernelParams {
  ProjectionOut o;
  int* status;
  int rows, E_out, tile_n, kblocks, stages, tmem_cols, ksplit;
  float inv_d;                  // 1 / d_model
  int acc_stride;               // TMEM columns between the accumulators
  uint32_t data_bytes;          // shared memory ahead of the barriers: max(pipeline stages, own fp32 slice)
  float* xchg;                  // [group][rank][tile_n][128] partial tiles of the K split
  int* flags;                   // [group][rank] peers that have delivered their part of slice `rank`
};

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

template <bool kOwnRope, int kMSub>   // kOwnRope: no RoPE table, every finishing thread derives the rotation of its one
                                      // row; kMSub: 128-row weight sub-tiles (accumulators) per CTA
__global__ void __launch_bounds__(kMaxThreads, 1)
qkv_gemm_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
                const __grid_constant__ CUtensorMap tm_w2, KernelParams p, BatchParams bp) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // carve: [stages][A 16 KiB | B tile_n*128] (later reused for this CTA's own token slice of
  // the fp32 partial tile, [token][128 features]) | full[stages] | empty[stages] | tmem_full |
  // tmem slot | abort
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage_b_bytes = (uint32_t)p.tile_n * 128u;
  const uint32_t stage_a_bytes = (uint32_t)kMSub * kStageABytes;
  const uint32_t stage_bytes = stage_a_bytes + stage_b_bytes;
  const uint32_t bar_base = base + p.data_bytes;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  uint8_t* ctl = gen_base + p.data_bytes + 16 * p.stages;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctl + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + 12);
  auto full_bar = [&](int s) { return bar_base + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (uint32_t)(p.stages + s); };
  const uint32_t tmem_full_bar = bar_base + 16u * (uint32_t)p.stages;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int epi_warps = ((int)blockDim.x >> 5) - 2;   // 4, 8 or 16
  const int tok_lanes = 2 * epi_warps;                // token rows finished side by side
  const int m0 = blockIdx.x * GEMM_BLOCK_M * kMSub;
  const int n0 = blockIdx.y * p.tile_n;
  const int kb0 = blockIdx.z * p.kblocks;      // blockIdx.z = rank in the K split

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tmem_full_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");   // (the only scope this fence has)
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_acc = *tmem_slot;
  VS_STAMP(bp, 1, 0);
  pdl_wait();                       // earlier kernels of the stream have completed
  pdl_launch_dependents();
  VS_STAMP(bp, 1, 1);

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int kb = 0; kb < p.kblocks; ++kb) {
        const int s = kb % p.stages;
        const uint32_t ph = (uint32_t)(kb / p.stages) & 1u;
        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) break;
        mbar_arrive_expect_tx(full_bar(s), stage_bytes);
        const uint32_t a_dst = base + (uint32_t)s * stage_bytes;
        const int kx = (kb0 + kb) * GEMM_BLOCK_K;
#pragma unroll
        for (int ms = 0; ms < kMSub; ++ms) {
          if (p.o.mode == 5) {
            // a 128-row tile = 64 rows of the gate matrix, then the same 64 rows of the up matrix
            const int r64 = (m0 + ms * GEMM_BLOCK_M) >> 1;
            tma_load_2d(a_dst + (uint32_t)ms * kStageABytes, &tm_w, kx, r64, full_bar(s));
            tma_load_2d(a_dst + (uint32_t)ms * kStageABytes + kStageABytes / 2, &tm_w2, kx, r64, full_bar(s));
          } else {
            tma_load_2d(a_dst + (uint32_t)ms * kStageABytes, &tm_w, kx, m0 + ms * GEMM_BLOCK_M, full_bar(s));
          }
        }
        tma_load_2d(a_dst + stage_a_bytes, &tm_x, kx, n0, full_bar(s));
        issued = kb + 1;
      }
      if (*abort_flag) {
        // let this CTA's copies land before its shared memory is given up
        for (int kb = (issued > p.stages ? issued - p.stages : 0); kb < issued; ++kb) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(full_bar(kb % p.stages), (uint32_t)(kb / p.stages) & 1u)) {
            if (global_ns() - t0 > kWaitLimitNs) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(p.tile_n);
      bool ok = true;
      for (int kb = 0; kb < p.kblocks; ++kb) {
        const int s = kb % p.stages;
        const uint32_t ph = (uint32_t)(kb / p.stages) & 1u;
        ok = mbar_wait(full_bar(s), ph, abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_addr = base + (uint32_t)s * stage_bytes;
        const uint32_t b_addr = a_addr + stage_a_bytes;
#pragma unroll
        for (int k = 0; k < GEMM_BLOCK_K / 16; ++k) {
          // 16 bf16 = 32 bytes further along K inside the 128-byte swizzle row
#pragma unroll
          for (int ms = 0; ms < kMSub; ++ms)
            umma_bf16(tmem_acc + (uint32_t)(ms * p.acc_stride), make_smem_desc(a_addr + (uint32_t)ms * kStageABytes + 32u * k),
                      make_smem_desc(b_addr + 32u * k), idesc, (uint32_t)((kb | k) != 0));
        }
        umma_commit(empty_bar(s));          // frees the stage once these MMAs have read it
      }
      if (ok) umma_commit(tmem_full_bar);   // accumulator complete
    }
  }

  // ---- epilogue ---------------------------------------------------------------------------
  // The tile's tokens are cut into ksplit slices; CTA r of the split owns slice r.
  // A  every CTA waits for its own accumulator (all its MMAs done, so all its TMA writes have
  //    landed and its stages are dead) and copies it out, fp32, as [token][128 features]: its own
  //    slice into its shared memory, the other slices into its part of the exchange buffer.
  // B  it then counts itself in on the flag of every other slice's owner, and waits until the
  //    ksplit - 1 peers have done the same on its own flag.
  // C  the owner of a slice sums the ksplit partials of its tokens, adds the bias, rotates,
  //    rounds and stores.
  const int slice = p.tile_n / p.ksplit;          // tile_n is a multiple of 16, ksplit is 1, 2 or 4
  const int rank = (int)blockIdx.z;
  const int group = (int)(blockIdx.y * gridDim.x + blockIdx.x);
  const int t_begin = rank * slice;
  // A step of a few rows brings no RoPE table: each finishing thread works out the (cos, sin) of
  // the four rotation pairs of its one row, in fp64 like the table kernel, while the main loop runs.
  float4 own_ra = make_float4(1.f, 0.f, 1.f, 0.f), own_rb = own_ra;
  if (kOwnRope && warp >= 2) {
    const int te = threadIdx.x - 64;
    const int half = p.o.D >> 1;
    const int p0 = (te & 15) * 4, hl = p0 / half, k0 = p0 - hl * half;
    const int row = n0 + t_begin + (te >> 4);
    if ((m0 + hl * p.o.D + k0) / p.o.D < p.o.Hq + p.o.Hkv && (te >> 4) < slice && row < p.rows) {
      const int b = row / bp.rows_per_stream;
      const double pos = (double)(bp.pos_base[b] + (row - b * bp.rows_per_stream));
      double sn, cs;
      float r[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        sincos(pos * p.o.inv_freq[k0 + i], &sn, &cs);
        r[2 * i] = (float)cs; r[2 * i + 1] = (float)sn;
      }
      own_ra = make_float4(r[0], r[1], r[2], r[3]);
      own_rb = make_float4(r[4], r[5], r[6], r[7]);
    }
  }
  // RMSNorm: the row scales of this CTA's token slice, worked out while the main loop runs
  float* rsc_s = reinterpret_cast<float*>(ctl + 64);             // [slice]
  if (warp >= 2 && p.o.row_ss != nullptr) {
    for (int t = threadIdx.x - 64; t < slice; t += (int)blockDim.x - 64) {
      const int row = n0 + t_begin + t;
      float tot = 0.f;
      if (row < p.rows)
        for (int i = 0; i < p.o.ss_parts; ++i) tot += p.o.row_ss[(size_t)row * p.o.ss_parts + i];
      rsc_s[t] = rsqrtf(tot * p.inv_d + p.o.norm_eps);
    }
  }
  bool acc_ok = true;
  if (warp >= 2) {
    acc_ok = __all_sync(0xffffffffu, mbar_wait(tmem_full_bar, 0, abort_flag));   // warp-uniform
  }
  tcgen05_fence_after();
  VS_STAMP_BY(bp, 1, 2, 64);          // accumulator complete

  // one pass per 128-row weight sub-tile (its own accumulator); the staging memory is shared
#pragma unroll 1
  for (int ms = 0; ms < kMSub; ++ms) {
  const int m0e = m0 + ms * GEMM_BLOCK_M;
  const uint32_t tmem_sub = tmem_acc + (uint32_t)(ms * p.acc_stride);
  float* part_local = reinterpret_cast<float*>(gen_base);      // [token - t_begin][128 features]
  if (warp >= 2 && acc_ok) {
    // warp w may touch TMEM lanes 32*(w%4) .. +31 (lane = feature)
    const int quarter = warp & 3;
    float* dst_own = part_local + quarter * 32 + lane;
    float* dst_far = p.xchg + ((size_t)group * p.ksplit + rank) * p.tile_n * GEMM_BLOCK_M + quarter * 32 + lane;
    for (int c = 16 * ((warp - 2) >> 2); c < p.tile_n; c += 16 * (epi_warps >> 2)) {
      if (n0 + c >= p.rows) break;                             // uniform across the warp
      uint32_t r[16];
      tmem_ld16(tmem_sub + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, r);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int t = c + j;
        if ((unsigned)(t - t_begin) < (unsigned)slice) dst_own[(t - t_begin) * GEMM_BLOCK_M] = __uint_as_float(r[j]);
        else if (VS_STORE_OK(bp, DR_GEMM_XCHG, dst_far + (size_t)t * GEMM_BLOCK_M, 4)) dst_far[(size_t)t * GEMM_BLOCK_M] = __uint_as_float(r[j]);
      }
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (p.ksplit > 1 && threadIdx.x == 64) {
    if (!*abort_flag) {
      // the barrier above ordered every thread's stores before this point; one cumulative fence
      // then orders them before the flag increments for whoever acquires a flag
      __threadfence();
      for (int s = 0; s < p.ksplit; ++s)
        if (s != rank) atomicAdd(p.flags + group * p.ksplit + s, 1);
    }
    int* mine = p.flags + group * p.ksplit + rank;
    uint32_t spins = 0;
    unsigned long long t0 = 0;
    while (!*abort_flag && ld_acquire_gpu(mine) < p.ksplit - 1) {
      if ((++spins & 255u) == 0u) {
        const unsigned long long now = global_ns();
        if (t0 == 0) t0 = now;
        else if (now - t0 > kWaitLimitNs) *abort_flag = 1;
      }
    }
    *mine = 0;                                                 // next launch starts from zero
  }
  if (p.ksplit > 1) __syncthreads();

  // phase C.  Thread = (group of 4 rotation pairs, token lane).  The reads of a row -- float4
  // pieces of the own slice in shared memory and of the peers' partials in the exchange buffer,
  // and the row's RoPE entries -- are all issued before the arithmetic.
  if (warp >= 2 && !*abort_flag) {
    const int te = threadIdx.x - 64;               // 0 .. 32 * epi_warps - 1
    const int D = p.o.D, half = D >> 1;
    const int p0 = (te & 15) * 4;                  // first of 4 rotation pairs inside the 128-feature tile
    const int hl = p0 / half, k0 = p0 - hl * half; // local head, index inside the half head
    const int f1 = hl * D + k0, f2 = f1 + half;
    const int hs = (m0e + f1) / D;                  // head slot: Q heads, then K heads, then V heads
    const bool rotate = p.o.mode < 4 && hs < p.o.Hq + p.o.Hkv;
    const float* far = p.xchg + (size_t)group * p.ksplit * p.tile_n * GEMM_BLOCK_M;
    const size_t far_stride = (size_t)p.tile_n * GEMM_BLOCK_M;
    if (m0e + f2 + 3 < p.E_out) {
      float bb1[4] = {0.f, 0.f, 0.f, 0.f}, bb2[4] = {0.f, 0.f, 0.f, 0.f};
      if (p.o.bias != nullptr) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          bb1[i] = __bfloat162float(p.o.bias[m0e + f1 + i]);
          bb2[i] = __bfloat162float(p.o.bias[m0e + f2 + i]);
        }
      }
      const int rps = bp.rows_per_stream;
      const int n_it = (slice - (te >> 4) + tok_lanes - 1) / tok_lanes;   // rows this thread finishes
      struct RowRegs { float4 v1[KSPLIT_MAX], v2[KSPLIT_MAX], ra, rb; float rsc; };
      auto valid_it = [&](int it) { return it < n_it && n0 + t_begin + (te >> 4) + tok_lanes * it < p.rows; };
      auto load_row = [&](RowRegs& R, int it) {
        const int t = t_begin + (te >> 4) + tok_lanes * it;
        const int row = n0 + t;
#pragma unroll
        for (int r = 0; r < KSPLIT_MAX; ++r) {
          if (r == rank) {
            R.v1[r] = *reinterpret_cast<const float4*>(part_local + (t - t_begin) * GEMM_BLOCK_M + f1);
            R.v2[r] = *reinterpret_cast<const float4*>(part_local + (t - t_begin) * GEMM_BLOCK_M + f2);
          } else if (r < p.ksplit) {
            // written by another SM during this launch: read past L1
            R.v1[r] = __ldcg(reinterpret_cast<const float4*>(far + r * far_stride + (size_t)t * GEMM_BLOCK_M + f1));
            R.v2[r] = __ldcg(reinterpret_cast<const float4*>(far + r * far_stride + (size_t)t * GEMM_BLOCK_M + f2));
          }
        }
        if (rotate) {
          if (!kOwnRope) {
            R.ra = *reinterpret_cast<const float4*>(p.o.rope + (size_t)row * half + k0);
            R.rb = *reinterpret_cast<const float4*>(p.o.rope + (size_t)row * half + k0 + 2);
          } else {                       // the thread's only row (the launch checks it)
            R.ra = own_ra; R.rb = own_rb;
          }
        }
        // RMSNorm's row scale commutes with the projection: applied here, in fp32
        R.rsc = (p.o.row_ss != nullptr) ? rsc_s[t - t_begin] : 1.f;
      };
      auto finish_row = [&](const RowRegs& R, int it) {
        const int t = t_begin + (te >> 4) + tok_lanes * it;
        const int row = n0 + t;
        float x1[4] = {0.f, 0.f, 0.f, 0.f}, x2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int r = 0; r < KSPLIT_MAX; ++r) {
          if (r < p.ksplit) {
            x1[0] += R.v1[r].x; x1[1] += R.v1[r].y; x1[2] += R.v1[r].z; x1[3] += R.v1[r].w;
            x2[0] += R.v2[r].x; x2[1] += R.v2[r].y; x2[2] += R.v2[r].z; x2[3] += R.v2[r].w;
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) { x1[i] = fmaf(x1[i], R.rsc, bb1[i]); x2[i] = fmaf(x2[i], R.rsc, bb2[i]); }
        if (rotate) {
          const float cs[4] = {R.ra.x, R.ra.z, R.rb.x, R.rb.z}, sn[4] = {R.ra.y, R.ra.w, R.rb.y, R.rb.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float y1 = x1[i] * cs[i] - x2[i] * sn[i];
            const float y2 = x2[i] * cs[i] + x1[i] * sn[i];
            x1[i] = y1; x2[i] = y2;
          }
        }
        if (p.o.mode == 5) {
          // SwiGLU: features f1.. are gate rows, f2 = f1 + 64.. the matching up rows
          __align__(8) bf16 av[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) av[i] = __float2bfloat16_rn(x1[i] / (1.f + __expf(-x1[i])) * x2[i]);
          bf16* dst = p.o.lin_out + (size_t)row * (p.E_out >> 1) + (m0e >> 1) + f1;
          if (VS_STORE_OK(bp, p.o.lin_out_region, dst, 8)) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(av);
          return;
        }
        if (p.o.mode == 6) {
          // plain linear layer, rows kept in fp32 (logits of the vocabulary projection); the buffer is the caller's
          float* fo = static_cast<float*>(p.o.final_out) + (size_t)row * p.E_out + m0e;
          *reinterpret_cast<float4*>(fo + f1) = make_float4(x1[0], x1[1], x1[2], x1[3]);
          *reinterpret_cast<float4*>(fo + f2) = make_float4(x2[0], x2[1], x2[2], x2[3]);
          return;
        }
        if (p.o.mode == 4) {
          // linear layer + residual; the rows as stored (bf16) also give the next RMSNorm its statistics
          const size_t c1 = (size_t)row * p.E_out + m0e + f1, c2 = (size_t)row * p.E_out + m0e + f2;
          if (p.o.lin_res != nullptr) {
            const uint2 r1 = *reinterpret_cast<const uint2*>(p.o.lin_res + c1), r2 = *reinterpret_cast<const uint2*>(p.o.lin_res + c2);
            const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r1.x)), a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r1.y));
            const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r2.x)), b1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r2.y));
            x1[0] += a0.x; x1[1] += a0.y; x1[2] += a1.x; x1[3] += a1.y;
            x2[0] += b0.x; x2[1] += b0.y; x2[2] += b1.x; x2[3] += b1.y;
          }
          __align__(8) bf16 s1[4], s2[4];
          float ss = 0.f;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            s1[i] = __float2bfloat16_rn(x1[i]); s2[i] = __float2bfloat16_rn(x2[i]);
            const float u1 = __bfloat162float(s1[i]), u2 = __bfloat162float(s2[i]);
            ss += u1 * u1 + u2 * u2;
          }
          if (VS_STORE_OK(bp, p.o.lin_out_region, p.o.lin_out + c1, 8) && VS_STORE_OK(bp, p.o.lin_out_region, p.o.lin_out + c2, 8)) {
            *reinterpret_cast<uint2*>(p.o.lin_out + c1) = *reinterpret_cast<const uint2*>(s1);
            *reinterpret_cast<uint2*>(p.o.lin_out + c2) = *reinterpret_cast<const uint2*>(s2);
          }
          if (p.o.final_out != nullptr) {
            if (p.o.final_fp32) {
              float* fo = static_cast<float*>(p.o.final_out);
              *reinterpret_cast<float4*>(fo + c1) = make_float4(__bfloat162float(s1[0]), __bfloat162float(s1[1]), __bfloat162float(s1[2]), __bfloat162float(s1[3]));
              *reinterpret_cast<float4*>(fo + c2) = make_float4(__bfloat162float(s2[0]), __bfloat162float(s2[1]), __bfloat162float(s2[2]), __bfloat162float(s2[3]));
            } else {
              bf16* fo = static_cast<bf16*>(p.o.final_out);
              *reinterpret_cast<uint2*>(fo + c1) = *reinterpret_cast<const uint2*>(s1);
              *reinterpret_cast<uint2*>(fo + c2) = *reinterpret_cast<const uint2*>(s2);
            }
          }
          if (p.o.ss_out != nullptr) {
            if (p.o.next_gain != nullptr) {
              __align__(8) bf16 g1[4], g2[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                g1[i] = __float2bfloat16_rn(__bfloat162float(s1[i]) * __bfloat162float(p.o.next_gain[m0e + f1 + i]));
                g2[i] = __float2bfloat16_rn(__bfloat162float(s2[i]) * __bfloat162float(p.o.next_gain[m0e + f2 + i]));
              }
              if (VS_STORE_OK(bp, DR_XN, p.o.xn_out + c1, 8) && VS_STORE_OK(bp, DR_XN, p.o.xn_out + c2, 8)) {
                *reinterpret_cast<uint2*>(p.o.xn_out + c1) = *reinterpret_cast<const uint2*>(g1);
                *reinterpret_cast<uint2*>(p.o.xn_out + c2) = *reinterpret_cast<const uint2*>(g2);
              }
            }
            // the 16 threads that share the row (a half warp) add their parts in a fixed order
            const unsigned hm = 0xFFFFu << (threadIdx.x & 16u);
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(hm, ss, o);
            float* sp = p.o.ss_out + (size_t)row * p.o.ss_out_parts + m0e / GEMM_BLOCK_M;
            if ((te & 15) == 0 && VS_STORE_OK(bp, DR_ROW_SS, sp, 4)) *sp = ss;
          }
          return;
        }
        __align__(8) bf16 o1[4], o2[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { o1[i] = __float2bfloat16_rn(x1[i]); o2[i] = __float2bfloat16_rn(x2[i]); }
        const uint2 w1 = *reinterpret_cast<const uint2*>(o1), w2 = *reinterpret_cast<const uint2*>(o2);
        if (hs < p.o.Hq) {
          // the query never leaves the step, so it is kept as a bf16 pair (hi + lo): the score
          // Q K^T then sees a 16-bit mantissa instead of 8 at the cost of a second MMA
          __align__(8) bf16 l1[4], l2[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            l1[i] = __float2bfloat16_rn(x1[i] - __bfloat162float(o1[i]));
            l2[i] = __float2bfloat16_rn(x2[i] - __bfloat162float(o2[i]));
          }
          if (p.o.q_tiled != nullptr) {
            // straight into the attention kernel's operand layout: one block per (batch entry, 16-token
            // row tile, KV head) holding [hi | lo][128 rows = g * 16 + token][D], rows of 128 bytes per
            // 64 dims with the 16-byte units XOR-ed by the row (the MMA's 128-byte swizzle)
            const int G = p.o.Hq / p.o.Hkv;
            const int b = row / rps, tt = row - b * rps;
            const int n_rt = (rps + 15) >> 4;
            const size_t tile = ((size_t)b * n_rt + (size_t)(tt >> 4)) * p.o.Hkv + (size_t)(hs / G);
            const int r = (hs % G) * 16 + (tt & 15);
            uint8_t* tb = reinterpret_cast<uint8_t*>(p.o.q_tiled) + tile * (size_t)(2 * 128 * D * 2);
            const int c1 = k0 >> 3, c2 = (k0 + half) >> 3;
            const uint32_t o_1 = (uint32_t)((c1 >> 3) * (128 * 128) + r * 128 + (((c1 & 7) ^ (r & 7)) << 4) + (k0 & 7) * 2);
            const uint32_t o_2 = (uint32_t)((c2 >> 3) * (128 * 128) + r * 128 + (((c2 & 7) ^ (r & 7)) << 4) + (k0 & 7) * 2);
            const uint32_t lo_off = (uint32_t)(128 * D * 2);
            if (VS_STORE_OK(bp, DR_Q_TILED, tb + o_1, 8) && VS_STORE_OK(bp, DR_Q_TILED, tb + lo_off + o_2, 8)) {
              *reinterpret_cast<uint2*>(tb + o_1) = w1;
              *reinterpret_cast<uint2*>(tb + o_2) = w2;
              *reinterpret_cast<uint2*>(tb + lo_off + o_1) = *reinterpret_cast<const uint2*>(l1);
              *reinterpret_cast<uint2*>(tb + lo_off + o_2) = *reinterpret_cast<const uint2*>(l2);
            }
          } else {
            const size_t qo = (size_t)row * p.o.Hq * D + (size_t)hs * D + k0;
            if (VS_STORE_OK(bp, DR_Q, p.o.q + qo, 8) && VS_STORE_OK(bp, DR_Q, p.o.q + qo + half, 8) &&
                VS_STORE_OK(bp, DR_Q_LO, p.o.q_lo + qo, 8) && VS_STORE_OK(bp, DR_Q_LO, p.o.q_lo + qo + half, 8)) {
              *reinterpret_cast<uint2*>(p.o.q + qo) = w1;
              *reinterpret_cast<uint2*>(p.o.q + qo + half) = w2;
              *reinterpret_cast<uint2*>(p.o.q_lo + qo) = *reinterpret_cast<const uint2*>(l1);
              *reinterpret_cast<uint2*>(p.o.q_lo + qo + half) = *reinterpret_cast<const uint2*>(l2);
            }
          }
        } else {
          const bool is_k = hs < p.o.Hq + p.o.Hkv;
          const int hkv = is_k ? hs - p.o.Hq : hs - p.o.Hq - p.o.Hkv;
          bf16* f = (is_k ? p.o.kf : p.o.vf) + (size_t)row * p.o.Hkv * D + (size_t)hkv * D + k0;
          if (VS_STORE_OK(bp, is_k ? DR_KF : DR_VF, f, 8) && VS_STORE_OK(bp, is_k ? DR_KF : DR_VF, f + half, 8)) {
            *reinterpret_cast<uint2*>(f) = w1;
            *reinterpret_cast<uint2*>(f + half) = w2;
          }
          const int b = row / rps, tt = row - b * rps;
          const int sid = bp.stream_id[b];
          bf16* dst = nullptr;
          if (p.o.mode == 0) {
            if (tt == rps - 1 && p.o.M > 0) {
              const int slot = p.o.free_slot[sid * p.o.free_slot_stride];
              dst = (is_k ? p.o.bank_k : p.o.bank_v) + (((size_t)sid * p.o.Hkv + hkv) * p.o.slots + slot) * D + k0;
            }
          } else if (p.o.mode != 3) {
            const int tb = (p.o.mode == 1) ? bp.prefix_len[b] : bp.text_len[b];
            dst = (is_k ? p.o.text_k : p.o.text_v) + (((size_t)sid * p.o.Hkv + hkv) * p.o.text_cap + tb + tt) * D + k0;
          }
          // (the carrier row goes to the bank, text rows to the prefix or the tail)
          const int dreg = (p.o.mode == 0) ? (is_k ? DR_BANK_K : DR_BANK_V)
                                           : (p.o.mode == 1 ? (is_k ? DR_PREFIX_K : DR_PREFIX_V) : (is_k ? DR_TAIL_K : DR_TAIL_V));
          if (dst != nullptr && VS_STORE_OK(bp, dreg, dst, 8) && VS_STORE_OK(bp, dreg, dst + half, 8)) {
            *reinterpret_cast<uint2*>(dst) = w1;
            *reinterpret_cast<uint2*>(dst + half) = w2;
          }
        }
      };
      // four warps per scheduler overlap one another's load latency; a thread holds one row at a time
#pragma unroll 1
      for (int it = 0; valid_it(it); ++it) {
        RowRegs A;
        load_row(A, it);
        finish_row(A, it);
      }
    }
  }
  if (ms + 1 < kMSub) { tcgen05_fence_before(); __syncthreads(); tcgen05_fence_after(); }   // rows finished before the staging memory is reused
  }

  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)p.tmem_cols) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, VS_ERR_DEVICE_TIMEOUT);
  VS_STAMP(bp, 1, 15);
}

constexpr int kMaxDynSmem = 227 * 1024;

}  // namespace

cudaError_t qkv_gemm_init() {
  cudaError_t e = cudaFuncSetAttribute(qkv_gemm_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(qkv_gemm_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(qkv_gemm_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
  return e;
}

cudaError_t launch_qkv_gemm(const GemmArgs& a, const BatchParams& bp, cudaStream_t st) {
  KernelParams p;
  p.o = a.out;
  p.status = a.status;
  p.rows = a.rows;
  p.E_out = a.E_out;
  p.tile_n = a.tile_n;
  p.ksplit = a.ksplit;
  p.inv_d = 1.f / (float)a.d;
  const int total_kb = a.d / GEMM_BLOCK_K;
  if (a.ksplit < 1 || a.ksplit > KSPLIT_MAX || (a.ksplit & (a.ksplit - 1)) || total_kb % a.ksplit != 0) return cudaErrorInvalidValue;
  if (a.tile_n < 16 || a.tile_n > 256 || (a.tile_n & 15)) return cudaErrorInvalidValue;
  if (a.m_sub != 1 && !(a.m_sub == 2 && a.ksplit == 1 && a.E_out % (2 * GEMM_BLOCK_M) == 0)) return cudaErrorInvalidValue;
  if (128 % a.out.D != 0) return cudaErrorInvalidValue;
  p.kblocks = total_kb / a.ksplit;
  p.xchg = a.xchg;
  p.flags = a.flags;
  const int stage_bytes = a.m_sub * kStageABytes + a.tile_n * 128;
  int stages = (kMaxDynSmem - 3072) / stage_bytes;
  if (stages > 8) stages = 8;
  if (stages > p.kblocks) stages = p.kblocks;
  if (stages < 1) return cudaErrorInvalidValue;
  p.stages = stages;
  int cols = 32;
  while (cols < a.tile_n) cols <<= 1;
  p.acc_stride = cols;
  p.tmem_cols = cols * a.m_sub;            // a power of two, at most 512
  size_t data = (size_t)stages * stage_bytes;
  const size_t own = (size_t)(a.tile_n / a.ksplit) * GEMM_BLOCK_M * 4;
  if (own > data) data = (own + 1023) / 1024 * 1024;
  p.data_bytes = (uint32_t)data;
  const size_t smem = 1024 + data + 16 * stages + 64 + 1024;     // + the slice's RMSNorm row scales
  if (smem > (size_t)kMaxDynSmem) return cudaErrorInvalidValue;
  // a token slice of a few rows is finished by 4 warps; wider ones by 16, which overlap one another's latency
  const int slice_rows = a.tile_n / a.ksplit;
  const int threads = 64 + 32 * (slice_rows <= 8 ? 4 : kMaxEpiWarps);
  // without a RoPE table every finishing thread must have at most one row
  if (a.out.rope == nullptr && (a.out.inv_freq == nullptr || slice_rows > 2 * (threads / 32 - 2))) return cudaErrorInvalidValue;
  const dim3 grid((a.E_out + GEMM_BLOCK_M * a.m_sub - 1) / (GEMM_BLOCK_M * a.m_sub), a.n_tiles, a.ksplit);
  if (a.ksplit > 1) {
    // the CTAs of a K split wait for one another: the whole grid has to be resident at once
    if (a.xchg == nullptr || a.flags == nullptr) return cudaErrorInvalidValue;
    int per_sm = 0;
    cudaError_t e = (a.out.rope == nullptr)
        ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, qkv_gemm_kernel<true, 1>, threads, smem)
        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, qkv_gemm_kernel<false, 1>, threads, smem);
    if (e != cudaSuccess) return e;
    if ((long long)grid.x * grid.y * grid.z > (long long)per_sm * a.n_sms) return cudaErrorInvalidValue;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (a.out.rope == nullptr) {
    if (a.m_sub != 1) return cudaErrorInvalidValue;
    return cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<true, 1>, a.tm_w, a.tm_x, a.tm_w2, p, bp);
  }
  if (a.m_sub == 2) return cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<false, 2>, a.tm_w, a.tm_x, a.tm_w2, p, bp);
  return cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<false, 1>, a.tm_w, a.tm_x, a.tm_w2, p, bp);
}

}  // namespace vs
