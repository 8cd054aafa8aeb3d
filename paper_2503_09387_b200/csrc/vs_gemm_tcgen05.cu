// QKV projection (Eq. 1: Q = X W_Q, K = X W_K, V = X W_V) on the 5th-generation tensor
// cores: tcgen05.mma with the accumulator in tensor memory, operands staged in shared
// memory by TMA, one elected thread issuing the MMAs.
//
// Orientation.  A frame brings only N + 1 (<= 256) token rows but E_out = (Hq + 2 Hkv) D
// output features (4608 at the Qwen2-7B shape), so the *features* take the MMA's M axis
// (128 weight rows per CTA, read K-major straight from the caller's [E_out, d] matrix) and
// the *tokens* take the MMA's N axis (any multiple of 16 up to 256: 170 tokens cost 176
// columns, 3.5 % padding instead of 33 % with 128-row token tiles).  The reduction dimension
// d is split over `ksplit` CTAs so that m_tiles * n_tiles * ksplit fills the 148 SMs; each
// CTA writes an fp32 partial tile which the finalize kernel sums.
//
// Per CTA: 6 warps.  Warp 0 lane 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer
// (lane 0), warps 2..5 = epilogue (tcgen05.ld of their 32-lane quarter -> global).
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, records
// VS_ERR_DEVICE_TIMEOUT, lets in-flight copies land, frees its tensor memory and exits.
#include "vs_common.cuh"

namespace vs {

namespace {

constexpr int kThreads = 192;
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
  float* partials;
  int* status;
  int rows, E_out, tile_n, kblocks, stages, tmem_cols;
};

__global__ void __launch_bounds__(kThreads, 1)
qkv_gemm_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, KernelParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // carve: [stages][A 16 KiB | B tile_n*128] | full[stages] | empty[stages] | tmem_full | tmem slot | abort
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage_b_bytes = (uint32_t)p.tile_n * 128u;
  const uint32_t stage_bytes = kStageABytes + stage_b_bytes;
  const uint32_t bar_base = base + (uint32_t)p.stages * stage_bytes;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  uint8_t* ctl = gen_base + (size_t)p.stages * stage_bytes + 16 * p.stages;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctl + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + 12);
  auto full_bar = [&](int s) { return bar_base + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (uint32_t)(p.stages + s); };
  const uint32_t tmem_full_bar = bar_base + 16u * (uint32_t)p.stages;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * GEMM_BLOCK_M;
  const int n0 = blockIdx.y * p.tile_n;
  const int kb0 = blockIdx.z * p.kblocks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tmem_full_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
        tma_load_2d(a_dst, &tm_w, kx, m0, full_bar(s));
        tma_load_2d(a_dst + kStageABytes, &tm_x, kx, n0, full_bar(s));
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
        const uint32_t b_addr = a_addr + kStageABytes;
#pragma unroll
        for (int k = 0; k < GEMM_BLOCK_K / 16; ++k) {
          // 16 bf16 = 32 bytes further along K inside the 128-byte swizzle row
          umma_bf16(tmem_acc, make_smem_desc(a_addr + 32u * k), make_smem_desc(b_addr + 32u * k), idesc,
                    (uint32_t)((kb | k) != 0));
        }
        umma_commit(empty_bar(s));          // frees the stage once these MMAs have read it
      }
      if (ok) umma_commit(tmem_full_bar);   // accumulator complete
    }
  } else {
    // epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31 (one lane = one output feature)
    const int quarter = warp & 3;
    const bool ok = __all_sync(0xffffffffu, mbar_wait(tmem_full_bar, 0, abort_flag));   // warp-uniform
    tcgen05_fence_after();
    if (ok) {
      const int feat = m0 + quarter * 32 + lane;
      float* dst = p.partials + ((size_t)blockIdx.z * p.rows) * p.E_out + feat;
      for (int c = 0; c < p.tile_n; c += 16) {
        if (n0 + c >= p.rows) break;               // uniform across the warp
        uint32_t r[16];
        tmem_ld16(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (feat < p.E_out) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int tok = n0 + c + j;
            if (tok < p.rows) dst[(size_t)tok * p.E_out] = __uint_as_float(r[j]);
          }
        }
      }
    }
  }

  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)p.tmem_cols) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, VS_ERR_DEVICE_TIMEOUT);
}

constexpr int kMaxDynSmem = 227 * 1024;

}  // namespace

cudaError_t qkv_gemm_init() {
  return cudaFuncSetAttribute(qkv_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
}

cudaError_t launch_qkv_gemm(const GemmArgs& a, cudaStream_t st) {
  KernelParams p;
  p.partials = a.partials;
  p.status = a.status;
  p.rows = a.rows;
  p.E_out = a.E_out;
  p.tile_n = a.tile_n;
  const int total_kb = a.d / GEMM_BLOCK_K;
  if (a.ksplit < 1 || total_kb % a.ksplit != 0) return cudaErrorInvalidValue;
  if (a.tile_n < 16 || a.tile_n > 256 || (a.tile_n & 15)) return cudaErrorInvalidValue;
  p.kblocks = total_kb / a.ksplit;
  const int stage_bytes = kStageABytes + a.tile_n * 128;
  int stages = (kMaxDynSmem - 2048) / stage_bytes;
  if (stages > 8) stages = 8;
  if (stages > p.kblocks) stages = p.kblocks;
  if (stages < 1) return cudaErrorInvalidValue;
  p.stages = stages;
  int cols = 32;
  while (cols < a.tile_n) cols <<= 1;
  p.tmem_cols = cols;
  const size_t smem = 1024 + (size_t)stages * stage_bytes + 16 * stages + 64;
  dim3 grid((a.E_out + GEMM_BLOCK_M - 1) / GEMM_BLOCK_M, a.n_tiles, a.ksplit);
  qkv_gemm_kernel<<<grid, kThreads, smem, st>>>(a.tm_w, a.tm_x, p);
  return cudaGetLastError();
}

}  // namespace vs
