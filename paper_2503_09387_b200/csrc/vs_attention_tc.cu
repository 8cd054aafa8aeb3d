// Frame-prefill / multi-token attention on the 5th-generation tensor cores
// (Eq. 1: Y = Softmax(Q K^T / sqrt(d_k)) V, grouped KV heads).
//
// One CTA = 16 query tokens x one KV head x one stream.  The G query heads of the group are
// stacked on the MMA's M axis (row = g * 16 + token, G * 16 <= 128), so K and V are staged
// once for the whole group.  Keys come from up to four segments -- prompt prefix, carrier bank
// (the free slot is masked), earlier text of the turn, the step's own rows (causal) -- laid end
// to end and cut into dense tiles of 128 keys.  The carrier is the last row of its frame
// (Section 3.2), so the causal rule alone gives it the whole frame.
// Per tile:  S = Q K^T  (tcgen05.mma, M 128 x N 128, Q as a bf16 hi + lo pair)     -> TMEM
//            softmax of the row in registers, P (bf16) -> shared memory (over the dead K tile)
//            O_tile = P V  (tcgen05.mma, M 128 x N D, V read MN-major)             -> TMEM
//            o_row = o_row * alpha + O_tile, one tile late (two O buffers)         (registers)
// Warps 0..7: two threads per row (each owns 64 keys of a tile and D/2 output dims).
// Warp 8: one thread issues every MMA, one tile of Q K^T ahead of the softmax (S is double
// buffered in TMEM); descriptors are built once.  Warps 9..11 fetch K/V with cp.async into the
// 128-byte-swizzled layout the MMA descriptors expect, one tile ahead.  Finished rows leave
// through shared memory as whole contiguous rows.  All mbarrier waits are bounded.
#include <type_traits>

#include "vs_common.cuh"
#include "vs_bank_update.cuh"

namespace vs {

namespace {

constexpr int kKeys = 128;       // keys per tile
constexpr int kRows = 128;       // MMA M
constexpr int kTok = 16;         // query tokens per CTA
constexpr unsigned long long kWaitLimitNs = 400ull * 1000ull * 1000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;   // 0 source bytes: the destination is zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
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
// consults the clock only every 1024 failed polls.
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

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
//   K-major operand : rows of 128 bytes along K, 8-row groups `sbo` bytes apart.
//   MN-major operand: rows of 128 bytes along MN (64 elements), 8 K-rows per group, groups
//                     `sbo` bytes apart along K, 64-element MN blocks `lbo` bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// kind::f16 instruction descriptor: D fp32, A = B = bf16, M = 128, N = n; b_mn = 1 when B is MN-major.
__device__ __forceinline__ uint32_t make_idesc(int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kRows >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// byte offset of 16-byte chunk c (8 bf16) of row r in a tile whose rows are `W` bf16 wide,
// stored as W/64 blocks of [rows x 128 bytes] with the 128-byte swizzle (chunk ^ (row & 7))
template <int ROWS>
__device__ __forceinline__ uint32_t sw_off(int r, int c) {
  return (uint32_t)((c >> 3) * (ROWS * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int D>
struct Smem {
  static constexpr int kQBytes = kRows * D * 2;           // one of hi / lo
  static constexpr int kKVBytes = kKeys * D * 2;          // one of K / V, one stage
  static constexpr int kQhi = 0;
  static constexpr int kQlo = kQBytes;
  static constexpr int kPBytes = kRows * kKeys * 2;
  static constexpr int kKStage = kKVBytes > kPBytes ? kKVBytes : kPBytes;   // K tile; P is written over it once S is done
  static constexpr int kK = 2 * kQBytes;                  // [stage] K tile / P
  static constexpr int kV = kK + 2 * kKStage;             // [stage] V tile
  static constexpr int kMax = kV + 2 * kKVBytes;          // float [2][2][128]: row maxima exchange
  static constexpr int kCtl = kMax + 2048;                // barriers, tmem slot, abort flag
  static constexpr int kExcl = kCtl + 128;                // chunk of frames: bitmap of masked bank-axis keys, per-tile flags
  static constexpr int kTotal = kExcl + ATTN_EXCL_BITS / 8 + 128 + 1024;   // + alignment slack
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// barrier 1 over the 256 softmax threads, AND-reducing a predicate (keeps their exits uniform)
__device__ __forceinline__ bool softmax_barrier_and(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 256, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred) : "memory");
  return r != 0;
}

constexpr int kSoftmaxThreads = 256;                     // warps 0..7
constexpr int kLoaderThreads = 96;                       // warps 9, 10, 11
constexpr int kAttnThreads = kSoftmaxThreads + 32 + kLoaderThreads;

__device__ __forceinline__ void umma_acc(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc) : "memory");
}
__device__ __forceinline__ void umma_new(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, 1, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1) prefill_attn_tc_kernel(AttnArgs a, BatchParams bp, int* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  using L = Smem<D>;
  constexpr int CPR = D / 8;
  constexpr int DH = D / 2;
  constexpr int KH = kKeys / 2;                 // keys of a tile owned by one thread of a row pair
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_s0 = base + L::kCtl;       // +0, +8: S buffer ready (tcgen05.commit)
  const uint32_t bar_o0 = base + L::kCtl + 16;  // +0, +64: O buffer ready (tcgen05.commit)
  const uint32_t bar_p = base + L::kCtl + 24;   // P written (256 arrivals)
  const uint32_t bar_kv0 = base + L::kCtl + 32; // +0, +8: K/V tile landed in a stage (one arrival per loader thread)
  const uint32_t bar_free0 = base + L::kCtl + 48;  // +0, +8: stage free again (tcgen05.commit after P V)
  const uint32_t bar_q = base + L::kCtl + 64;   // Q tile and the K tile of key tile 0 landed (256 arrivals)
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::kCtl + 72);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kCtl + 76);
  float* max_x = reinterpret_cast<float*>(gbase + L::kMax);
  uint32_t* excl = reinterpret_cast<uint32_t*>(gbase + L::kExcl);                      // [ATTN_EXCL_BITS / 32]
  uint8_t* tile_excl = gbase + L::kExcl + ATTN_EXCL_BITS / 8;                          // [128]

  const int tid = threadIdx.x, warp = tid >> 5;
  // ---- bank update CTAs (frame steps): the first a.bank_blocks of each stream.  What they read --
  // carrier embeddings, the bank's order and metadata -- was complete before the kernel ahead of
  // this one let it start, and nothing else in this launch touches what they write.
  if ((int)blockIdx.x < a.bank_blocks) {
    if (blockIdx.y == 0) bank_update_block(a.bank, bp, (int)blockIdx.z, (int)blockIdx.x);
    return;
  }
  // ---- set-up that needs nothing from earlier kernels: barriers, tensor memory ------------------
  if (tid == 0) {
    mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1);
    mbar_init(bar_o0, 1); mbar_init(bar_o0 + 64, 1);
    mbar_init(bar_p, kSoftmaxThreads);
    mbar_init(bar_kv0, kLoaderThreads); mbar_init(bar_kv0 + 8, kLoaderThreads);
    mbar_init(bar_free0, 1); mbar_init(bar_free0 + 8, 1);
    mbar_init(bar_q, kSoftmaxThreads);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // (the key axis below is laid out from the kernel's parameters alone, so it too comes before the wait)
  const int b = blockIdx.z, hkv = blockIdx.y;
  const int r0 = ((int)blockIdx.x - a.bank_blocks) * kTok;
  const int rps = bp.rows_per_stream;
  const int sid = bp.stream_id[b];
  const int G = a.Hq / a.Hkv;
  const int count = a.chunk_mode ? a.chunk_count0 : bp.count[b];
  const bool bank_full = (a.M > 0 && count == a.M);

  // ---- the virtual key axis: segments end to end ----------------------------------------------
  // key v of segment s lives at seg_k[s] + v * seg_stride[s] (the segment's first key index is
  // folded into the pointer)
  int seg_end[4];
  const bf16* seg_k[4];
  const bf16* seg_v[4];
  int seg_stride[4];
  int total = 0, causal_start = 0x3fffffff, hole = -1, bank_begin = 0;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    seg_k[s] = a.q; seg_v[s] = a.q; seg_stride[s] = 0;
    if (s < a.n_seg) {
      const AttnSegment sg = a.seg[s];
      int len;
      if (sg.kind == 0) len = bp.prefix_len[b];
      else if (sg.kind == 1) {
        len = (a.M == 0) ? 0 : (bank_full ? a.M + 1 : count);
        bank_begin = total;
      }
      else if (sg.kind == 2) len = bp.text_len[b];
      else if (sg.kind == 4) len = (a.M == 0) ? 0 : b;   // carriers of the chunk's frames before this one
      else { len = min(rps, r0 + kTok); causal_start = total; }  // later keys are visible to no row of this tile
      const long long off = (long long)(sg.by_batch ? b : sid) * sg.stream_stride + (long long)hkv * sg.head_stride -
                            (long long)total * sg.row_stride;
      seg_k[s] = sg.k + off; seg_v[s] = sg.v + off; seg_stride[s] = (int)sg.row_stride;
      total += len;
    }
    seg_end[s] = total;
  }
  const int n_tiles = (total + kKeys - 1) / kKeys;

  pdl_wait();                       // earlier kernels of the stream have completed
  pdl_launch_dependents();
  if (bank_full && !a.chunk_mode) hole = bank_begin + a.free_slot[sid * a.free_slot_stride];   // the slot being refilled holds no carrier
  // chunk of frames in one launch: bank-axis keys this frame must not see, as a bitmap
  const int excl_range = (a.chunk_mode && a.M > 0) ? (bank_full ? a.M + 1 : count) + b : 0;   // bank slots, then earlier frames' carriers
  if (a.chunk_mode) {
    for (int i = tid; i < ATTN_EXCL_BITS / 32; i += kAttnThreads) excl[i] = 0u;
    if (tid < 128) tile_excl[tid] = 0;
    __syncthreads();
    if (tid < b) {
      const int v = a.chunk_victim[tid];
      if (v >= 0 && v < excl_range) {
        atomicOr(&excl[v >> 5], 1u << (v & 31));
        const int ti_ = (bank_begin + v) / kKeys;
        if (ti_ < 128) tile_excl[ti_] = 1;
      }
    }
    if (tid == kAttnThreads - 1 && bank_full) {        // the slot that was free when the chunk began
      const int v = a.free_slot[0];
      atomicOr(&excl[v >> 5], 1u << (v & 31));
      const int ti_ = (bank_begin + v) / kKeys;
      if (ti_ < 128) tile_excl[ti_] = 1;
    }
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_o = tmem + 256;                    // S buffers at columns 0 and 128, O buffers at 256 and 384

  // ---- K/V tile fetch: cp.async into the swizzled tiles ------------------------------------------
  // Thread `lt` of `NT` cooperating threads owns one 16-byte column c of the key rows r = rsub,
  // rsub + NT / CPR, ...; it walks the tile segment by segment so that inside a segment a row
  // costs one pointer step.
  auto fetch_tile = [&](int ti, int lt, auto nt_c, bool do_k, bool do_v) {
    constexpr int kRowStep = decltype(nt_c)::value / CPR;     // key rows covered per pass
    const int c = lt % CPR, rsub = lt / CPR;
    const int stage = ti & 1;
    const uint32_t kdst = base + L::kK + (uint32_t)stage * L::kKStage + (uint32_t)((c >> 3) * (kKeys * 128));
    const uint32_t vdst = base + L::kV + (uint32_t)stage * L::kKVBytes + (uint32_t)((c >> 3) * (kKeys * 128));
    const int t_begin = ti * kKeys;
    int seg_begin = 0;
#pragma unroll
    for (int sgi = 0; sgi < 4; ++sgi) {
      const int lo = max(seg_begin, t_begin) - t_begin;            // rows of this segment inside the tile
      const int hi = min(seg_end[sgi], t_begin + kKeys) - t_begin;
      seg_begin = seg_end[sgi];
      if (lo >= hi) continue;
      int r = lo + ((rsub - lo) % kRowStep + kRowStep) % kRowStep;  // first row >= lo owned by this thread
      const long long step = (long long)kRowStep * seg_stride[sgi];
      const bf16* kp = seg_k[sgi] + (long long)(t_begin + r) * seg_stride[sgi] + c * 8;
      const bf16* vp = seg_v[sgi] + (long long)(t_begin + r) * seg_stride[sgi] + c * 8;
      for (; r < hi; r += kRowStep, kp += step, vp += step) {
        const uint32_t so = (uint32_t)(r * 128 + (((c & 7) ^ (r & 7)) << 4));
        if (do_k) cp_async16(kdst + so, kp, true);
        if (do_v) cp_async16(vdst + so, vp, true);
      }
    }
    // rows past the end of the key axis (last tile only): zero-filled
    for (int r = max(total - t_begin, 0) + ((rsub - max(total - t_begin, 0)) % kRowStep + kRowStep) % kRowStep; r < kKeys;
         r += kRowStep) {
      const uint32_t so = (uint32_t)(r * 128 + (((c & 7) ^ (r & 7)) << 4));
      if (do_k) cp_async16(kdst + so, a.q, false);
      if (do_v) cp_async16(vdst + so, a.q, false);
    }
  };

  if (warp >= 9) {
    // ---- K/V loaders, one tile ahead.  The K tile of key tile 0 is fetched by the softmax threads
    // together with Q (they are idle until the first scores exist); the loaders bring its V tile.
    const int lt = tid - (kSoftmaxThreads + 32);         // 0..95
    using NT = std::integral_constant<int, kLoaderThreads>;
    auto issue_tile = [&](int ti) { fetch_tile(ti, lt, NT(), ti != 0, true); cp_async_commit(); };
    // Two tiles are put in flight at once; afterwards tile ti+2 can only be fetched once P V of
    // tile ti has released its stage.  A tile is always published BEFORE the loader waits for a
    // stage to be released: the issuer runs Q K^T of tile ti+1 ahead of P V of tile ti, so the
    // release of tile ti's stage depends on tile ti+1 having been published.
    issue_tile(0);
    if (n_tiles > 1) { issue_tile(1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
    fence_async_proxy();             // cp.async writes -> visible to the tensor-core proxy
    mbar_arrive(bar_kv0);            // tile 0
    for (int ti = 0; ti + 1 < n_tiles; ++ti) {
      cp_async_wait<0>();            // tile ti+1 has landed
      fence_async_proxy();
      mbar_arrive(bar_kv0 + 8u * (uint32_t)((ti + 1) & 1));
      if (ti + 2 < n_tiles) {
        if (!mbar_wait(bar_free0 + 8u * (uint32_t)(ti & 1), (uint32_t)((ti >> 1) & 1), abort_flag)) break;
        issue_tile(ti + 2);
      }
    }
    cp_async_wait<0>();
  } else if (warp == 8) {
    // ---- MMA issuer: descriptors are built once, each MMA costs one add ----------------------------
    if ((tid & 31) == 0) {
      const uint32_t idesc_qk = make_idesc(kKeys, 0);
      const uint32_t idesc_pv = make_idesc(D, 1);
      uint64_t dq_hi[D / 16], dq_lo[D / 16];
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        // k-step ks: block ks/4 of 64 elements, 32 bytes per step inside the 128-byte row
        const uint32_t qo = (uint32_t)(ks >> 2) * (kRows * 128) + (uint32_t)(ks & 3) * 32u;
        dq_hi[ks] = make_desc(base + L::kQhi + qo, 16, 1024);
        dq_lo[ks] = make_desc(base + L::kQlo + qo, 16, 1024);
      }
      uint64_t dk0[2], dv0[2];
#pragma unroll
      for (int st = 0; st < 2; ++st) {
        dk0[st] = make_desc(base + L::kK + (uint32_t)st * L::kKStage, 16, 1024);            // K tile (later P), K-major
        dv0[st] = make_desc(base + L::kV + (uint32_t)st * L::kKVBytes, kKeys * 128, 1024);  // V tile, MN-major
      }
      auto issue_qk = [&](int t) {
        const uint32_t tmem_s = tmem + 128u * (uint32_t)(t & 1);
        const uint64_t dk = dk0[t & 1];
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t dkk = dk + (uint64_t)(((ks >> 2) * (kKeys * 128) + (ks & 3) * 32) >> 4);
          if (ks == 0) umma_new(tmem_s, dq_hi[ks], dkk, idesc_qk); else umma_acc(tmem_s, dq_hi[ks], dkk, idesc_qk);
          umma_acc(tmem_s, dq_lo[ks], dkk, idesc_qk);
        }
        umma_commit(bar_s0 + 8u * (uint32_t)(t & 1));
      };
      bool ok = mbar_wait(bar_q, 0, abort_flag);                 // Q and K(0)
      if (ok) { tc_fence_after(); issue_qk(0); }
      ok = ok && mbar_wait(bar_kv0, 0, abort_flag);              // V(0)
      for (int ti = 0; ti < n_tiles && ok; ++ti) {
        if (ti + 1 < n_tiles) {      // next S tile first: it has a whole softmax of lead time
          ok = mbar_wait(bar_kv0 + 8u * (uint32_t)((ti + 1) & 1), (uint32_t)(((ti + 1) >> 1) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_qk(ti + 1);
        }
        ok = mbar_wait(bar_p, (uint32_t)(ti & 1), abort_flag);   // P(ti) in place
        if (!ok) break;
        tc_fence_after();
        const uint64_t dp = dk0[ti & 1], dv = dv0[ti & 1];
#pragma unroll
        for (int kk = 0; kk < kKeys / 16; ++kk) {
          // A = P, K-major: 64-key blocks of kRows*128 bytes, 32 bytes per 16 keys inside a block.
          // B = V, MN-major: 16 key rows = 2048 bytes further per step.
          const uint64_t dpk = dp + (uint64_t)(((kk >> 2) * (kRows * 128) + (kk & 3) * 32) >> 4);
          const uint64_t dvk = dv + (uint64_t)((kk * 2048) >> 4);
          const uint32_t tmem_ob = tmem_o + 128u * (uint32_t)(ti & 1);
          if (kk == 0) umma_new(tmem_ob, dpk, dvk, idesc_pv); else umma_acc(tmem_ob, dpk, dvk, idesc_pv);
        }
        umma_commit(bar_o0 + 64u * (uint32_t)(ti & 1));
        umma_commit(bar_free0 + 8u * (uint32_t)(ti & 1));
      }
    }
  } else {
    // ---- softmax / accumulation threads: two per row --------------------------------------------------
    const int row = tid & 127, half = tid >> 7;
    const int tok = r0 + (row & 15);
    // Q tile (hi and lo) -> shared memory
    for (int idx = tid; idx < kRows * CPR; idx += kSoftmaxThreads) {
      const int r = idx / CPR, c = idx - r * CPR;
      const int gg = r >> 4, tt = r0 + (r & 15);
      const bool valid = (gg < G) && (tt < rps);
      const size_t off = valid ? (((size_t)b * rps + tt) * a.Hq + (size_t)hkv * G + gg) * D + c * 8 : 0;
      cp_async16(base + L::kQhi + sw_off<kRows>(r, c), a.q + off, valid);
      cp_async16(base + L::kQlo + sw_off<kRows>(r, c), a.q_lo + off, valid);
    }
    fetch_tile(0, tid, std::integral_constant<int, kSoftmaxThreads>(), true, false);
    cp_async_commit();
    cp_async_wait<0>();
    fence_async_proxy();
    mbar_arrive(bar_q);

    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;   // warp w may touch TMEM lanes 32*(w%4)..+31
    float o_acc[DH];
#pragma unroll
    for (int i = 0; i < DH; ++i) o_acc[i] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;      // m_run in the log2 domain (score * scale_log2e)
    const float scale = a.scale_log2e;
    const int lim = min(total, (causal_start == 0x3fffffff) ? total : causal_start + tok + 1);  // first invisible key
    bool ok = true;
    // O(ti) = P(ti) V(ti) is folded into the row one tile late, after P(ti+1) has been handed to
    // the tensor core, so the softmax of a tile overlaps the P V product of the tile before it
    // (two O buffers in TMEM): o = o * alpha(ti) + O(ti) with alpha(ti) = 2^(m(ti-1) - m(ti)).
    float alpha_prev = 0.f;
    auto fold_o = [&](int t, float al) {
      if (!mbar_wait(bar_o0 + 64u * (uint32_t)(t & 1), (uint32_t)((t >> 1) & 1), abort_flag)) return false;
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < DH; c0 += 32) {
        float tv[32];
        tmem_ld32(tmem_o + 128u * (uint32_t)(t & 1) + lane_base + DH * half + c0, tv);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) o_acc[c0 + j] = fmaf(o_acc[c0 + j], al, tv[j]);
      }
      tc_fence_before();
      return true;
    };

    for (int ti = 0; ti < n_tiles; ++ti) {
      const uint32_t tmem_s = tmem + 128u * (uint32_t)(ti & 1);
      ok = ok && mbar_wait(bar_s0 + 8u * (uint32_t)(ti & 1), (uint32_t)((ti >> 1) & 1), abort_flag);
      tc_fence_after();
      const int v0 = ti * kKeys + KH * half;       // first key of this thread's half tile
      // a tile needs masking at the ragged end of the key axis, around the bank's free slot and
      // on the causal diagonal (uniform over the CTA)
      const bool need_mask = ((ti + 1) * kKeys > min(total, causal_start + r0 + 1)) ||
                             (hole >= ti * kKeys && hole < (ti + 1) * kKeys) || (a.chunk_mode && (ti >= 128 || tile_excl[ti]));
      float mx = -INFINITY;
      float sc[KH];
      if (ok) {
        tmem_ld32(tmem_s + lane_base + KH * half, sc);
        tmem_ld32(tmem_s + lane_base + KH * half + 32, sc + 32);
        tmem_ld_wait();
        if (need_mask && a.chunk_mode) {
          const int nvis = lim - v0, e0 = v0 - bank_begin;          // e0: this thread's first key on the bank axis
#pragma unroll
          for (int j = 0; j < KH; ++j) {
            const int e = e0 + j;
            const bool out = (unsigned)e < (unsigned)excl_range && ((excl[e >> 5] >> (e & 31)) & 1u);
            sc[j] = (j < nvis && !out) ? sc[j] : -INFINITY;
            mx = fmaxf(mx, sc[j]);
          }
        } else if (need_mask) {
          const int nvis = lim - v0, hj = hole - v0;
#pragma unroll
          for (int j = 0; j < KH; ++j) {
            sc[j] = (j < nvis && j != hj) ? sc[j] : -INFINITY;
            mx = fmaxf(mx, sc[j]);
          }
        } else {
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
          for (int j = 0; j < KH; j += 4) {
            m0 = fmaxf(m0, sc[j]); m1 = fmaxf(m1, sc[j + 1]); m2 = fmaxf(m2, sc[j + 2]); m3 = fmaxf(m3, sc[j + 3]);
          }
          mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        }
      }
      max_x[(ti & 1) * 256 + half * 128 + row] = mx;
      if (!softmax_barrier_and(ok)) { ok = false; break; }      // uniform over the 256 threads
      mx = fmaxf(mx, max_x[(ti & 1) * 256 + (half ^ 1) * 128 + row]) * scale;   // scale > 0: max commutes with it
      const float m_new = fmaxf(m_run, mx);
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
      const float alpha = ex2_approx(m_run - m_use);               // ex2(-inf) = 0 on the first tile
      m_run = m_new;
      float rs0 = 0.f, rs1 = 0.f;
      // S(ti) is complete, so the K tile is dead: P takes its place
      uint8_t* ptile = gbase + L::kK + (size_t)(ti & 1) * L::kKStage;
#pragma unroll
      for (int c = 0; c < KH / 8; ++c) {
        float p[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) p[j] = ex2_approx(fmaf(sc[c * 8 + j], scale, -m_use));
        rs0 += (p[0] + p[1]) + (p[2] + p[3]);
        rs1 += (p[4] + p[5]) + (p[6] + p[7]);
        uint4 pk;
        __nv_bfloat162 t0 = __floats2bfloat162_rn(p[0], p[1]), t1 = __floats2bfloat162_rn(p[2], p[3]);
        __nv_bfloat162 t2 = __floats2bfloat162_rn(p[4], p[5]), t3 = __floats2bfloat162_rn(p[6], p[7]);
        pk.x = *reinterpret_cast<uint32_t*>(&t0); pk.y = *reinterpret_cast<uint32_t*>(&t1);
        pk.z = *reinterpret_cast<uint32_t*>(&t2); pk.w = *reinterpret_cast<uint32_t*>(&t3);
        *reinterpret_cast<uint4*>(ptile + sw_off<kRows>(row, (KH / 8) * half + c)) = pk;
      }
      l_run = l_run * alpha + (rs0 + rs1);
      fence_async_proxy();           // P stores -> visible to the tensor-core proxy
      tc_fence_before();
      mbar_arrive(bar_p);

      if (ti >= 1) ok = fold_o(ti - 1, alpha_prev);
      alpha_prev = alpha;
    }
    if (ok && n_tiles >= 1) ok = fold_o(n_tiles - 1, alpha_prev);

    // the two halves of a row hold partial sums of the softmax denominator
    max_x[half * 128 + row] = l_run;
    const bool all_ok = softmax_barrier_and(ok);
    l_run += max_x[(half ^ 1) * 128 + row];

    // Every MMA has completed, so the Q tiles are dead: the normalised rows go through them
    // (fp32, 16-byte units XOR-swizzled by the row) and leave as whole contiguous rows.
    constexpr int F4 = D / 4;                                      // float4 units per row
    if (all_ok) {
      float4* stage_o = reinterpret_cast<float4*>(gbase + L::kQhi);
      const float inv = (l_run > 0.f) ? 1.f / l_run : 0.f;
#pragma unroll
      for (int c = 0; c < DH; c += 4)
        stage_o[row * F4 + (((DH * half + c) >> 2) ^ (row & (F4 - 1)))] =
            make_float4(o_acc[c] * inv, o_acc[c + 1] * inv, o_acc[c + 2] * inv, o_acc[c + 3] * inv);
    }
    if (!all_ok) *abort_flag = 1;
  }

  // ---- rows out: all 12 warps, a warp per row, four rows' reads ahead of their stores ---------------
  __syncthreads();
  if (!*abort_flag) {
    constexpr int F4 = D / 4;
    constexpr int kWarps = kAttnThreads / 32;
    const float4* stage_o = reinterpret_cast<const float4*>(gbase + L::kQhi);
    const int lane = tid & 31;
    const int G = a.Hq / a.Hkv;
    const int rps = bp.rows_per_stream;
    const int b = blockIdx.z, hkv = blockIdx.y;
    const int r0 = ((int)blockIdx.x - a.bank_blocks) * kTok;
    for (int rb = warp; rb < kRows; rb += 4 * kWarps) {
      float4 v[4];
      bool valid[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int r = rb + k * kWarps;
        valid[k] = r < kRows && (r >> 4) < G && r0 + (r & 15) < rps && lane < F4;      // row part uniform over the warp
        if (valid[k]) v[k] = stage_o[r * F4 + (lane ^ (r & (F4 - 1)))];
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (!valid[k]) continue;
        const int r = rb + k * kWarps;
        const int gg = r >> 4, tt = r0 + (r & 15);
        const size_t obase = (((size_t)b * rps + tt) * a.Hq + (size_t)hkv * G + gg) * D;
        const int u = lane;
        if (a.out_fp32) {
          *reinterpret_cast<float4*>(static_cast<float*>(a.out) + obase + 4 * u) = v[k];
        } else {
          __nv_bfloat162 lo = __floats2bfloat162_rn(v[k].x, v[k].y), hi = __floats2bfloat162_rn(v[k].z, v[k].w);
          uint2 w; w.x = *reinterpret_cast<uint32_t*>(&lo); w.y = *reinterpret_cast<uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(static_cast<bf16*>(a.out) + obase + 4 * u) = w;
        }
        if (a.h_out != nullptr) {
          const uint2 hraw = *reinterpret_cast<const uint2*>(a.h_in + obase + 4 * u);
          const float2 h0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hraw.x));
          const float2 h1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hraw.y));
          __nv_bfloat162 lo = __floats2bfloat162_rn(h0.x + v[k].x, h0.y + v[k].y), hi = __floats2bfloat162_rn(h1.x + v[k].z, h1.y + v[k].w);
          uint2 w; w.x = *reinterpret_cast<uint32_t*>(&lo); w.y = *reinterpret_cast<uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(a.h_out + obase + 4 * u) = w;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
  if (tid == 0 && *abort_flag) atomicExch(status, VS_ERR_DEVICE_TIMEOUT);
}

}  // namespace

cudaError_t prefill_attention_tc_init() {
  cudaError_t e = cudaFuncSetAttribute(prefill_attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Smem<128>::kTotal);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(prefill_attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Smem<64>::kTotal);
}

cudaError_t launch_prefill_attention_tc(const AttnArgs& a, const BatchParams& bp, int* status, cudaStream_t st) {
  dim3 grid((bp.rows_per_stream + kTok - 1) / kTok + a.bank_blocks, a.Hkv, bp.n_active);
  if (a.D == 128) return launch_pdl(prefill_attn_tc_kernel<128>, grid, dim3(kAttnThreads), (size_t)Smem<128>::kTotal, st, a, bp, status);
  if (a.D == 64) return launch_pdl(prefill_attn_tc_kernel<64>, grid, dim3(kAttnThreads), (size_t)Smem<64>::kTotal, st, a, bp, status);
  return cudaErrorInvalidValue;
}

}  // namespace vs
