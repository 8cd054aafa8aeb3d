// Frame-prefill / multi-token attention on the 5th-generation tensor cores
// (Eq. 1: Y = Softmax(Q K^T / sqrt(d_k)) V, grouped KV heads).
//
// One CTA = 16 query tokens x one KV head x one stream (x one share of the key tiles).  The G
// query heads of the group are stacked on the MMA's M axis (row = g * 16 + token, G * 16 <= 128),
// so K and V are staged once for the whole group.  Keys come from up to four segments -- prompt
// prefix, carrier bank (the free slot is masked), earlier text of the turn, the step's own rows
// (causal) -- laid end to end, each starting on a multiple of 64 keys (the padding is masked),
// and cut into tiles of 128 keys.  The carrier is the last row of its frame (Section 3.2), so
// the causal rule alone gives it the whole frame.
// Per tile:  S = Q K^T  (tcgen05.mma, M 128 x N 128, Q as a bf16 hi + lo pair)     -> TMEM
//            softmax of the row in registers, P (bf16) -> TMEM, over the columns of S (tcgen05.st)
//            O += P V  (tcgen05.mma, A = P from TMEM, M 128 x N D, V read MN-major) -> TMEM; the rows
//            of O are rescaled in TMEM only when a row's maximum grows by more than 2^8
// Warps 0..15: four threads per row (each owns 32 keys of a tile and D/4 output dims).
// Warp 16: one thread issues every MMA, one tile of Q K^T ahead of the softmax (S is double
// buffered in TMEM); descriptors are built once.  Warps 17 and 18: one thread each fetches the K
// tiles (and Q), resp. the V tiles, by bulk tensor copies (TMA, boxes of 64 keys x 64 dims through
// per-segment tensor maps, 128-byte swizzle as the MMA descriptors expect), two tiles in flight
// (a K stage is free again once Q K^T has read it, a V stage once P V has); tiles that hold only
// keys of earlier steps (prefix, bank, tail) are requested before the wait on the stream's
// earlier kernels.  The query tile arrives by one bulk copy when the projection left it in
// operand layout.
// The key tiles of a row tile may be shared by the CTAs of a thread-block cluster: each takes a
// contiguous run of tiles, leaves its unnormalised rows with their (max, denominator) in its own
// shared memory, and after the cluster's barrier every CTA finishes the rows of some tokens,
// reading the peers' parts through distributed shared memory.  All mbarrier waits are bounded.
#include "vs_common.cuh"
#include "vs_bank_update.cuh"

namespace vs {

namespace {

constexpr int kKeys = 128;       // keys per tile
constexpr int kRows = 128;       // MMA M
constexpr int kTok = 16;         // query tokens per CTA
constexpr int kBox = ATTN_KEY_BOX;   // key rows per bulk tensor copy
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
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// untiled bulk copy: both addresses 16-byte aligned, size a multiple of 16
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
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
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
// A operand from tensor memory (128 lanes x 8 columns per 16 bf16 of K, two elements per column)
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
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
__device__ __forceinline__ void tmem_ld16f(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 consecutive 32-bit columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

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
  static constexpr int kK = 2 * kQBytes;                  // [stage] K tile
  static constexpr int kV = kK + 2 * kKVBytes;            // [stage] V tile
  static constexpr int kMax = kV + 2 * kKVBytes;          // float [2][4][128]: row maxima exchange
  static constexpr int kLsum = kMax + 4096;               // float [4][128]: the row parts' softmax denominators
  static constexpr int kRowML = kLsum + 2048;             // float2 [128]: (max, denominator) of the rows over this CTA's keys
  static constexpr int kCtl = kRowML + 1024;              // barriers, tmem slot, abort flag
  static constexpr int kExcl = kCtl + 128;                // chunk of frames: bitmap of masked bank-axis keys, per-tile flags
  static constexpr int kPartTab = kExcl + ATTN_EXCL_BITS / 8 + 128;   // int4 [128 tiles][4]: masking of each 32-key quarter tile
  static constexpr int kSegTab = kPartTab + 128 * 4 * 16;             // int [16]: the key axis, for tiles beyond the table
  static constexpr int kTotal = kSegTab + 64 + 1024;                  // + alignment slack
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

constexpr int kParts = 4;                                // threads per row: each owns 32 keys of a tile and D/4 output dims
constexpr int kSoftmaxThreads = 128 * kParts;            // warps 0..15: four warps per scheduler hide one another's latency
constexpr int kIssuerWarp = kSoftmaxThreads / 32, kLoaderWarp = kIssuerWarp + 1, kVLoaderWarp = kIssuerWarp + 2;
constexpr int kAttnThreads = kSoftmaxThreads + 96;       // + the MMA issuer's warp + the Q/K loader's + the V loader's

// barrier 1 over the softmax threads, AND-reducing a predicate (keeps their exits uniform)
__device__ __forceinline__ bool softmax_barrier_and(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 512, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred) : "memory");
  return r != 0;
}
static_assert(kSoftmaxThreads == 512, "the named barrier above counts 512 threads");

// ---- thread-block cluster: the key splits of one (row tile, KV head, batch entry) -----------------------
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_shared_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}

// Masking of the 32 keys at padded position `pos` of the key axis described by seg (lengths [0..3], first
// positions [4..7], kinds [8..11], bank segment [12], bank length [13]):
//   x = keys of the quarter tile that exist (before the causal rule), y = index of its first key among the step's
//   own rows (causal rule: key y + j is visible to rows >= y + j) or very negative, z = bank slot of its first key
//   (the free slot is masked) or very large, w = index of its first key on a chunk's bank axis or very negative.
__device__ __forceinline__ int4 quarter_mask(const int* seg, int pos) {
  int4 d = make_int4(0, -(1 << 29), 1 << 29, -(1 << 30));
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const int len = seg[s], beg = seg[4 + s], kind = seg[8 + s];
    if (pos >= beg && pos < beg + ((len + kBox - 1) & ~(kBox - 1))) {
      const int local = pos - beg;
      d.x = len - local;
      d.y = (kind == 3) ? local : -(1 << 29);
      d.z = (s == seg[12]) ? local : (1 << 29);
      d.w = (s == seg[12]) ? local : ((kind == 4) ? seg[13] + local : -(1 << 30));
    }
  }
  return d;
}

constexpr int kMaxSplit = 4;     // most CTAs sharing the key tiles of one row tile (one cluster)

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1) prefill_attn_tc_kernel(const __grid_constant__ AttnArgs a,
                                                                          const __grid_constant__ BatchParams bp, int* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  using L = Smem<D>;
  constexpr int CPR = D / 8;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_s0 = base + L::kCtl;       // +0, +8: S buffer ready (tcgen05.commit)
  const uint32_t bar_o0 = base + L::kCtl + 16;  // P V of a tile complete (tcgen05.commit), one phase per tile
  const uint32_t bar_p = base + L::kCtl + 32;   // P written (512 arrivals)
  const uint32_t bar_k0 = base + L::kCtl + 40;  // +0, +8: K tile landed in a stage (bulk copies' bytes)
  const uint32_t bar_v0 = base + L::kCtl + 56;  // +0, +8: V tile landed in a stage
  const uint32_t bar_vfree0 = base + L::kCtl + 72;  // +0, +8: V stage free again (tcgen05.commit after P V)
  const uint32_t bar_q = base + L::kCtl + 88;   // Q tile copied row by row (512 arrivals)
  const uint32_t bar_qb = base + L::kCtl + 96;  // Q tile fetched by one bulk copy (its bytes)
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::kCtl + 104);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kCtl + 108);
  const uint32_t bar_kfree0 = base + L::kCtl + 112;  // +0, +8: K stage free again (tcgen05.commit after Q K^T)
  float* max_x = reinterpret_cast<float*>(gbase + L::kMax);
  float* l_x = reinterpret_cast<float*>(gbase + L::kLsum);
  float2* row_ml = reinterpret_cast<float2*>(gbase + L::kRowML);                       // [128] (max, denominator) over this CTA's keys
  uint32_t* excl = reinterpret_cast<uint32_t*>(gbase + L::kExcl);                      // [ATTN_EXCL_BITS / 32]
  uint8_t* tile_mask = gbase + L::kExcl + ATTN_EXCL_BITS / 8;                          // [128] tile needs masking
  int4* part_tab = reinterpret_cast<int4*>(gbase + L::kPartTab);                       // [128][4]
  int* seg_tab = reinterpret_cast<int*>(gbase + L::kSegTab);                           // [16]

  const int tid = threadIdx.x, warp = tid >> 5;
  // ---- bank update CTAs (frame steps, last layer): one more plane of the grid.  What they read --
  // carrier embeddings, the bank's order and metadata -- was complete before the kernel ahead of
  // this one let it start, and nothing else in this launch touches what they write.  Their clusters
  // hold no attention CTA, and they take part in no cluster barrier.
  if ((int)blockIdx.y == a.Hkv) {
    pdl_launch_dependents();
    for (int blk = (int)blockIdx.x; blk < a.bank_blocks; blk += (int)gridDim.x) {
      bank_update_block(a.bank, bp, (int)blockIdx.z, blk);
      __syncthreads();
    }
    pdl_wait();      // so that this launch has completed only once the kernel ahead of it has
    return;
  }
  // ---- set-up that needs nothing from earlier kernels: barriers, tensor memory ------------------
  if (tid == 0) {
    mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1);
    mbar_init(bar_o0, 1);
    mbar_init(bar_p, kSoftmaxThreads);
    mbar_init(bar_k0, 1); mbar_init(bar_k0 + 8, 1);
    mbar_init(bar_v0, 1); mbar_init(bar_v0 + 8, 1);
    mbar_init(bar_vfree0, 1); mbar_init(bar_vfree0 + 8, 1);
    mbar_init(bar_kfree0, 1); mbar_init(bar_kfree0 + 8, 1);
    mbar_init(bar_q, kSoftmaxThreads);
    mbar_init(bar_qb, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_proxy();
  }
  if (warp == kIssuerWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // (the key axis below is laid out from the kernel's parameters alone, so it too comes before the wait)
  const int nsplit = a.nsplit;                                // CTAs of the cluster = key splits of this row tile
  const int split = (int)blockIdx.x % nsplit;                 // = rank in the cluster (clusters run along x)
  const int b = blockIdx.z, hkv = blockIdx.y;
  const int r0 = ((int)blockIdx.x / nsplit) * kTok;
  const int rps = bp.rows_per_stream;
  const int sid = bp.stream_id[b];
  const int G = a.Hq / a.Hkv;
  const int count = a.chunk_mode ? a.chunk_count0 : bp.count[b];
  const bool bank_full = (a.M > 0 && count == a.M);

  // ---- the virtual key axis: segments end to end, each starting on a multiple of kBox keys --------
  int seg_len[4], seg_beg[4], seg_kind[4];
  int ptotal = 0, bank_seg = -1, carr_seg = -1, bank_len = 0;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    int len = 0, kind = -1;
    if (s < a.n_seg) {
      kind = a.seg[s].kind;
      if (kind == 0) len = bp.prefix_len[b];
      else if (kind == 1) { len = (a.M == 0) ? 0 : (bank_full ? a.M + 1 : count); bank_seg = s; bank_len = len; }
      else if (kind == 2) len = bp.text_len[b];
      else if (kind == 4) { len = (a.M == 0) ? 0 : b; carr_seg = s; }   // carriers of the chunk's frames before this one
      else len = min(rps, r0 + kTok);                                  // later keys are visible to no row of this tile
    }
    seg_kind[s] = kind; seg_len[s] = len; seg_beg[s] = ptotal;
    ptotal += (len + kBox - 1) & ~(kBox - 1);
  }
  const int n_tiles_all = (ptotal + kKeys - 1) / kKeys;
  // this CTA's share of the row tile's key tiles
  const int t_lo = (n_tiles_all * split) / nsplit, t_hi = (n_tiles_all * (split + 1)) / nsplit;
  const int n_tiles = t_hi - t_lo;
  // segment holding padded position pos (a multiple of 32), or -1 past the end; local = its key index there
  auto find_seg = [&](int pos, int& local) {
    int found = -1;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      if (pos >= seg_beg[s] && pos < seg_beg[s] + ((seg_len[s] + kBox - 1) & ~(kBox - 1))) { found = s; local = pos - seg_beg[s]; }
    }
    return found;
  };
  // what can be said of a tile from the parameters alone: the masking of its four quarters, and
  // whether it needs any -- where a segment ends short of its last box, past the end of the key
  // axis and on the causal diagonal
  if (tid < 4) { seg_tab[tid] = seg_len[tid]; seg_tab[4 + tid] = seg_beg[tid]; seg_tab[8 + tid] = seg_kind[tid]; }
  if (tid == 4) { seg_tab[12] = bank_seg; seg_tab[13] = bank_len; }
  {
    int sg[14];
#pragma unroll
    for (int s = 0; s < 4; ++s) { sg[s] = seg_len[s]; sg[4 + s] = seg_beg[s]; sg[8 + s] = seg_kind[s]; }
    sg[12] = bank_seg; sg[13] = bank_len;
    for (int i = tid; i < 128; i += kAttnThreads) {
      bool m = false;
#pragma unroll
      for (int q = 0; q < kParts; ++q) {
        const int4 d = quarter_mask(sg, (t_lo + i) * kKeys + q * (kKeys / kParts));
        part_tab[i * kParts + q] = d;
        if (d.x < kKeys / kParts || d.y + kKeys / kParts > r0 + 1) m = true;
      }
      tile_mask[i] = m ? 1 : 0;
    }
  }
  if (a.chunk_mode)
    for (int i = tid; i < ATTN_EXCL_BITS / 32; i += kAttnThreads) excl[i] = 0u;

  tc_fence_before();
  __syncthreads();                  // barriers initialised, tensor memory allocated
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_o = tmem + 256;                    // S buffers at columns 0 and 128, O at 256

  // ---- K/V loaders: one thread each, bulk tensor copies ---------------------------------------------
  // A tile is two boxes of kBox keys; each box lies in one segment (or past the end of the key axis,
  // where a row coordinate beyond the tensor makes the copy write zeros).  Local tile i is tile t_lo + i.
  int tiles_issued = 0;
  const bool is_loader = (tid == kLoaderWarp * 32), is_vloader = (tid == kVLoaderWarp * 32);
  auto issue_kv = [&](int i, bool do_k, bool do_v) {
    const uint32_t st = (uint32_t)(i & 1);
    const uint32_t kdst = base + L::kK + st * L::kKVBytes, vdst = base + L::kV + st * L::kKVBytes;
    if (do_k) mbar_arrive_expect_tx(bar_k0 + 8u * st, (uint32_t)L::kKVBytes);
    if (do_v) mbar_arrive_expect_tx(bar_v0 + 8u * st, (uint32_t)L::kKVBytes);
#pragma unroll 1
    for (int u = 0; u < kKeys / kBox; ++u) {
      int local = 0;
      const int s = find_seg((t_lo + i) * kKeys + u * kBox, local);
      const AttnSegment* sg = &a.seg[s < 0 ? 0 : s];
      const int row = (s < 0) ? (1 << 28) : b * sg->rows_per_batch + local;
      const int z = (s < 0) ? 0 : sg->z0 + sid * sg->z_per_stream + hkv;
#pragma unroll
      for (int blk = 0; blk < D / 64; ++blk) {
        const uint32_t off = (uint32_t)(blk * (kKeys * 128) + u * (kBox * 128));
        if (do_k) tma_load_3d(kdst + off, &sg->tk, blk * 64, row, z, bar_k0 + 8u * st);
        if (do_v) tma_load_3d(vdst + off, &sg->tv, blk * 64, row, z, bar_v0 + 8u * st);
      }
    }
  };
  // keys of earlier steps only (prefix, bank, tail): nothing the kernel ahead of this one writes is
  // visible in such a tile (the bank slot it fills is masked or beyond the bank's count)
  auto tile_is_old = [&](int i) {
    bool old = true;
    for (int u = 0; u < kKeys / kBox; ++u) {
      int local = 0;
      const int s = find_seg((t_lo + i) * kKeys + u * kBox, local);
      if (s >= 0 && seg_kind[s] >= 3) old = false;
    }
    return old;
  };
  if (is_loader || is_vloader) {
    while (tiles_issued < min(2, n_tiles) && tile_is_old(tiles_issued)) { issue_kv(tiles_issued, is_loader, is_vloader); ++tiles_issued; }
  }

  VS_STAMP(bp, 2, 0);
  pdl_wait();                       // earlier kernels of the stream have completed
  pdl_launch_dependents();
  VS_STAMP(bp, 2, 1);
  const int hole_local = (bank_full && !a.chunk_mode) ? a.free_slot[sid * a.free_slot_stride] : -1;   // the slot being refilled holds no carrier
  const int hole_tile = (hole_local >= 0 && bank_seg >= 0) ? (seg_beg[bank_seg] + hole_local) / kKeys - t_lo : -1;
  // chunk of frames in one launch: bank-axis keys this frame must not see, as a bitmap
  const int excl_range = (a.chunk_mode && a.M > 0) ? bank_len + b : 0;   // bank slots, then earlier frames' carriers
  if (a.chunk_mode) {
    // tile (of this CTA) holding bank-axis index v
    auto axis_tile = [&](int v) {
      const int pos = (v < bank_len) ? seg_beg[bank_seg < 0 ? 0 : bank_seg] + v : seg_beg[carr_seg < 0 ? 0 : carr_seg] + (v - bank_len);
      return pos / kKeys - t_lo;
    };
    if (tid < b) {
      const int v = a.chunk_victim[tid];
      if (v >= 0 && v < excl_range) {
        atomicOr(&excl[v >> 5], 1u << (v & 31));
        const int ti_ = axis_tile(v);
        if (ti_ >= 0 && ti_ < 128) tile_mask[ti_] = 1;
      }
    }
    if (tid == kAttnThreads - 1 && bank_full) {        // the slot that was free when the chunk began
      const int v = a.free_slot[0];
      atomicOr(&excl[v >> 5], 1u << (v & 31));
      const int ti_ = axis_tile(v);
      if (ti_ >= 0 && ti_ < 128) tile_mask[ti_] = 1;
    }
    __syncthreads();
  }

  if (warp == kLoaderWarp || warp == kVLoaderWarp) {
    if ((is_loader || is_vloader) && n_tiles > 0) {
      const uint32_t q_bytes = 2u * (uint32_t)L::kQBytes;
      if (is_loader && a.q_tiled != nullptr) {
        // the query tile as the projection left it: [hi | lo] in operand layout, one copy
        const int n_rt = (rps + kTok - 1) / kTok;
        const size_t tile = ((size_t)b * n_rt + (size_t)(r0 / kTok)) * a.Hkv + hkv;
        mbar_arrive_expect_tx(bar_qb, q_bytes);
        bulk_load(base + L::kQhi, a.q_tiled + tile * (size_t)(2 * kRows * D), q_bytes, bar_qb);
      }
      while (tiles_issued < min(2, n_tiles)) { issue_kv(tiles_issued, is_loader, is_vloader); ++tiles_issued; }
      // K of tile i+2 can be fetched once Q K^T of tile i has read its stage (P lives in tensor memory),
      // V of tile i+2 once P V of tile i has
      const uint32_t bar_land0 = is_loader ? bar_k0 : bar_v0, bar_done0 = is_loader ? bar_kfree0 : bar_vfree0;
      for (int i = 0; i + 2 < n_tiles; ++i) {
        if (!mbar_wait(bar_done0 + 8u * (uint32_t)(i & 1), (uint32_t)((i >> 1) & 1), abort_flag)) break;
        issue_kv(i + 2, is_loader, is_vloader);
        tiles_issued = i + 3;
      }
      if (*abort_flag) {
        // let the copies in flight land before the shared memory is given up
        for (int i = max(tiles_issued - 2, 0); i < tiles_issued; ++i) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(bar_land0 + 8u * (uint32_t)(i & 1), (uint32_t)((i >> 1) & 1))) {
            if (global_ns() - t0 > kWaitLimitNs) break;
          }
        }
        if (is_loader && a.q_tiled != nullptr) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(bar_qb, 0)) { if (global_ns() - t0 > kWaitLimitNs) break; }
        }
      }
    }
  } else if (warp == kIssuerWarp) {
    // ---- MMA issuer: descriptors are built once, each MMA costs one add ----------------------------
    if ((tid & 31) == 0 && n_tiles > 0) {
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
        dk0[st] = make_desc(base + L::kK + (uint32_t)st * L::kKVBytes, 16, 1024);            // K tile, K-major
        dv0[st] = make_desc(base + L::kV + (uint32_t)st * L::kKVBytes, kKeys * 128, 1024);  // V tile, MN-major
      }
      auto issue_qk = [&](int t) {
        const uint32_t tmem_s = tmem + 128u * (uint32_t)(t & 1);
        const uint64_t dk = dk0[t & 1];
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t dkk = dk + (uint64_t)(((ks >> 2) * (kKeys * 128) + (ks & 3) * 32) >> 4);
          umma_ss(tmem_s, dq_hi[ks], dkk, idesc_qk, (uint32_t)(ks != 0));
          umma_ss(tmem_s, dq_lo[ks], dkk, idesc_qk, 1u);
        }
        umma_commit(bar_s0 + 8u * (uint32_t)(t & 1));
        umma_commit(bar_kfree0 + 8u * (uint32_t)(t & 1));
      };
      bool ok = mbar_wait(a.q_tiled != nullptr ? bar_qb : bar_q, 0, abort_flag);   // Q
      ok = ok && mbar_wait(bar_k0, 0, abort_flag);                                 // K(0)
      if (ok) { tc_fence_after(); issue_qk(0); }
      for (int ti = 0; ti < n_tiles && ok; ++ti) {
        if (ti + 1 < n_tiles) {      // next S tile first: it has a whole softmax of lead time
          ok = mbar_wait(bar_k0 + 8u * (uint32_t)((ti + 1) & 1), (uint32_t)(((ti + 1) >> 1) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_qk(ti + 1);
        }
        ok = mbar_wait(bar_p, (uint32_t)(ti & 1), abort_flag);   // P(ti) in place, O rescaled where needed
        ok = ok && mbar_wait(bar_v0 + 8u * (uint32_t)(ti & 1), (uint32_t)((ti >> 1) & 1), abort_flag);   // V(ti)
        if (!ok) break;
        tc_fence_after();
        const uint64_t dv = dv0[ti & 1];
        const uint32_t tmem_p = tmem + 128u * (uint32_t)(ti & 1);     // P(ti) over the first 64 columns of S(ti)
#pragma unroll
        for (int kk = 0; kk < kKeys / 16; ++kk) {
          // A = P from tensor memory: 16 keys = 8 columns.  B = V, MN-major: 16 key rows = 2048 bytes further per step.
          // One accumulator for all tiles of this CTA.
          umma_ts(tmem_o, tmem_p + 8u * (uint32_t)kk, dv + (uint64_t)((kk * 2048) >> 4), idesc_pv, (uint32_t)((ti | kk) != 0));
        }
        umma_commit(bar_o0);
        umma_commit(bar_vfree0 + 8u * (uint32_t)(ti & 1));
      }
    }
  } else {
    // ---- softmax / accumulation threads: four per row ------------------------------------------------
    constexpr int KP = kKeys / kParts;             // keys of a tile owned by one thread
    constexpr int DP = D / kParts;                 // output dims owned by one thread
    const int row = tid & 127, part = tid >> 7;
    const int tok = r0 + (row & 15);
    if (a.q_tiled == nullptr && n_tiles > 0) {
      // Q rows (hi and lo) as a matrix-vector projection left them -> the operand layout in shared memory
      for (int idx = tid; idx < kRows * CPR; idx += kSoftmaxThreads) {
        const int r = idx / CPR, c = idx - r * CPR;
        const int gg = r >> 4, tt = r0 + (r & 15);
        const bool valid = (gg < G) && (tt < rps);
        const size_t off = valid ? (((size_t)b * rps + tt) * a.Hq + (size_t)hkv * G + gg) * D + c * 8 : 0;
        cp_async16(base + L::kQhi + sw_off<kRows>(r, c), a.q + off, valid);
        cp_async16(base + L::kQlo + sw_off<kRows>(r, c), a.q_lo + off, valid);
      }
      cp_async_commit();
      cp_async_wait<0>();
      fence_async_proxy();
      mbar_arrive(bar_q);
    }

    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;   // warp w may touch TMEM lanes 32*(w%4)..+31
    float m_run = -INFINITY, l_run = 0.f;      // m_run in the log2 domain (score * scale_log2e): the reference of P and O
    const float scale = a.scale_log2e;
    bool ok = true;
    // O accumulates in tensor memory over all tiles.  Its rows -- and l -- are relative to m_run, which follows
    // the row's running maximum lazily: it moves (and the row of O is rescaled, in tensor memory, by the row's
    // four threads, a quarter each) only when the maximum has grown by more than 8, so 2^(score - m_run) <= 2^8.
    constexpr float kLazy = 8.f;

    for (int ti = 0; ti < n_tiles; ++ti) {       // ti: local tile index (tile t_lo + ti of the key axis)
      const uint32_t tmem_s = tmem + 128u * (uint32_t)(ti & 1);
      ok = ok && mbar_wait(bar_s0 + 8u * (uint32_t)(ti & 1), (uint32_t)((ti >> 1) & 1), abort_flag);
      tc_fence_after();
      // uniform over the CTA: the ragged ends, the causal diagonal, the bank's free slot, what a
      // chunk's frame must not see
      const bool need_mask = ti >= 128 || tile_mask[ti] || ti == hole_tile;
      float mx = -INFINITY;
      float sc[KP];
      if (ok) {
        tmem_ld32(tmem_s + lane_base + KP * part, sc);
        tmem_ld_wait();
        if (need_mask) {
          const int4 qd = (ti < 128) ? part_tab[ti * kParts + part] : quarter_mask(seg_tab, (t_lo + ti) * kKeys + KP * part);
          const int nvis = min(qd.x, tok - qd.y + 1);     // key i of the step is visible to rows >= i
          const int hj = hole_local - qd.z;               // the bank's free slot
          const int e0 = qd.w;                            // index on the chunk's bank axis
          if (a.chunk_mode) {
#pragma unroll
            for (int j = 0; j < KP; ++j) {
              const int e = e0 + j;
              const bool out = (unsigned)e < (unsigned)excl_range && ((excl[e >> 5] >> (e & 31)) & 1u);
              sc[j] = (j < nvis && !out) ? sc[j] : -INFINITY;
              mx = fmaxf(mx, sc[j]);
            }
          } else {
#pragma unroll
            for (int j = 0; j < KP; ++j) {
              sc[j] = (j < nvis && j != hj) ? sc[j] : -INFINITY;
              mx = fmaxf(mx, sc[j]);
            }
          }
        } else {
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
          for (int j = 0; j < KP; j += 4) {
            m0 = fmaxf(m0, sc[j]); m1 = fmaxf(m1, sc[j + 1]); m2 = fmaxf(m2, sc[j + 2]); m3 = fmaxf(m3, sc[j + 3]);
          }
          mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        }
      }
      float* mrow = max_x + (ti & 1) * (kParts * 128) + row;
      mrow[part * 128] = mx;
      if (!softmax_barrier_and(ok)) { ok = false; break; }      // uniform over the softmax threads
      mx = fmaxf(fmaxf(mrow[0], mrow[128]), fmaxf(mrow[256], mrow[384])) * scale;   // scale > 0: max commutes with it
      // the row's four threads see the same mx and m_run, so they take the same decision
      const bool move = mx > m_run + kLazy || (m_run == -INFINITY && mx > -INFINITY);
      const float m_new = move ? mx : m_run;
      const float alpha = move ? ex2_approx(m_run - m_new) : 1.f;      // ex2(-inf) = 0: nothing accumulated yet
      m_run = m_new;
      const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
      float rs0 = 0.f, rs1 = 0.f;
      // P(ti), bf16 pairs, goes back into tensor memory over the first 64 columns of S(ti): this thread's
      // 32 keys are columns 16 * part .. + 15.  Every thread of the row has read its scores (the
      // barrier above), so the columns are free.
      {
        uint32_t pw[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float p0 = ex2_approx(fmaf(sc[2 * j], scale, -m_use));
          const float p1 = ex2_approx(fmaf(sc[2 * j + 1], scale, -m_use));
          if (j & 1) rs1 += p0 + p1; else rs0 += p0 + p1;
          const __nv_bfloat162 t = __floats2bfloat162_rn(p0, p1);
          pw[j] = *reinterpret_cast<const uint32_t*>(&t);
        }
        tmem_st16(tmem_s + lane_base + 16u * (uint32_t)part, pw);
      }
      l_run = l_run * alpha + (rs0 + rs1);
      // The tile before must have been added to O before this tile's P V may follow it.  Every thread
      // waits for it, every tile: a parity wait tells the phase in progress from the one before it and
      // nothing older, so a thread that skipped phases would take a stale phase for the one it wants.
      if (ti >= 1 && !mbar_wait(bar_o0, (uint32_t)((ti - 1) & 1), abort_flag)) ok = false;
      // rows whose reference moved: O *= alpha (uniform over the warp)
      if (ti >= 1 && __any_sync(0xffffffffu, move)) {
        tc_fence_after();
        float tv[DP];
        if constexpr (DP == 32) tmem_ld32(tmem_o + lane_base + DP * part, tv); else tmem_ld16f(tmem_o + lane_base + DP * part, tv);
        tmem_ld_wait();
        uint32_t tw[DP];
#pragma unroll
        for (int j = 0; j < DP; ++j) tw[j] = __float_as_uint(tv[j] * alpha);
        tmem_st16(tmem_o + lane_base + DP * part, tw);
        if constexpr (DP == 32) tmem_st16(tmem_o + lane_base + DP * part + 16, tw + 16);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bar_p);
    }
    // the accumulated rows: this thread's quarter
    float o_acc[DP];
#pragma unroll
    for (int i = 0; i < DP; ++i) o_acc[i] = 0.f;
    if (ok && n_tiles >= 1) {
      ok = mbar_wait(bar_o0, (uint32_t)((n_tiles - 1) & 1), abort_flag);
      tc_fence_after();
      if constexpr (DP == 32) tmem_ld32(tmem_o + lane_base + DP * part, o_acc); else tmem_ld16f(tmem_o + lane_base + DP * part, o_acc);
      tmem_ld_wait();
      tc_fence_before();
    }

    // the four threads of a row hold partial sums of the softmax denominator
    l_x[part * 128 + row] = l_run;
    const bool all_ok = softmax_barrier_and(ok);
    l_run = (l_x[row] + l_x[128 + row]) + (l_x[256 + row] + l_x[384 + row]);

    // Every MMA has completed, so the Q tiles are dead: this CTA's part of the rows -- the sum over
    // its keys of 2^(score - max) V, not yet normalised -- goes through them (fp32, 16-byte units
    // XOR-swizzled by the row) with the row's (max, denominator) beside it.
    constexpr int F4 = D / 4;                                      // float4 units per row
    {
      float4* stage_o = reinterpret_cast<float4*>(gbase + L::kQhi);
#pragma unroll
      for (int c = 0; c < DP; c += 4)
        stage_o[row * F4 + (((DP * part + c) >> 2) ^ (row & (F4 - 1)))] =
            make_float4(o_acc[c], o_acc[c + 1], o_acc[c + 2], o_acc[c + 3]);
      if (part == 0) row_ml[row] = make_float2(m_run, l_run);
    }
    if (!all_ok) *abort_flag = 1;
  }

  // ---- rows out.  The nsplit CTAs of the cluster hold the parts of the same 128 rows over their
  // own key tiles; CTA `split` finishes the rows of tokens split, split + nsplit, ... (all heads of
  // a token, so that the token's sum of squares can be formed here): it reads the parts of such a
  // row from every CTA's shared memory, weighs them by 2^(max_i - max), normalises, adds the
  // residual and stores the row.  A warp per row, four rows in flight.
  __syncthreads();
  VS_STAMP(bp, 2, 2);               // this CTA's tiles done
  if (nsplit > 1) cluster_arrive(); // this CTA's parts are in place; the peers' are waited for below
  float* ss_stage = max_x;          // [8 heads][16 tokens]: sum of squares of the stored residual rows (dead memory by now)
  {
    constexpr int F4 = D / 4;
    constexpr int kWarps = kAttnThreads / 32;
    const int lane = tid & 31;
    const uint32_t stage_addr = base + L::kQhi, ml_addr = base + L::kRowML;
    uint32_t peer_o[kMaxSplit], peer_ml[kMaxSplit];
#pragma unroll
    for (int s = 0; s < kMaxSplit; ++s) {
      peer_o[s] = (s < nsplit && nsplit > 1) ? map_shared_rank(stage_addr, (uint32_t)s) : stage_addr;
      peer_ml[s] = (s < nsplit && nsplit > 1) ? map_shared_rank(ml_addr, (uint32_t)s) : ml_addr;
    }
    const float4* stage_o = reinterpret_cast<const float4*>(gbase + L::kQhi);
    const int my_tokens = (kTok - split + nsplit - 1) / nsplit;       // tokens split, split + nsplit, ... < 16
    const int my_rows = my_tokens * 8;                                // row j: head j % 8 of my token j / 8
    // the residual input of this warp's first rows is asked for while the peers finish
    uint2 hpre[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int j = warp + k * kWarps;
      const int r = (j & 7) * 16 + split + (j >> 3) * nsplit;
      hpre[k] = make_uint2(0u, 0u);
      if (a.h_out != nullptr && j < my_rows && (r >> 4) < G && r0 + (r & 15) < rps && lane < F4)
        hpre[k] = *reinterpret_cast<const uint2*>(a.h_in + (((size_t)b * rps + r0 + (r & 15)) * a.Hq + (size_t)hkv * G + (r >> 4)) * D + 4 * lane);
    }
    if (nsplit > 1) cluster_wait();
    VS_STAMP(bp, 2, 3);
    for (int jb = warp; jb < my_rows; jb += 4 * kWarps) {
      float4 v[4];
      bool valid[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int j = jb + k * kWarps;
        const int r = (j & 7) * 16 + split + (j >> 3) * nsplit;
        valid[k] = j < my_rows && (r >> 4) < G && r0 + (r & 15) < rps;      // uniform over the warp
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!valid[k] || lane >= F4) continue;
        const uint32_t off = (uint32_t)((r * F4 + (lane ^ (r & (F4 - 1)))) * 16);
        if (nsplit == 1) {
          const float2 ml = row_ml[r];
          const float inv = (ml.y > 0.f) ? 1.f / ml.y : 0.f;
          const float4 o = stage_o[r * F4 + (lane ^ (r & (F4 - 1)))];
          v[k] = make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
        } else {
          float2 ml[kMaxSplit];
          float4 o[kMaxSplit];
#pragma unroll
          for (int s = 0; s < kMaxSplit; ++s) {
            if (s < nsplit) { ml[s] = ld_cluster_f2(peer_ml[s] + (uint32_t)r * 8u); o[s] = ld_cluster_f4(peer_o[s] + off); }
          }
          float mm = -INFINITY;
#pragma unroll
          for (int s = 0; s < kMaxSplit; ++s) if (s < nsplit) mm = fmaxf(mm, ml[s].x);
          float den = 0.f;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int s = 0; s < kMaxSplit; ++s) {
            if (s < nsplit) {
              const float w = (ml[s].x == -INFINITY) ? 0.f : ex2_approx(ml[s].x - mm);   // a CTA without visible keys adds nothing
              den = fmaf(ml[s].y, w, den);
              acc.x = fmaf(o[s].x, w, acc.x); acc.y = fmaf(o[s].y, w, acc.y);
              acc.z = fmaf(o[s].z, w, acc.z); acc.w = fmaf(o[s].w, w, acc.w);
            }
          }
          const float inv = (den > 0.f) ? 1.f / den : 0.f;
          v[k] = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (!valid[k]) continue;
        const int j = jb + k * kWarps;
        const int r = (j & 7) * 16 + split + (j >> 3) * nsplit;
        const int gg = r >> 4, tt = r0 + (r & 15);
        const size_t obase = (((size_t)b * rps + tt) * a.Hq + (size_t)hkv * G + gg) * D;
        const int u = lane;
        float ss = 0.f;
        if (lane < F4) {
          if (a.out == nullptr) {
            // a layer whose rows only feed the residual stream
          } else if (a.out_fp32) {
            *reinterpret_cast<float4*>(static_cast<float*>(a.out) + obase + 4 * u) = v[k];
          } else {
            __nv_bfloat162 lo = __floats2bfloat162_rn(v[k].x, v[k].y), hi = __floats2bfloat162_rn(v[k].z, v[k].w);
            uint2 w; w.x = *reinterpret_cast<uint32_t*>(&lo); w.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(static_cast<bf16*>(a.out) + obase + 4 * u) = w;
          }
          if (a.h_out != nullptr) {
            const uint2 hraw = (jb == warp) ? hpre[k] : *reinterpret_cast<const uint2*>(a.h_in + obase + 4 * u);
            const float2 h0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hraw.x));
            const float2 h1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hraw.y));
            __nv_bfloat162 lo = __floats2bfloat162_rn(h0.x + v[k].x, h0.y + v[k].y), hi = __floats2bfloat162_rn(h1.x + v[k].z, h1.y + v[k].w);
            uint2 w; w.x = *reinterpret_cast<uint32_t*>(&lo); w.y = *reinterpret_cast<uint32_t*>(&hi);
            if (VS_STORE_OK(bp, a.h_out_region, a.h_out + obase + 4 * u, 8)) *reinterpret_cast<uint2*>(a.h_out + obase + 4 * u) = w;
            if (a.ss_out != nullptr) {
              // RMSNorm of the next layer: its statistics are those of the rows as stored (bf16)
              const float2 s0 = __bfloat1622float2(lo), s1 = __bfloat1622float2(hi);
              ss = (s0.x * s0.x + s0.y * s0.y) + (s1.x * s1.x + s1.y * s1.y);
              if (a.next_gain != nullptr) {
                // ... and, with a gain vector, the projection reads bf16(h * gain) instead of h
                const uint2 graw = *reinterpret_cast<const uint2*>(a.next_gain + ((size_t)hkv * G + gg) * D + 4 * u);
                const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&graw.x));
                const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&graw.y));
                __nv_bfloat162 x0 = __floats2bfloat162_rn(s0.x * g0.x, s0.y * g0.y), x1 = __floats2bfloat162_rn(s1.x * g1.x, s1.y * g1.y);
                uint2 xw; xw.x = *reinterpret_cast<uint32_t*>(&x0); xw.y = *reinterpret_cast<uint32_t*>(&x1);
                if (VS_STORE_OK(bp, DR_XN, a.xn_out + obase + 4 * u, 8)) *reinterpret_cast<uint2*>(a.xn_out + obase + 4 * u) = xw;
              }
            }
          }
        }
        if (a.ss_out != nullptr) {
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
          if (lane == 0) ss_stage[gg * 16 + (r & 15)] = ss;
        }
      }
    }
    if (a.ss_out != nullptr) {
      // the token's sum of squares over this KV head's query heads, in head order; the projection adds
      // the KV heads' parts in order: the same bits whatever the launch shape
      __syncthreads();
      if (tid < kTok && tid % nsplit == split && r0 + tid < rps) {
        float tot = 0.f;
        for (int gg = 0; gg < G; ++gg) tot += ss_stage[gg * 16 + tid];
        float* sp = a.ss_out + ((size_t)b * rps + r0 + tid) * a.Hkv + hkv;
        if (VS_STORE_OK(bp, DR_ROW_SS, sp, 4)) *sp = tot;
      }
    }
  }
  // nobody's shared memory goes away while a peer may still be reading it
  if (nsplit > 1) { cluster_arrive(); cluster_wait(); }

  tc_fence_before();
  __syncthreads();
  if (warp == kIssuerWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
  if (tid == 0 && *abort_flag) atomicExch(status, VS_ERR_DEVICE_TIMEOUT);
  VS_STAMP(bp, 2, 15);
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
  if (a.nsplit < 1 || a.nsplit > kMaxSplit) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(((bp.rows_per_stream + kTok - 1) / kTok) * a.nsplit, a.Hkv + (a.bank_blocks > 0 ? 1 : 0), bp.n_active);
  cfg.blockDim = dim3(kAttnThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;            // the key splits of a row tile are one cluster
  attr[1].val.clusterDim.x = a.nsplit; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.nsplit > 1 ? 2 : 1;
  if (a.D == 128) { cfg.dynamicSmemBytes = Smem<128>::kTotal; return cudaLaunchKernelEx(&cfg, prefill_attn_tc_kernel<128>, a, bp, status); }
  if (a.D == 64) { cfg.dynamicSmemBytes = Smem<64>::kTotal; return cudaLaunchKernelEx(&cfg, prefill_attn_tc_kernel<64>, a, bp, status); }
  return cudaErrorInvalidValue;
}

// Clusters of `s` CTAs of this kernel that can be resident at once (every CTA takes a whole SM and a
// cluster's CTAs sit in one GPC); 0 if the query fails.  Asked once per handle.
int prefill_attention_max_clusters(int head_dim, int s) {
  if (s < 2 || s > kMaxSplit) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(s * 64); cfg.blockDim = dim3(kAttnThreads);
  cfg.dynamicSmemBytes = head_dim == 128 ? Smem<128>::kTotal : Smem<64>::kTotal;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = s; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int clusters = 0;
  const cudaError_t e = head_dim == 128 ? cudaOccupancyMaxActiveClusters(&clusters, prefill_attn_tc_kernel<128>, &cfg)
                                        : cudaOccupancyMaxActiveClusters(&clusters, prefill_attn_tc_kernel<64>, &cfg);
  if (e != cudaSuccess) { cudaGetLastError(); return 0; }
  return clusters;
}

}  // namespace vs
