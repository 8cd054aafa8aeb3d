// vs_evict_choose_static: the eviction decision of the memory mechanism (largest cosine
// similarity, oldest on ties) as a stand-alone call for callers that cannot allocate device
// memory.  Its scratch (per-carrier scores and the block counter of the last-block argmax)
// lives in a file-scope __device__ array instead of a caller workspace.
#include <mutex>

#include "vs_common.cuh"

namespace {

constexpr int kStaticMaxBank = VS_STATIC_MAX_BANK;
constexpr int kMaxDevices = 64;

struct __align__(256) StaticScratch {
  double scores[kStaticMaxBank];
  int ticket;
};

// Held by every GPU that loads the library until the process exits: 32 KiB + 256 B.
static __device__ __align__(256) StaticScratch g_evict_scratch;

__device__ __forceinline__ double tree_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Same arithmetic and summation order as the library's in-stream scoring kernel: lane p adds
// elements k = p (mod 32) in ascending k in fp64, then a butterfly 16, 8, 4, 2, 1.
__global__ void __launch_bounds__(256)
evict_choose_static_kernel(const vs::bf16* __restrict__ bank, const vs::bf16* __restrict__ incoming, int count, int d,
                           int policy, StaticScratch* scratch, int* victim_out) {
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (j < count) {
    const vs::bf16* va = bank + (size_t)j * d;
    const vs::bf16* vb = (policy == 1 && j + 1 < count) ? bank + (size_t)(j + 1) * d : incoming;
    double dot = 0.0, na = 0.0, nb = 0.0;
    for (int k = lane; k < d; k += 32) {
      const double x = (double)__bfloat162float(va[k]);
      const double y = (double)__bfloat162float(vb[k]);
      dot = __dadd_rn(dot, __dmul_rn(x, y));
      na = __dadd_rn(na, __dmul_rn(x, x));
      nb = __dadd_rn(nb, __dmul_rn(y, y));
    }
    dot = tree_sum(dot); na = tree_sum(na); nb = tree_sum(nb);
    if (lane == 0) {
      double s = 0.0;
      if (na != 0.0 && nb != 0.0) s = __ddiv_rn(dot, __dmul_rn(__dsqrt_rn(na), __dsqrt_rn(nb)));
      if (!(s >= -2.0 && s <= 2.0)) s = 0.0;          // Inf or NaN in a vector: no cosine, counted as 0
      scratch->scores[j] = s;
    }
  }
  __shared__ int is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(&scratch->ticket, 1) == (int)gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  __shared__ double best_s[256];
  __shared__ int best_j[256];
  double bs = -4.0; int bj = 0x7fffffff;              // every score lies in [-2, 2]
  for (int i = threadIdx.x; i < count; i += blockDim.x) {
    const double s = __ldcg(scratch->scores + i);
    if (s > bs) { bs = s; bj = i; }
  }
  best_s[threadIdx.x] = bs; best_j[threadIdx.x] = bj;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) {
      const double s2 = best_s[threadIdx.x + o]; const int j2 = best_j[threadIdx.x + o];
      if (s2 > best_s[threadIdx.x] || (s2 == best_s[threadIdx.x] && j2 < best_j[threadIdx.x])) {
        best_s[threadIdx.x] = s2; best_j[threadIdx.x] = j2;
      }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    *victim_out = (policy == 2 || (unsigned)best_j[0] >= (unsigned)count) ? 0 : best_j[0];
    scratch->ticket = 0;
  }
}

std::mutex g_setup_mutex;
StaticScratch* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the static array on the current device.  In host code the symbol's name
// is only a handle; the address a kernel can use comes from cudaGetSymbolAddress.
int scratch_for_current_device(StaticScratch** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_evict_scratch) != cudaSuccess || p == nullptr) return VS_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<StaticScratch*>(p);
  }
  *out = g_scratch_addr[dev];
  return VS_OK;
}

}  // namespace

extern "C" int vs_evict_choose_static(const void* bank_emb, const void* incoming, int32_t count, int32_t d_model,
                                      int32_t policy, int32_t* victim_out, void* cuda_stream) {
  if (bank_emb == nullptr || incoming == nullptr || victim_out == nullptr) return VS_ERR_INVALID_ARG;
  if (count < 1 || d_model < 1 || policy < 0 || policy > 2) return VS_ERR_INVALID_ARG;
  if (count > kStaticMaxBank) return VS_ERR_CAPACITY;      // the static scratch holds VS_STATIC_MAX_BANK scores
  StaticScratch* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != VS_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the block counter must start at zero even if an earlier call was cut short
  if (cudaMemsetAsync(&scratch->ticket, 0, sizeof(int), st) != cudaSuccess) return VS_ERR_CUDA;
  evict_choose_static_kernel<<<(count + 7) / 8, 256, 0, st>>>(
      static_cast<const vs::bf16*>(bank_emb), static_cast<const vs::bf16*>(incoming), count, d_model, policy, scratch,
      victim_out);
  return cudaGetLastError() == cudaSuccess ? VS_OK : VS_ERR_CUDA;
}
