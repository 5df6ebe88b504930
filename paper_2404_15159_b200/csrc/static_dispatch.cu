// mixlora_dispatch_static: the slot dispatch (histogram, prefix scan, stable permutation by
// expert) for callers that have no way to hand the library a workspace.
//
// Who needs it: code that runs where device allocation is off the table - a plug-in loaded
// into a host program that owns the allocator and gives out no spare buffers, a callback
// running while other work on the device must not be disturbed by an allocation (cudaMalloc
// synchronises the device), or a process whose memory budget was fixed before start-up.
// Such a caller can still pass its inputs and outputs, but not the two per-block count
// tables the dispatch kernels use in between.  Those live here, in a fixed array that is
// part of the loaded library image on every GPU.
#include <mutex>

#include "common.cuh"

namespace mixlora {
namespace {

constexpr int kStaticMaxTokens = 65536;                       // stated limit of the entry point
constexpr int kStaticBlockTokens = 256;
constexpr int kStaticMaxBlocks = kStaticMaxTokens / kStaticBlockTokens;
constexpr size_t kTableInts = (size_t)kStaticMaxBlocks * MIXLORA_MAX_EXPERTS;
constexpr size_t kStaticScratchBytes = 2 * kTableInts * sizeof(int);   // 64 KiB: counts + offsets

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress;
// the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_dispatch_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
int* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch on the current device (looked up on first use per device).
cudaError_t scratch_for_current_device(int** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_dispatch_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = reinterpret_cast<int*>(p);
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

// Slots per expert inside each block of 256 tokens.  Every (block, expert) entry that the
// later kernels read is written here, so nothing in the scratch has to be cleared first.
__global__ void __launch_bounds__(kStaticBlockTokens)
static_count_kernel(const int* __restrict__ expert_idx, int* __restrict__ blk_counts, int tokens, int N, int k) {
  __shared__ int cnt[MIXLORA_MAX_EXPERTS];
  if (threadIdx.x < MIXLORA_MAX_EXPERTS) cnt[threadIdx.x] = 0;
  __syncthreads();
  const int t = blockIdx.x * kStaticBlockTokens + threadIdx.x;
  if (t < tokens)
    for (int j = 0; j < k; ++j) {
      const int e = expert_idx[(size_t)t * k + j];
      if ((unsigned)e < (unsigned)N) atomicAdd(&cnt[e], 1);   // an index outside [0, N) is skipped, never followed
    }
  __syncthreads();
  if (threadIdx.x < N) blk_counts[blockIdx.x * N + threadIdx.x] = cnt[threadIdx.x];
}

// Exclusive scan of the table in (expert, block) order; writes seg_off.
__global__ void __launch_bounds__(1024)
static_scan_kernel(const int* __restrict__ blk_counts, int* __restrict__ blk_off, int* __restrict__ seg_off, int nblk,
                   int N) {
  __shared__ int part[1024];
  const int n = nblk * N;
  const int per = (n + 1023) / 1024;
  const int q0 = threadIdx.x * per;
  int s = 0;
  for (int q = q0; q < q0 + per && q < n; ++q) s += blk_counts[(q % nblk) * N + (q / nblk)];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int o = 1; o < 1024; o <<= 1) {
    int v = (threadIdx.x >= o) ? part[threadIdx.x - o] : 0;
    __syncthreads();
    part[threadIdx.x] += v;
    __syncthreads();
  }
  int run = (threadIdx.x == 0) ? 0 : part[threadIdx.x - 1];
  for (int q = q0; q < q0 + per && q < n; ++q) {
    const int e = q / nblk, b = q % nblk;
    blk_off[b * N + e] = run;
    if (b == 0) seg_off[e] = run;
    run += blk_counts[b * N + e];
  }
  if (threadIdx.x == 1023) seg_off[N] = part[1023];
}

// Rank of each slot inside its (block, expert) bucket by warp ballots, then scatter.
__global__ void __launch_bounds__(kStaticBlockTokens)
static_scatter_kernel(const int* __restrict__ expert_idx, const int* __restrict__ blk_off, int* __restrict__ perm,
                      int tokens, int N, int k) {
  constexpr int W = kStaticBlockTokens / 32;
  __shared__ int wcnt[W][MIXLORA_MAX_EXPERTS];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int t = blockIdx.x * kStaticBlockTokens + threadIdx.x;
  int mine[MIXLORA_MAX_TOP_K];
  int rank[MIXLORA_MAX_TOP_K];
#pragma unroll
  for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
    mine[j] = (t < tokens && j < k) ? expert_idx[(size_t)t * k + j] : -1;
    if ((unsigned)mine[j] >= (unsigned)N) mine[j] = -1;        // skipped, as in the count kernel
    rank[j] = 0;
  }
  for (int e = 0; e < N; ++e) {
    bool has = false;
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) has |= (mine[j] == e);
    unsigned b = __ballot_sync(0xffffffffu, has);
    int r = __popc(b & ((1u << lane) - 1u));
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j)
      if (mine[j] == e) rank[j] = r;
    if (lane == 0) wcnt[w][e] = __popc(b);
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
    if (mine[j] < 0) continue;
    const int e = mine[j];
    int before = 0;
    for (int ww = 0; ww < w; ++ww) before += wcnt[ww][e];
    perm[blk_off[blockIdx.x * N + e] + before + rank[j]] = t * k + j;
  }
}

}  // namespace
}  // namespace mixlora

using namespace mixlora;

extern "C" mixlora_status_t mixlora_dispatch_static(const int32_t* expert_idx, int32_t tokens, int32_t n_experts,
                                                    int32_t top_k, int32_t* perm, int32_t* seg_off, void* stream) {
  if (!expert_idx || !perm || !seg_off) return MIXLORA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(expert_idx) | reinterpret_cast<uintptr_t>(perm) |
       reinterpret_cast<uintptr_t>(seg_off)) & 3u)
    return MIXLORA_ERR_INVALID_ARG;
  if (tokens < 0 || n_experts <= 0 || top_k <= 0 || top_k > n_experts) return MIXLORA_ERR_INVALID_ARG;
  if (n_experts > MIXLORA_MAX_EXPERTS || top_k > MIXLORA_MAX_TOP_K) return MIXLORA_ERR_UNSUPPORTED;
  if (tokens > kStaticMaxTokens) return MIXLORA_ERR_UNSUPPORTED;   // beyond the fixed scratch
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (tokens == 0) {
    if (cudaMemsetAsync(seg_off, 0, sizeof(int32_t) * (n_experts + 1), st) != cudaSuccess) return MIXLORA_ERR_CUDA;
    return MIXLORA_OK;
  }
  int* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return MIXLORA_ERR_CUDA;
  int* blk_counts = scratch;
  int* blk_off = scratch + kTableInts;
  const int nblk = (tokens + kStaticBlockTokens - 1) / kStaticBlockTokens;
  static_count_kernel<<<nblk, kStaticBlockTokens, 0, st>>>(expert_idx, blk_counts, tokens, n_experts, top_k);
  static_scan_kernel<<<1, 1024, 0, st>>>(blk_counts, blk_off, seg_off, nblk, n_experts);
  static_scatter_kernel<<<nblk, kStaticBlockTokens, 0, st>>>(expert_idx, blk_off, perm, tokens, n_experts, top_k);
  if (cudaGetLastError() != cudaSuccess) return MIXLORA_ERR_CUDA;
  return MIXLORA_OK;
}

extern "C" int32_t mixlora_dispatch_static_max_tokens(void) { return kStaticMaxTokens; }
