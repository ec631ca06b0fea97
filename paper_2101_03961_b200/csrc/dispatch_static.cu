// switch_moe_dispatch_plan_static: the dispatch plan (expert counts, token-order slot positions, capacity cut) for
// callers that must not allocate device memory and have no workspace to lend.
//
// Who that is: a process that handed the whole device heap to another allocator at start-up (an inference server's
// arena, a framework's caching pool) and cannot get a scratch buffer out of it from this call site; or a caller on
// a latency-critical path where cudaMalloc is unacceptable because it synchronises the device.  For them the scratch
// the plan needs between its three kernels -- the per-block expert histograms and their column scan -- lives in a
// file-scope __device__ array that every GPU loading this library holds until the process exits (512 KiB).
//
// The array's name in host code is only a host-side stand-in for the device symbol: its device address is obtained
// once per device with cudaGetSymbolAddress and that pointer is what the kernels receive.
#include <mutex>

#include "switch_common.cuh"

namespace swmoe {
namespace {

constexpr int kStaticMaxTokens = SWITCH_MOE_STATIC_PLAN_MAX_TOKENS;
constexpr int kStaticMaxBlocks = kStaticMaxTokens / kPlanBlockTokens;          // 256 histogram rows
constexpr size_t kStaticWords = 2ull * kStaticMaxBlocks * kMaxExperts;         // hist + scanned hist: 131072 ints

static __device__ __align__(256) int32_t g_plan_scratch[kStaticWords];

constexpr int kMaxDevices = 64;
int32_t* g_scratch_ptr[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

// hist[b][e] = tokens of block b routed to expert e (every word of the rows in use is written: nothing is assumed
// about what an earlier call left in the array)
__global__ void __launch_bounds__(kPlanBlockTokens)
static_plan_hist_kernel(const int* __restrict__ expert_index, int T, int E, int* __restrict__ hist) {
  __shared__ int h[kMaxExperts];
  for (int e = threadIdx.x; e < E; e += blockDim.x) h[e] = 0;
  __syncthreads();
  const int t = blockIdx.x * kPlanBlockTokens + threadIdx.x;
  const int e = t < T ? expert_index[t] : -1;
  if ((unsigned)e < (unsigned)E) atomicAdd(&h[e], 1);        // negative or out-of-range index: no vote
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) hist[(size_t)blockIdx.x * E + e] = h[e];
}

__global__ void __launch_bounds__(kMaxExperts)
static_plan_scan_kernel(const int* __restrict__ hist, int blocks, int E, int C, int* __restrict__ hist_base,
                        int* __restrict__ count, int* __restrict__ kept) {
  const int e = threadIdx.x;
  if (e >= E) return;
  int run = 0;
  for (int b = 0; b < blocks; ++b) {
    hist_base[(size_t)b * E + e] = run;
    run += hist[(size_t)b * E + e];
  }
  count[e] = run;
  kept[e] = min(run, C);
}

__global__ void __launch_bounds__(kPlanBlockTokens)
static_plan_assign_kernel(const int* __restrict__ expert_index, const int* __restrict__ hist_base,
                          const int* __restrict__ kept, int T, int E, int C, int* __restrict__ slot,
                          int* __restrict__ token_of_slot) {
  constexpr int kWarps = kPlanBlockTokens / 32;
  __shared__ int warp_cnt[kWarps][kMaxExperts];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < kWarps * kMaxExperts; i += blockDim.x) (&warp_cnt[0][0])[i] = 0;
  __syncthreads();
  const int t = blockIdx.x * kPlanBlockTokens + tid;
  int e = t < T ? expert_index[t] : -1;
  if ((unsigned)e >= (unsigned)E) e = -1;                     // "no expert" (-1, as the library's own marker) takes no slot
  const unsigned same = __match_any_sync(0xffffffffu, e >= 0 ? e : -1 - lane);   // distinct dummies for those lanes
  const int rank = __popc(same & ((1u << lane) - 1u));
  if (e >= 0 && rank == 0) warp_cnt[warp][e] = __popc(same);
  __syncthreads();
  if (t < T && e < 0) slot[t] = -1;
  if (e >= 0) {
    int pos = hist_base[(size_t)blockIdx.x * E + e] + rank;
    for (int w = 0; w < warp; ++w) pos += warp_cnt[w][e];
    const int s = pos < C ? e * C + pos : -1;
    slot[t] = s;
    if (s >= 0) token_of_slot[s] = t;
  }
  const int total = E * C;
  for (int s = blockIdx.x * blockDim.x + tid; s < total; s += gridDim.x * blockDim.x) {
    const int ex = s / C, pos = s - ex * C;
    if (pos >= kept[ex]) token_of_slot[s] = -1;
  }
}

// Device address of the static scratch on the current device, resolved on first use.
int scratch_for_current_device(int32_t** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SWITCH_MOE_CUDA_ERROR;
  if (dev < 0 || dev >= kMaxDevices) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    int32_t* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_plan_scratch) != cudaSuccess || ptr == nullptr)
      return SWITCH_MOE_CUDA_ERROR;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return SWITCH_MOE_OK;
}

}  // namespace
}  // namespace swmoe

extern "C" int switch_moe_dispatch_plan_static(const switch_moe_config* cfg, const int32_t* expert_index,
                                               int32_t* count, int32_t* kept, int32_t* slot, int32_t* token_of_slot,
                                               void* stream) {
  using namespace swmoe;
  Shape s;
  int rc = resolve_shape(cfg, &s);
  if (rc != SWITCH_MOE_OK) return rc;
  if (!expert_index || !count || !kept || !slot || !token_of_slot) return SWITCH_MOE_INVALID_ARGUMENT;
  // This entry point is the top-1 plan of one routing group only: the variants that place more than T assignments
  // or run a second stage need the workspace-based call.
  if (s.G != 1 || (cfg->flags & (SWITCH_MOE_FLAG_TOP2 | SWITCH_MOE_FLAG_REROUTE)) != 0)
    return SWITCH_MOE_UNSUPPORTED_SHAPE;
  const int blocks = (s.T + kPlanBlockTokens - 1) / kPlanBlockTokens;
  if (s.T > kStaticMaxTokens || blocks > kStaticMaxBlocks)   // the static scratch holds 256 x 256 counters twice
    return SWITCH_MOE_UNSUPPORTED_SHAPE;
  int32_t* scratch = nullptr;
  rc = scratch_for_current_device(&scratch);
  if (rc != SWITCH_MOE_OK) return rc;
  int32_t* hist = scratch;
  int32_t* hist_base = scratch + (size_t)kStaticMaxBlocks * kMaxExperts;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static_plan_hist_kernel<<<blocks, kPlanBlockTokens, 0, st>>>(expert_index, s.T, s.E, hist);
  static_plan_scan_kernel<<<1, kMaxExperts, 0, st>>>(hist, blocks, s.E, s.C, hist_base, count, kept);
  static_plan_assign_kernel<<<blocks, kPlanBlockTokens, 0, st>>>(expert_index, hist_base, kept, s.T, s.E, s.C,
                                                                        slot, token_of_slot);
  return launch_status();
}
