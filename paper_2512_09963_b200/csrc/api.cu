#include "common.cuh"
#include "sm100_ptx.cuh"
#include <atomic>

namespace gs {
static std::atomic<unsigned long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
static std::atomic<int> g_dependent_launch{1};
bool dependent_launch_enabled() { return g_dependent_launch.load(std::memory_order_relaxed) != 0; }
}  // namespace gs

extern "C" gs_status gs_set_dependent_launch(int on) {
  gs::g_dependent_launch.store(on != 0 ? 1 : 0, std::memory_order_relaxed);
  return GS_OK;
}

extern "C" unsigned long long gs_launch_count(void) { return gs::g_launches.load(std::memory_order_relaxed); }

extern "C" const char* gs_status_str(gs_status s) {
  switch (s) {
    case GS_OK: return "ok";
    case GS_ERR_INVALID_ARG: return "invalid argument";
    case GS_ERR_SHAPE: return "inconsistent shape or offsets";
    case GS_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case GS_ERR_WORKSPACE: return "workspace missing or too small";
    case GS_ERR_CUDA: return "CUDA call failed";
    case GS_ERR_TIMEOUT: return "bounded device wait ran out";
  }
  return "unknown status";
}

extern "C" int gs_version(void) { return 100; }

// ------------------------------------------------------------------------------------------------
// gs_selftest_wait_timeout: shows that the bounded wait every kernel of this library uses gives up.
// One warp waits, with the library's own mbar_wait, for a barrier phase that nothing will ever
// complete; after limit_us the wait raises the CTA's abort flag and returns, and the kernel reports
// GS_ERR_TIMEOUT through the device status exactly as the production kernels do, then ends normally.
namespace gs {
__global__ void wait_probe_kernel(unsigned long long limit_ns, int32_t* d_status, unsigned long long* waited_ns) {
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&s_bar), 1);
    s_abort = 0;
    fence_barrier_init();
  }
  __syncthreads();
  const uint64_t t0 = global_timer_ns();
  const bool done = mbar_wait_warp(smem_u32(&s_bar), 0u, &s_abort, limit_ns);
  if (threadIdx.x == 0) {
    if (waited_ns != nullptr) *waited_ns = global_timer_ns() - t0;
    if (!done && s_abort) set_status(d_status, GS_ERR_TIMEOUT);
  }
}
}  // namespace gs

extern "C" gs_status gs_selftest_wait_timeout(unsigned int limit_us, int32_t* d_status, unsigned long long* d_waited_ns,
                                              void* stream) {
  if (limit_us == 0 || limit_us > 1000000u || d_status == nullptr) return GS_ERR_INVALID_ARG;
  gs::wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>((unsigned long long)limit_us * 1000ull, d_status,
                                                                         d_waited_ns);
  gs::count_launches(1);
  return gs::launch_status();
}
