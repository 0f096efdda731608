#include "common.cuh"
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
