// Shared device/host helpers of the GoodSpeed CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <float.h>
#include <limits.h>

#include "../../include/goodspeed.h"

#define GS_DEVINL __device__ __forceinline__

namespace gs {

constexpr int kNumSMsFallback = 148;

// Softmax statistics of one row over one stretch of the vocabulary: maximum, its lowest index, and
// the sum of 2^((l - m) * log2(e)/tau).  Written by the statistics pass of gs_spec_accept or by the
// LM-head epilogue, merged by the acceptance pass.
struct ChunkStat {   // 16 bytes
  float m;
  int arg;
  double z;
};

// Sticky device status: the first non-zero code wins.
GS_DEVINL void set_status(int32_t* st, int code) {
  if (st != nullptr) atomicCAS(st, 0, code);
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Number of kernels this library has launched (host-side count, all threads).
void count_launches(int n);

inline gs_status launch_status() {
  return cudaGetLastError() == cudaSuccess ? GS_OK : GS_ERR_CUDA;
}

// Programmatic dependent launch.  A kernel launched with the attribute may start while its
// predecessor on the stream is still running; it must execute pdl_wait() before its first access
// to global memory (the wait returns once the predecessor grid has finished and its writes are
// visible).  pdl_launch_dependents() tells the scheduler that the successor may be started.
// Both are no-ops in a kernel launched without the attribute.
GS_DEVINL void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
GS_DEVINL void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Whether launches carry the programmatic-dependent-launch attribute (process-wide switch).
bool dependent_launch_enabled();

// Kernel launch with optional attributes: programmatic dependent launch and a cluster width.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_ex(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             bool dependent, int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (dependent && dependent_launch_enabled()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr; cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Per-device host state (function attributes set, SM counts, addresses of __device__ arrays) is kept
// in tables indexed by the CUDA device that is current when the entry point is called.
constexpr int kMaxDevices = 64;
inline int device_slot() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

// True once per device: the caller then sets its kernels' attributes (cudaFuncSetAttribute applies to
// the current device only) and calls mark() when that succeeded.
struct PerDeviceOnce {
  bool done[kMaxDevices] = {};
  bool needed(int slot) const { return slot < 0 || !done[slot]; }
  void mark(int slot) { if (slot >= 0) done[slot] = true; }
};

inline int sm_count() {
  static int cached[kMaxDevices] = {};
  const int slot = device_slot();
  if (slot >= 0 && cached[slot] > 0) return cached[slot];
  int n = 0;
  if (slot < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, slot) != cudaSuccess || n <= 0)
    return kNumSMsFallback;
  cached[slot] = n;
  return n;
}

// 2^x by the special-function unit (relative error about 2 ulp); 2^-inf = 0.
GS_DEVINL float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

GS_DEVINL double shfl_xor_f64(double v, int mask) {
  int lo = __double2loint(v), hi = __double2hiint(v);
  lo = __shfl_xor_sync(0xffffffffu, lo, mask);
  hi = __shfl_xor_sync(0xffffffffu, hi, mask);
  return __hiloint2double(hi, lo);
}

GS_DEVINL double shfl_up_f64(double v, int delta) {
  int lo = __double2loint(v), hi = __double2hiint(v);
  lo = __shfl_up_sync(0xffffffffu, lo, delta);
  hi = __shfl_up_sync(0xffffffffu, hi, delta);
  return __hiloint2double(hi, lo);
}

// Butterfly sum: every lane ends with the same value, order fixed by the lane ids.
GS_DEVINL double warp_sum_f64(double v) {
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) v += shfl_xor_f64(v, m);
  return v;
}

GS_DEVINL float warp_sum_f32(float v) {
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
  return v;
}

GS_DEVINL float warp_max_f32(float v) {
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
  return v;
}

// (value, index) maximum with the lowest index winning ties.
GS_DEVINL void argmax_merge(float& m, int& a, float m2, int a2) {
  if (m2 > m || (m2 == m && a2 < a)) { m = m2; a = a2; }
}

GS_DEVINL void warp_argmax(float& m, int& a) {
#pragma unroll
  for (int k = 16; k > 0; k >>= 1) {
    float m2 = __shfl_xor_sync(0xffffffffu, m, k);
    int a2 = __shfl_xor_sync(0xffffffffu, a, k);
    argmax_merge(m, a, m2, a2);
  }
}

// The acceptance step as the host-buffer round calls it (spec_accept.cu): like gs_spec_accept /
// gs_spec_accept_prestats (stats != NULL), but the row of a server's first rejection is read from q_near
// when its position is below q_near_rows and from q_probs otherwise.
gs_status spec_accept_near(const float* logits, const float* q_probs, const float* q_near, int q_near_rows,
                           const int32_t* draft_tok, const int32_t* cu_q, const float* u_accept, const float* u_sample,
                           float temperature, int N, int Tq, int V, int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                           float* ratio, float* p_tok, double* alpha_hat, double* X, double eta, double beta,
                           double alpha_min, double alpha_max, const void* stats, int n_chunk, void* ws,
                           size_t ws_bytes, int32_t* d_status, void* stream);

}  // namespace gs
