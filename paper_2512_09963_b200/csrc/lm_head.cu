// gs_lm_head_logits: logits = H W (Sec. II-A1).  fp32 inputs use a plain FMA kernel.
#include "common.cuh"
#include "attn_generic.cuh"

namespace gs {

constexpr int kHeadRows = 16;      // rows of H per CTA
constexpr int kHeadCols = 256;     // one column per thread
constexpr int kHeadKc = 64;        // k-slice staged in shared memory

template <typename T>
__global__ void __launch_bounds__(kHeadCols)
lm_head_plain_kernel(const T* __restrict__ H, const T* __restrict__ W, float* __restrict__ logits,
                     int Trows, int d, int V) {
  __shared__ float sH[kHeadRows][kHeadKc];
  const int v = blockIdx.x * kHeadCols + threadIdx.x;
  const int t0 = blockIdx.y * kHeadRows;
  float acc[kHeadRows];
#pragma unroll
  for (int r = 0; r < kHeadRows; ++r) acc[r] = 0.f;
  for (int c0 = 0; c0 < d; c0 += kHeadKc) {
    __syncthreads();
    for (int e = threadIdx.x; e < kHeadRows * kHeadKc; e += kHeadCols) {
      const int r = e / kHeadKc, c = e % kHeadKc;
      sH[r][c] = (t0 + r < Trows && c0 + c < d) ? to_f32(H[(size_t)(t0 + r) * d + c0 + c]) : 0.f;
    }
    __syncthreads();
    if (v < V) {
      const int kc = min(kHeadKc, d - c0);
      for (int c = 0; c < kc; ++c) {
        const float w = to_f32(W[(size_t)(c0 + c) * V + v]);
#pragma unroll
        for (int r = 0; r < kHeadRows; ++r) acc[r] = fmaf(sH[r][c], w, acc[r]);
      }
    }
  }
  if (v < V) {
#pragma unroll
    for (int r = 0; r < kHeadRows; ++r)
      if (t0 + r < Trows) logits[(size_t)(t0 + r) * V + v] = acc[r];
  }
}

template <typename T>
inline gs_status launch_lm_head_plain(const void* H, const void* W, float* logits, int T_, int d, int V,
                                      cudaStream_t st) {
  dim3 grid((V + kHeadCols - 1) / kHeadCols, (T_ + kHeadRows - 1) / kHeadRows);
  lm_head_plain_kernel<T><<<grid, kHeadCols, 0, st>>>(static_cast<const T*>(H), static_cast<const T*>(W),
                                                     logits, T_, d, V);
  return launch_status();
}

}  // namespace gs

extern "C" size_t gs_lm_head_workspace(int T, int d, int V, gs_dtype dt) {
  (void)T; (void)d; (void)V; (void)dt;
  return 256;
}

extern "C" gs_status gs_lm_head_logits(const void* H, const void* W, float* logits, int T, int d, int V,
                                       gs_dtype dt, void* ws, size_t ws_bytes, int32_t* d_status,
                                       void* stream) {
  using namespace gs;
  (void)d_status;
  if (T < 0 || d < 0 || V < 0) return GS_ERR_INVALID_ARG;
  if (dt != GS_F32 && dt != GS_BF16) return GS_ERR_INVALID_ARG;
  if (T == 0 || V == 0) return GS_OK;
  if (!H || !W || !logits) return GS_ERR_INVALID_ARG;
  if (ws == nullptr || ws_bytes < gs_lm_head_workspace(T, d, V, dt)) return GS_ERR_WORKSPACE;
  if ((T + kHeadRows - 1) / kHeadRows > 65535) return GS_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dt == GS_F32) return launch_lm_head_plain<float>(H, W, logits, T, d, V, st);
  return launch_lm_head_plain<__nv_bfloat16>(H, W, logits, T, d, V, st);
}
