// Plain attention kernel for any dtype/head size: one CTA per (query row, query head), one warp
// per key, lanes across the head dimension.  It is the fp32 path (small problems) and it serves
// bf16 shapes that the tensor-core kernel does not cover.
#pragma once
#include "common.cuh"

namespace gs {

template <typename T> GS_DEVINL float to_f32(T x);
template <> GS_DEVINL float to_f32<float>(float x) { return x; }
template <> GS_DEVINL float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> GS_DEVINL T from_f32(float x);
template <> GS_DEVINL float from_f32<float>(float x) { return x; }
template <> GS_DEVINL __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Largest i in [0, N) with cu[i] <= r.
GS_DEVINL int find_server(const int32_t* __restrict__ cu, int N, int r) {
  int lo = 0, hi = N;   // invariant: cu[lo] <= r, answer in [lo, hi)
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= r) lo = mid; else hi = mid;
  }
  return lo;
}

constexpr int kGenAttnThreads = 128;
constexpr int kGenAttnMaxPerLane = 8;   // hd <= 256

template <typename T>
__global__ void __launch_bounds__(kGenAttnThreads)
attn_generic_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V, T* __restrict__ O,
                    const int32_t* __restrict__ cu_q, const int32_t* __restrict__ cu_kv,
                    int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv, int hd, float scale,
                    int32_t* d_status) {
  extern __shared__ float smem[];   // [nwarp][hd + 2]
  const int h = blockIdx.x, r = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  constexpr int nwarp = kGenAttnThreads / 32;
  if (r >= cu_q[N]) return;
  const int i = find_server(cu_q, N, r);
  const int q0 = cu_q[i], n_new = cu_q[i + 1] - q0;
  const int k0 = cu_kv[i], Lkv = cu_kv[i + 1] - k0;
  // the same per-server checks as the tensor-core kernel, plus: this row must lie inside the server the
  // search returned (offsets that do not start at 0 or that decrease would otherwise hand it another
  // server's keys).  Such rows are flagged and left unwritten.
  if (n_new <= 0 || Lkv < n_new || Lkv > max_kv_len || k0 < 0 || k0 + Lkv > total_kv || q0 < 0 ||
      q0 + n_new > Tq || r < q0 || r >= q0 + n_new) {
    if (tid == 0) set_status(d_status, GS_ERR_SHAPE);
    return;
  }
  const int t = r - q0;
  const int visible = Lkv - n_new + t + 1;
  const int g = h / (Hq / Hkv);
  const int per_lane = (hd + 31) / 32;

  float q[kGenAttnMaxPerLane], acc[kGenAttnMaxPerLane];
#pragma unroll
  for (int e = 0; e < kGenAttnMaxPerLane; ++e) {
    const int c = lane + 32 * e;
    q[e] = (e < per_lane && c < hd) ? to_f32(Q[((size_t)r * Hq + h) * hd + c]) * scale : 0.f;
    acc[e] = 0.f;
  }
  float m = -INFINITY, l = 0.f;
  for (int k = wid; k < visible; k += nwarp) {
    const T* krow = K + ((size_t)(k0 + k) * Hkv + g) * hd;
    const T* vrow = V + ((size_t)(k0 + k) * Hkv + g) * hd;
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < kGenAttnMaxPerLane; ++e) {
      const int c = lane + 32 * e;
      if (e < per_lane && c < hd) s += q[e] * to_f32(krow[c]);
    }
    s = warp_sum_f32(s);
    const float m_new = fmaxf(m, s);
    const float corr = expf(m - m_new);   // exp(-inf) = 0 on the first key
    const float p = expf(s - m_new);
    l = l * corr + p;
#pragma unroll
    for (int e = 0; e < kGenAttnMaxPerLane; ++e) {
      const int c = lane + 32 * e;
      if (e < per_lane && c < hd) acc[e] = acc[e] * corr + p * to_f32(vrow[c]);
    }
    m = m_new;
  }
  float* mine = smem + wid * (hd + 2);
#pragma unroll
  for (int e = 0; e < kGenAttnMaxPerLane; ++e) {
    const int c = lane + 32 * e;
    if (e < per_lane && c < hd) mine[c] = acc[e];
  }
  if (lane == 0) { mine[hd] = m; mine[hd + 1] = l; }
  __syncthreads();
  float M = -INFINITY;
  for (int w = 0; w < nwarp; ++w) M = fmaxf(M, smem[w * (hd + 2) + hd]);
  float Lsum = 0.f;
  for (int w = 0; w < nwarp; ++w) {
    const float mw = smem[w * (hd + 2) + hd];
    if (mw > -INFINITY) Lsum += smem[w * (hd + 2) + hd + 1] * expf(mw - M);
  }
  for (int c = tid; c < hd; c += kGenAttnThreads) {
    float o = 0.f;
    for (int w = 0; w < nwarp; ++w) {
      const float mw = smem[w * (hd + 2) + hd];
      if (mw > -INFINITY) o += smem[w * (hd + 2) + c] * expf(mw - M);
    }
    O[((size_t)r * Hq + h) * hd + c] = from_f32<T>(o / Lsum);
  }
}

template <typename T>
inline gs_status launch_attn_generic(const void* Q, const void* K, const void* V, void* O,
                                     const int32_t* cu_q, const int32_t* cu_kv, int N, int Tq, int total_kv,
                                     int max_kv_len, int Hq, int Hkv, int hd, float scale,
                                     int32_t* d_status, cudaStream_t st) {
  dim3 grid(Hq, Tq);
  const size_t smem = (size_t)(kGenAttnThreads / 32) * (hd + 2) * sizeof(float);
  attn_generic_kernel<T><<<grid, kGenAttnThreads, smem, st>>>(
      static_cast<const T*>(Q), static_cast<const T*>(K), static_cast<const T*>(V), static_cast<T*>(O),
      cu_q, cu_kv, N, Tq, total_kv, max_kv_len, Hq, Hkv, hd, scale, d_status);
  count_launches(1);
  return launch_status();
}

}  // namespace gs
