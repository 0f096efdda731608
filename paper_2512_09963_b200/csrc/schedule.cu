// gs_schedule: GoodSpeed-sched (Eq. goodspeed_sched, Sec. III-C) solved by marginal allocation.
//
// One CTA.  Thread i owns server i and keeps its current marginal gain
// Delta_i = alpha_hat_i^(S_i+1) / X_i in a register (fp64, formed by repeated multiplication).
// Each of the C budget steps is a block-wide arg-max over (gain, lowest index); the winner
// multiplies its gain by alpha_hat_i and increments S_i.  For N <= 32 the arg-max is three
// warp-wide integer reductions on the bit pattern of the (non-negative) gain.
#include "common.cuh"

namespace gs {

// Non-negative doubles order like their bit patterns.  Ineligible servers use key 0 with flag.
GS_DEVINL unsigned long long gain_key(double g) {
  return (unsigned long long)__double_as_longlong(g);
}

__global__ void __launch_bounds__(1024)
schedule_kernel(const double* __restrict__ X, const double* __restrict__ alpha_hat, int N, int C,
                const int32_t* __restrict__ s_min, const int32_t* __restrict__ s_max,
                int32_t* __restrict__ S_out, int32_t* d_status) {
  __shared__ unsigned long long s_key[32];
  __shared__ int s_idx[32];
  __shared__ int s_sum[32];
  __shared__ int s_winner;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int nwarp = (blockDim.x + 31) >> 5;
  const bool live = tid < N;
  double a = 0.0, gain = 0.0;
  int S = 0, cap = 0;
  if (live) {
    a = alpha_hat[tid];
    S = s_min ? s_min[tid] : 0;
    cap = s_max ? s_max[tid] : C;
    if (S < 0) S = 0;
    gain = a / X[tid];
    for (int k = 0; k < S; ++k) gain = __dmul_rn(gain, a);
    if (!(gain >= 0.0)) gain = 0.0;   // negative or NaN inputs never win
  }
  // budget left after the floors
  int part = live ? S : 0;
  part = __reduce_add_sync(0xffffffffu, part);
  if (lane == 0) s_sum[wid] = part;
  __syncthreads();
  int used = 0;
  for (int w = 0; w < nwarp; ++w) used += s_sum[w];
  int budget = C - used;
  if (budget < 0) {
    if (tid == 0) set_status(d_status, GS_ERR_SHAPE);
    budget = 0;
  }
  for (int step = 0; step < budget; ++step) {
    const bool elig = live && S < cap;
    // key: eligible servers get (gain bits + 1) so that an eligible zero gain still beats "none"
    const unsigned long long key = elig ? gain_key(gain) + 1ull : 0ull;
    const unsigned hi = (unsigned)(key >> 32), lo = (unsigned)key;
    const unsigned mhi = __reduce_max_sync(0xffffffffu, hi);
    const unsigned mlo = __reduce_max_sync(0xffffffffu, hi == mhi ? lo : 0u);
    const unsigned who = __ballot_sync(0xffffffffu, hi == mhi && lo == mlo);
    const int wlane = __ffs(who) - 1;
    int winner;
    if (nwarp == 1) {
      winner = ((((unsigned long long)mhi << 32) | mlo) != 0ull) ? wlane : -1;
    } else {
      if (lane == 0) {
        s_key[wid] = ((unsigned long long)mhi << 32) | mlo;
        s_idx[wid] = wid * 32 + wlane;
      }
      __syncthreads();
      if (tid == 0) {
        unsigned long long bk = 0ull; int bi = -1;
        for (int w = 0; w < nwarp; ++w) {
          if (s_key[w] > bk) { bk = s_key[w]; bi = s_idx[w]; }   // strict: lowest warp wins ties
        }
        s_winner = bi;
      }
      __syncthreads();
      winner = s_winner;
    }
    if (winner < 0) break;          // every server is at its cap
    if (tid == winner) {
      S += 1;
      gain = __dmul_rn(gain, a);
    }
  }
  if (live) S_out[tid] = S;
}

}  // namespace gs

extern "C" gs_status gs_schedule(const double* X, const double* alpha_hat, int N, int C,
                                 const int32_t* s_min, const int32_t* s_max, int32_t* S_out,
                                 int32_t* d_status, void* stream) {
  if (N < 0 || C < 0) return GS_ERR_INVALID_ARG;
  if (N == 0) return GS_OK;
  if (!X || !alpha_hat || !S_out) return GS_ERR_INVALID_ARG;
  if (N > 1024) return GS_ERR_UNSUPPORTED;
  const int threads = (N + 31) / 32 * 32;
  gs::schedule_kernel<<<1, threads, 0, static_cast<cudaStream_t>(stream)>>>(
      X, alpha_hat, N, C, s_min, s_max, S_out, d_status);
  gs::count_launches(1);
  return gs::launch_status();
}
