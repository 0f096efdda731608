// gs_schedule: GoodSpeed-sched (Eq. goodspeed_sched, Sec. III-C) solved by marginal allocation.
//
// The greedy gives the budget, one token at a time, to the largest marginal gain
// Delta_i(s) = alpha_hat_i^(s+1) / X_i (fp64, formed by repeated multiplication), lowest index on
// ties.  Because every server's gains are non-increasing, the tokens the greedy hands out are exactly
// the `budget` first entries of all (server, step) pairs ordered by (gain descending, server
// ascending, step ascending).  Two kernels produce that allocation:
//   * schedule_rank_kernel (N <= 32): warp i owns server i.  One lane writes the server's gain list
//     to shared memory (the same chain of fp64 multiplications as the greedy); then the warp finds,
//     by bisection over its own list, how many of its entries rank among the first `budget`: the rank
//     of an entry is its own step plus, per other server j (one lane each), the number of j's entries
//     that precede it (a bisection in j's list).  About log^2 steps instead of `budget` rounds.
//   * schedule_kernel: the greedy itself, one block-wide arg-max per token; any N <= 1024, and the
//     path taken when an alpha_hat lies outside [0, 1] (gains no longer non-increasing).
#include "common.cuh"
#include <new>

namespace gs {

// 0 = automatic (the rank kernel where it applies), 1 = always the greedy kernel.
static int g_schedule_variant = 0;

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
  pdl_wait();
  pdl_launch_dependents();
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


// Gains are compared through their bit patterns: non-negative doubles order like unsigned integers.
// cnt = number of entries of list[0..len) that precede key k: entries > k, or >= k when `ties_first`
// (the list is non-increasing, so they form a prefix).
GS_DEVINL int precede_count(const unsigned long long* list, int len, unsigned long long k, bool ties_first) {
  int lo = 0, hi = len;                       // first index whose entry does NOT precede k
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    const unsigned long long e = list[mid];
    const bool before = ties_first ? (e >= k) : (e > k);
    if (before) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(1024)
schedule_rank_kernel(const double* __restrict__ X, const double* __restrict__ alpha_hat, int N, int C,
                     const int32_t* __restrict__ s_min, const int32_t* __restrict__ s_max,
                     int32_t* __restrict__ S_out, int32_t* d_status) {
  extern __shared__ __align__(8) unsigned char sched_smem[];
  unsigned long long* table = reinterpret_cast<unsigned long long*>(sched_smem);      // [N][C]
  __shared__ int s_S0[32], s_len[32], s_bad;
  __shared__ double s_a[32], s_g0[32];
  const int tid = threadIdx.x, lane = tid & 31, i = tid >> 5;       // warp i = server i
  pdl_wait();
  pdl_launch_dependents();
  if (tid == 0) s_bad = 0;
  __syncthreads();
  if (tid < N) {
    const double a = alpha_hat[tid];
    int S = s_min ? s_min[tid] : 0;
    int cap = s_max ? s_max[tid] : C;
    if (S < 0) S = 0;
    double gain = a / X[tid];
    for (int k = 0; k < S; ++k) gain = __dmul_rn(gain, a);
    if (!(gain >= 0.0)) gain = 0.0;           // negative or NaN inputs never win
    if (!(a >= 0.0 && a <= 1.0)) s_bad = 1;   // the ordering argument needs non-increasing gains
    s_a[tid] = a; s_g0[tid] = gain; s_S0[tid] = S;
    s_len[tid] = max(0, min(cap - S, C));
  }
  __syncthreads();
  int used = 0;
  for (int j = 0; j < N; ++j) used += s_S0[j];
  int budget = C - used;
  if (budget < 0) {
    if (tid == 0) set_status(d_status, GS_ERR_SHAPE);
    budget = 0;
  }
  if (s_bad) {
    // plain greedy by warp 0 (lane = server)
    if (i == 0) {
      const bool live = lane < N;
      double a = live ? s_a[lane] : 0.0, gain = live ? s_g0[lane] : 0.0;
      int S = live ? s_S0[lane] : 0;
      const int cap = live ? S + s_len[lane] : 0;
      for (int step = 0; step < budget; ++step) {
        const bool elig = live && S < cap;
        const unsigned long long key = elig ? (unsigned long long)__double_as_longlong(gain) + 1ull : 0ull;
        const unsigned hi = (unsigned)(key >> 32), lo = (unsigned)key;
        const unsigned mhi = __reduce_max_sync(0xffffffffu, hi);
        const unsigned mlo = __reduce_max_sync(0xffffffffu, hi == mhi ? lo : 0u);
        if ((((unsigned long long)mhi << 32) | mlo) == 0ull) break;
        const int winner = __ffs(__ballot_sync(0xffffffffu, hi == mhi && lo == mlo)) - 1;
        if (lane == winner) { S += 1; gain = __dmul_rn(gain, a); }
      }
      if (live) S_out[lane] = S;
    }
    return;
  }
  const int len_i = (i < N) ? min(s_len[i], budget) : 0;
  if (i < N && lane == 0) {
    const double a = s_a[i];
    double g = s_g0[i];
    unsigned long long* mine = table + (size_t)i * C;
    for (int t = 0; t < len_i; ++t) {
      mine[t] = (unsigned long long)__double_as_longlong(g);
      g = __dmul_rn(g, a);
    }
  }
  __syncthreads();
  if (i >= N) return;
  // Largest c in [0, len_i] with c == 0 or rank(i, c-1) < budget; ranks grow with the step.
  const unsigned long long* mine = table + (size_t)i * C;
  const int len_j = (lane < N && lane != i) ? min(s_len[lane], budget) : 0;
  const unsigned long long* theirs = table + (size_t)min(lane, N - 1) * C;
  int lo = 0, hi = len_i;                     // invariant: entries < lo are in, entries >= hi are out
  while (lo < hi) {
    const int t = (lo + hi) >> 1;
    const unsigned long long k = mine[t];
    const int cnt = len_j > 0 ? precede_count(theirs, len_j, k, lane < i) : 0;
    const int rank = t + __reduce_add_sync(0xffffffffu, cnt);
    if (rank < budget) lo = t + 1; else hi = t;
  }
  if (lane == 0) S_out[i] = s_S0[i] + lo;
}

}  // namespace gs

extern "C" gs_status gs_schedule_select(int variant) {
  if (variant < 0 || variant > 1) return GS_ERR_INVALID_ARG;
  gs::g_schedule_variant = variant;
  return GS_OK;
}

extern "C" gs_status gs_schedule(const double* X, const double* alpha_hat, int N, int C,
                                 const int32_t* s_min, const int32_t* s_max, int32_t* S_out,
                                 int32_t* d_status, void* stream) {
  if (N < 0 || C < 0) return GS_ERR_INVALID_ARG;
  if (N == 0) return GS_OK;
  if (!X || !alpha_hat || !S_out) return GS_ERR_INVALID_ARG;
  if (N > 1024) return GS_ERR_UNSUPPORTED;
  const size_t table = (size_t)N * (size_t)(C > 0 ? C : 1) * 8;
  if (N <= 32 && table <= 160 * 1024 && gs::g_schedule_variant != 1) {
    static gs::PerDeviceOnce attr_set;
    const int slot = gs::device_slot();
    if (attr_set.needed(slot)) {
      if (cudaFuncSetAttribute(gs::schedule_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024) !=
          cudaSuccess)
        return GS_ERR_CUDA;
      attr_set.mark(slot);
    }
    if (gs::launch_ex(gs::schedule_rank_kernel, dim3(1), dim3(32 * N), table, static_cast<cudaStream_t>(stream), true, 1,
                      X, alpha_hat, N, C, s_min, s_max, S_out, d_status) != cudaSuccess) {
      (void)cudaGetLastError();
      return GS_ERR_CUDA;
    }
    gs::count_launches(1);
    return GS_OK;
  }
  const int threads = (N + 31) / 32 * 32;
  if (gs::launch_ex(gs::schedule_kernel, dim3(1), dim3(threads), 0, static_cast<cudaStream_t>(stream), true, 1,
                    X, alpha_hat, N, C, s_min, s_max, S_out, d_status) != cudaSuccess) {
    (void)cudaGetLastError();
    return GS_ERR_CUDA;
  }
  gs::count_launches(1);
  return GS_OK;
}


// The same allocation for estimator state that lives in host memory (a scheduler that runs beside
// the GPU, or ranks that have just exchanged their estimates): plain C++, no CUDA call.  The gains
// follow the device kernels bit for bit: alpha_hat / X, then one fp64 multiplication per step
// (nothing here can contract into a fused multiply-add), negative or NaN gains count as zero, the
// lowest index wins ties, an eligible zero gain still beats "no server left".
extern "C" gs_status gs_schedule_host(const double* X, const double* alpha_hat, int N, int C,
                                      const int32_t* s_min, const int32_t* s_max, int32_t* S_out) {
  if (N < 0 || C < 0) return GS_ERR_INVALID_ARG;
  if (N == 0) return GS_OK;
  if (!X || !alpha_hat || !S_out) return GS_ERR_INVALID_ARG;
  if (N > (1 << 20)) return GS_ERR_UNSUPPORTED;
  double* gain = new (std::nothrow) double[N];
  int32_t* cap = new (std::nothrow) int32_t[N];
  if (gain == nullptr || cap == nullptr) { delete[] gain; delete[] cap; return GS_ERR_INVALID_ARG; }
  long long used = 0;
  for (int i = 0; i < N; ++i) {
    const double a = alpha_hat[i];
    int S = s_min ? s_min[i] : 0;
    if (S < 0) S = 0;
    cap[i] = s_max ? s_max[i] : C;
    double g = a / X[i];
    for (int k = 0; k < S; ++k) g = g * a;
    gain[i] = (g >= 0.0) ? g : 0.0;
    S_out[i] = S;
    used += S;
  }
  gs_status rc = GS_OK;
  long long budget = (long long)C - used;
  if (budget < 0) { rc = GS_ERR_SHAPE; budget = 0; }      // floors above the budget: returned as they are
  for (long long step = 0; step < budget; ++step) {
    int best = -1;
    for (int i = 0; i < N; ++i)
      if (S_out[i] < cap[i] && (best < 0 || gain[i] > gain[best])) best = i;
    if (best < 0) break;                                    // every server is at its cap
    S_out[best] += 1;
    gain[best] = gain[best] * alpha_hat[best];
  }
  delete[] gain;
  delete[] cap;
  return rc;
}
