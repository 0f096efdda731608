// gs_spec_accept: temperature softmax statistics, sequential accept/reject, correction or bonus
// token by inverse CDF, and the estimator updates (Sec. II-A2; Eq. updatealpha, Eq. updateX).
//
// Two launches on one stream:
//   1. sa_row_stats   every logit row is cut into chunks of 8192 floats; one CTA per (chunk,row)
//                     streams its chunk once with 16-byte loads and writes (max, argmax, sum exp).
//                     (Not launched by gs_spec_accept_prestats: the LM head's epilogue wrote the
//                     statistics.)
//   2. the finish step.  Every CTA of a server first repeats the small "decide" step (a warp per row
//                     merges that row's chunk statistics, evaluates p(s_j), q(s_j), the ratio; one
//                     thread scans for the first rejection), which selects the one row the last token
//                     is drawn from (max(0, p - q) after a rejection, p for the bonus row).
//      sa_finish_cluster (default) one thread-block cluster per server, CTA k owning the k-th slice of
//                     the vocabulary: slice masses in shared memory, slice totals exchanged through
//                     distributed shared memory, the owner of u * total scans its own slice.
//      sa_finish      (V not a multiple of 4, or a slice too large for shared memory) one CTA per
//                     (chunk, server): chunk masses through the workspace; the last CTA of a server
//                     to finish (an atomic ticket, nobody waits) scans them, finds the chunk that
//                     holds u * total and does an ordered prefix scan inside it.
//                     CTA 0 of a server writes the outputs and the estimator update.
// Only one row per server is read a second time.  All cross-thread sums are fp64 in a fixed
// order, so two runs give identical bits.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace gs {

constexpr int kSaThreads = 256;
constexpr int kSaChunk = 8192;                   // floats per CTA
constexpr int kSaPerThread = kSaChunk / kSaThreads;  // 32
constexpr float kLog2e = 1.4426950408889634f;

struct SaWorkspace {
  ChunkStat* stats;   // [Tq * n_chunk]
  int* tickets;       // [N] CTAs of a server that have delivered their chunk mass
  double* mass;       // [N * n_chunk]
};

static size_t sa_layout(int N, int Tq, int V, SaWorkspace* w, char* base) {
  size_t n_chunk = (size_t)(V + kSaChunk - 1) / kSaChunk;
  size_t off = 0;
  size_t stats = off; off = align_up(off + sizeof(ChunkStat) * n_chunk * (size_t)Tq, 256);
  size_t sel = off;   off = align_up(off + sizeof(int) * (size_t)N, 256);
  size_t mass = off;  off = align_up(off + sizeof(double) * n_chunk * (size_t)N, 256);
  if (w != nullptr) {
    w->stats = reinterpret_cast<ChunkStat*>(base + stats);
    w->tickets = reinterpret_cast<int*>(base + sel);
    w->mass = reinterpret_cast<double*>(base + mass);
  }
  return off;
}

// Loads the 32 floats a thread owns in a chunk: element (k*256 + tid)*4 + j, k in 0..7, j in 0..3.
// Out-of-range elements read as `fill`.
template <bool VEC>
GS_DEVINL void load_chunk(const float* __restrict__ row, int base, int V, int tid, float (&v)[kSaPerThread],
                          float fill = -INFINITY) {
#pragma unroll
  for (int k = 0; k < kSaPerThread / 4; ++k) {
    int idx = base + (k * kSaThreads + tid) * 4;
    if (VEC && idx + 3 < V) {
      float4 t = __ldg(reinterpret_cast<const float4*>(row + idx));
      v[4 * k + 0] = t.x; v[4 * k + 1] = t.y; v[4 * k + 2] = t.z; v[4 * k + 3] = t.w;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[4 * k + j] = (idx + j < V) ? __ldg(row + idx + j) : fill;
    }
  }
}

GS_DEVINL int chunk_elem_index(int base, int tid, int e) {
  return base + ((e >> 2) * kSaThreads + tid) * 4 + (e & 3);
}

// Fixed-order block sum of one double per thread (256 threads): butterfly inside a warp,
// then warp 0..7 added in order by thread 0.  Result valid in thread 0.
GS_DEVINL double block_sum_f64(double v, double* smem8) {
  v = warp_sum_f64(v);
  int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (lane == 0) smem8[wid] = v;
  __syncthreads();
  double s = 0.0;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 0; w < kSaThreads / 32; ++w) s += smem8[w];
  }
  return s;
}

template <bool VEC>
__global__ void __launch_bounds__(kSaThreads)
sa_row_stats(const float* __restrict__ logits, int V, int n_chunk, float k2, ChunkStat* __restrict__ stats,
             int* __restrict__ tickets, int N) {
  __shared__ float s_m[kSaThreads / 32];
  __shared__ int s_a[kSaThreads / 32];
  __shared__ double s_z[kSaThreads / 32];
  __shared__ float s_bm;
  const int tid = threadIdx.x, c = blockIdx.x, r = blockIdx.y;
  // The successor is released only after this kernel's own wait: whatever it reads before ITS wait
  // was then complete before this kernel touched memory.
  pdl_wait();
  pdl_launch_dependents();
  if (c == 0 && r == 0)
    for (int i = tid; i < N; i += kSaThreads) tickets[i] = 0;     // for the next kernel
  const float* row = logits + (size_t)r * V;
  const int base = c * kSaChunk;
  float v[kSaPerThread];
  load_chunk<VEC>(row, base, V, tid, v);

  float m = -INFINITY;
  int a = INT_MAX;
#pragma unroll
  for (int e = 0; e < kSaPerThread; ++e) {
    if (v[e] > m) { m = v[e]; a = chunk_elem_index(base, tid, e); }
  }
  warp_argmax(m, a);
  if ((tid & 31) == 0) { s_m[tid >> 5] = m; s_a[tid >> 5] = a; }
  __syncthreads();
  if (tid == 0) {
    float bm = s_m[0]; int ba = s_a[0];
#pragma unroll
    for (int w = 1; w < kSaThreads / 32; ++w) argmax_merge(bm, ba, s_m[w], s_a[w]);
    s_bm = bm; s_a[0] = ba;
  }
  __syncthreads();
  const float bm = s_bm;
  float z = 0.f;
  if (k2 > 0.f && bm > -INFINITY) {
#pragma unroll
    for (int e = 0; e < kSaPerThread; ++e) z += fast_exp2((v[e] - bm) * k2);
  }
  double zs = block_sum_f64((double)z, s_z);
  if (tid == 0) {
    ChunkStat st;
    st.m = bm; st.arg = (s_a[0] == INT_MAX) ? base : s_a[0]; st.z = zs;
    stats[(size_t)r * n_chunk + c] = st;
  }
}

// 0 = automatic (a cluster per server where the shape allows it), 1 = the ticket kernel.
static int g_sa_finish_variant = 0;

struct SaFinishArgs {
  const float* logits; const float* q_probs; const int32_t* draft_tok; const int32_t* cu_q;
  const float* u_accept; const float* u_sample;
  int N, Tq, V, n_chunk, Gamma;
  float tau, k2;
  int32_t* accepted; int32_t* out_tok; int32_t* n_out;
  float* ratio; float* p_tok; float* margin;
  double* alpha_hat; double* X; double eta, beta, alpha_min, alpha_max;
  const ChunkStat* stats; int* tickets; double* mass;
  int32_t* d_status;
  int smem_bytes;
  int stats_from_predecessor;   // the statistics come from the kernel right before this one: read nothing of its output before the wait
  // Second home of the first draft rows of every server (same layout as q_probs): the row of the first
  // rejection is read from there when its position is below q_near_rows, from q_probs otherwise.  The
  // host-buffer round sets it when q_probs is host memory read over the bus and the first rows have been
  // copied to the device meanwhile; everywhere else q_near == q_probs.
  const float* q_near; int q_near_rows;
};
GS_DEVINL const float* sa_q_row(const SaFinishArgs& A, int g0, int a) {
  return ((a < A.q_near_rows) ? A.q_near : A.q_probs) + (size_t)(g0 + a) * A.V;
}

// Mass of element v of the selected row: max(0, p - q) or p, in fp64 from an fp32 exponential.
GS_DEVINL double elem_mass(float l, float M, float k2, double invZ, bool resid, float q) {
  double p = (double)fast_exp2((l - M) * k2) * invZ;
  if (resid) { p -= (double)q; p = p > 0.0 ? p : 0.0; }
  return p;
}

// Ordered scan of one chunk: thread t owns the 32 consecutive elements base + 32 t .. +31.
// Returns through s_tok the smallest index whose inclusive prefix (offset by `before`) exceeds
// thr, or INT_MAX; s_last = largest index with positive mass.
template <bool VEC>
GS_DEVINL void scan_chunk(const float* __restrict__ lrow, const float* __restrict__ qrow, int base, int V,
                          float M, float k2, double invZ, double before, double thr,
                          int* s_tok, int* s_last, double* s_lo, double* s_hi, double* s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int first = base + tid * kSaPerThread;
  double w[kSaPerThread];
  double run = 0.0;
  int last_pos = -1;
  // the thread's 32 consecutive elements: 16-byte loads when the row allows it
  float lv[kSaPerThread], qv[kSaPerThread];
  const bool vec_ok = VEC && first + kSaPerThread <= V;
  if (vec_ok) {
#pragma unroll
    for (int e = 0; e < kSaPerThread; e += 4) {
      const float4 t = __ldg(reinterpret_cast<const float4*>(lrow + first + e));
      lv[e] = t.x; lv[e + 1] = t.y; lv[e + 2] = t.z; lv[e + 3] = t.w;
    }
    if (qrow != nullptr) {
#pragma unroll
      for (int e = 0; e < kSaPerThread; e += 4) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(qrow + first + e));
        qv[e] = t.x; qv[e + 1] = t.y; qv[e + 2] = t.z; qv[e + 3] = t.w;
      }
    }
  } else {
#pragma unroll
    for (int e = 0; e < kSaPerThread; ++e) {
      const int idx = first + e;
      lv[e] = idx < V ? lrow[idx] : -INFINITY;
      qv[e] = (idx < V && qrow != nullptr) ? qrow[idx] : 0.f;
    }
  }
#pragma unroll
  for (int e = 0; e < kSaPerThread; ++e) {
    const int idx = first + e;
    double x = 0.0;
    if (idx < V) x = elem_mass(lv[e], M, k2, invZ, qrow != nullptr, qrow != nullptr ? qv[e] : 0.f);
    if (x > 0.0) last_pos = idx;
    run += x;
    w[e] = run;   // inclusive prefix inside the thread
  }
  // exclusive scan of the thread totals: inside warps by shuffles, across warps by thread order
  double incl = run;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    double t = shfl_up_f64(incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) s_warp[wid] = incl;
  __syncthreads();
  double woff = 0.0;
  for (int k = 0; k < wid; ++k) woff += s_warp[k];
  const double excl = before + woff + (incl - run);
  int found = INT_MAX;
  double lo = 0.0, hi = 0.0;
#pragma unroll
  for (int e = 0; e < kSaPerThread; ++e) {
    const int idx = first + e;
    if (found == INT_MAX && idx < V && excl + w[e] > thr) {
      found = idx;
      hi = excl + w[e];
      lo = excl + (e > 0 ? w[e - 1] : 0.0);
    }
  }
  if (found != INT_MAX) atomicMin(s_tok, found);
  if (last_pos >= 0) atomicMax(s_last, last_pos);
  __syncthreads();
  if (found != INT_MAX && *s_tok == found) { *s_lo = lo; *s_hi = hi; }
  __syncthreads();
}

// Pointers into the dynamic shared memory of a finish kernel: merged row statistics (rows
// j = 0..gamma) and the scalars of the draft positions (j = 0..gamma-1).
struct SaDecideSmem {
  float* sM; int* sArg; int* sRej; double* sZ; double* sRatio; float* sL; float* sQ; float* sU; int* sTok;
};
inline size_t sa_decide_bytes(size_t rows) { return align_up(3 * rows * 4, 8) + 2 * rows * 8 + 4 * rows * 4; }
GS_DEVINL SaDecideSmem sa_decide_carve(unsigned char* raw, int gamma) {
  SaDecideSmem S;
  S.sM = reinterpret_cast<float*>(raw);
  S.sArg = reinterpret_cast<int*>(S.sM + (gamma + 1));
  S.sRej = S.sArg + (gamma + 1);
  size_t off = (size_t)(3 * (gamma + 1)) * 4;
  off = (off + 7) / 8 * 8;
  S.sZ = reinterpret_cast<double*>(raw + off);
  S.sRatio = S.sZ + (gamma + 1);
  S.sL = reinterpret_cast<float*>(S.sRatio + (gamma + 1));
  S.sQ = S.sL + (gamma + 1);
  S.sU = S.sQ + (gamma + 1);
  S.sTok = reinterpret_cast<int*>(S.sU + (gamma + 1));
  return S;
}

// Offsets of server i that keep every access of the finish step inside its arrays: at least one row,
// at least one row left for each server before it (its per-draft offset r0 - i is then >= 0) and for
// each server after it (its last draft entry r1 - 2 - i then lies below Gamma = Tq - N, and its
// r1 - r0 rows fit the shared memory sized for Tq - N + 1).  Any other server is skipped and flagged.
GS_DEVINL bool sa_server_ok(int i, int r0, int r1, int N, int Tq) {
  return r0 >= i && r1 > r0 && r1 <= Tq - (N - 1 - i);
}

// First half of the "decide" step: the scalars of every draft position of server i (token, its
// logit and draft probability -- dependent loads -- and the uniform) go to shared memory.  Reads
// nothing the statistics pass writes.  The caller synchronises the CTA before sa_decide.
// part: 0 = everything, 1 = all but the logits, 2 = the logits only (for the tokens part 1 stored; the
// same thread handles the same j in both parts).
GS_DEVINL void sa_fetch_scalars(const SaFinishArgs& A, int i, int r0, int gamma, bool writer, const SaDecideSmem& S,
                                int part = 0) {
  const int g0 = r0 - i;
  for (int j = threadIdx.x; j < gamma; j += blockDim.x) {
    if (part == 2) {
      const int s = S.sTok[j];
      S.sL[j] = (s >= 0) ? A.logits[(size_t)(r0 + j) * A.V + s] : 0.f;
      continue;
    }
    const int s = A.draft_tok[g0 + j];
    const bool in = (s >= 0 && s < A.V);
    S.sTok[j] = in ? s : -1;
    if (part == 0) S.sL[j] = in ? A.logits[(size_t)(r0 + j) * A.V + s] : 0.f;
    S.sQ[j] = in ? A.q_probs[(size_t)(g0 + j) * A.V + s] : 0.f;
    S.sU[j] = A.u_accept[g0 + j];
    if (!in && writer) set_status(A.d_status, GS_ERR_INVALID_ARG);
  }
}

// Second half, run by a whole CTA after a barrier: a warp per row merges that row's chunk
// statistics (weights 2^((m_c - M) k2) from the special-function unit, sums in fp64), evaluates
// p(s_j), the ratio and the accept test; one thread scans for the first rejection.  `writer` CTAs
// also store ratio / p_tok / margin / accepted / n_out, and one of their threads does the estimator
// update off the other threads' path.  Returns a_i (uniform over the CTA).
GS_DEVINL int sa_decide(const SaFinishArgs& A, int i, int r0, int gamma, bool writer, const SaDecideSmem& S,
                        int* s_acc) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nthr = blockDim.x, nwarp = nthr >> 5;
  const int g0 = r0 - i;
  const double inv_tau = A.tau > 0.f ? 1.0 / (double)A.tau : 0.0;
  for (int j = wid; j <= gamma; j += nwarp) {
    const ChunkStat* st = A.stats + (size_t)(r0 + j) * A.n_chunk;
    float M = -INFINITY; int arg = INT_MAX;
    double z = 0.0;
    if (A.n_chunk <= 64) {
      // at most two chunks per lane: read them once
      ChunkStat c0s, c1s;
      c0s.m = -INFINITY; c0s.arg = INT_MAX; c0s.z = 0.0; c1s = c0s;
      if (lane < A.n_chunk) c0s = st[lane];
      if (lane + 32 < A.n_chunk) c1s = st[lane + 32];
      argmax_merge(M, arg, c0s.m, c0s.arg);
      argmax_merge(M, arg, c1s.m, c1s.arg);
      warp_argmax(M, arg);
      if (A.tau > 0.f) {
        if (c0s.m > -INFINITY) z += c0s.z * (double)fast_exp2((c0s.m - M) * A.k2);
        if (c1s.m > -INFINITY) z += c1s.z * (double)fast_exp2((c1s.m - M) * A.k2);
      }
    } else if (A.n_chunk <= 160) {
      // up to five per lane (the LM head writes one entry per CTA: 148 on this device): one round of loads
      ChunkStat c[5];
#pragma unroll
      for (int k = 0; k < 5; ++k) {
        c[k].m = -INFINITY; c[k].arg = INT_MAX; c[k].z = 0.0;
        if (lane + 32 * k < A.n_chunk) c[k] = st[lane + 32 * k];
      }
#pragma unroll
      for (int k = 0; k < 5; ++k) argmax_merge(M, arg, c[k].m, c[k].arg);
      warp_argmax(M, arg);
      if (A.tau > 0.f) {
#pragma unroll
        for (int k = 0; k < 5; ++k)
          if (c[k].m > -INFINITY) z += c[k].z * (double)fast_exp2((c[k].m - M) * A.k2);
      }
    } else {
      for (int cc = lane; cc < A.n_chunk; cc += 32) argmax_merge(M, arg, st[cc].m, st[cc].arg);
      warp_argmax(M, arg);
      if (A.tau > 0.f)
        for (int cc = lane; cc < A.n_chunk; cc += 32)
          if (st[cc].m > -INFINITY) z += st[cc].z * (double)fast_exp2((st[cc].m - M) * A.k2);
    }
    const double Z = warp_sum_f64(z);
    if (lane == 0) {
      S.sM[j] = M; S.sArg[j] = arg; S.sZ[j] = Z;
      if (j < gamma) {
        const int s = S.sTok[j];
        double p = 0.0, q = 0.0, rho = 0.0;
        if (s >= 0) {
          const float l = S.sL[j];
          if (A.tau > 0.f) p = (Z > 0.0) ? exp(((double)l - (double)M) * inv_tau) / Z : 0.0;
          else p = (s == arg) ? 1.0 : 0.0;
          q = (double)S.sQ[j];
          if (q > 0.0) rho = p / q;
          else rho = (p > 0.0) ? (double)INFINITY : 0.0;
        }
        const double u = (double)S.sU[j];
        S.sRej[j] = (u > rho) ? 1 : 0;
        const double clipped = rho < 1.0 ? rho : 1.0;
        S.sRatio[j] = clipped;
        if (writer) {
          A.ratio[g0 + j] = (float)clipped;
          A.p_tok[g0 + j] = (float)p;
          if (A.margin != nullptr) A.margin[g0 + j] = (float)(u - rho);
        }
      }
    }
  }
  __syncthreads();
  if (tid == 0) {
    int a = gamma;
    for (int j = 0; j < gamma; ++j) {
      if (S.sRej[j]) { a = j; break; }
    }
    *s_acc = a;
  }
  __syncthreads();
  const int a = *s_acc;
  // Estimator update (Eq. updatealpha, Eq. updateX): one thread of another warp, so that its
  // loads of the old state do not hold up the CTA.
  if (writer && tid == (nthr > 32 ? 32 : 0)) {
    A.accepted[i] = a;
    A.n_out[i] = a + 1;
    if (A.alpha_hat != nullptr && A.X != nullptr) {
      const double x_old = A.X[i];
      if (gamma > 0) {
        const double ah_old = A.alpha_hat[i];
        double sum = 0.0;
        for (int j = 0; j < gamma; ++j) sum += S.sRatio[j];
        const double obs = sum / (double)gamma;
        double ah = (1.0 - A.eta) * ah_old + A.eta * obs;
        ah = ah < A.alpha_min ? A.alpha_min : ah;
        ah = ah > A.alpha_max ? A.alpha_max : ah;
        A.alpha_hat[i] = ah;
      }
      A.X[i] = (1.0 - A.beta) * x_old + A.beta * (double)(a + 1);
    }
  }
  return a;
}

template <bool VEC>
__global__ void __launch_bounds__(kSaThreads) sa_finish(SaFinishArgs A) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ int s_acc, s_is_last, s_chunk, s_tok, s_last;
  __shared__ double s_before, s_thr, s_total, s_lo, s_hi;
  __shared__ double s_warp[kSaThreads / 32];
  pdl_wait();
  pdl_launch_dependents();
  const int c = blockIdx.x, i = blockIdx.y, tid = threadIdx.x;
  const bool writer = (c == 0);           // one CTA per server owns the outputs
  const int r0 = A.cu_q[i], r1 = A.cu_q[i + 1];
  const int gamma = r1 - r0 - 1;
  if (!sa_server_ok(i, r0, r1, A.N, A.Tq)) {
    if (writer && tid == 0) {
      set_status(A.d_status, GS_ERR_SHAPE);
      A.accepted[i] = 0; A.n_out[i] = 0;
    }
    return;
  }
  const int g0 = r0 - i;
  const SaDecideSmem S = sa_decide_carve(smem_raw, gamma);
  sa_fetch_scalars(A, i, r0, gamma, writer, S);
  __syncthreads();
  sa_decide(A, i, r0, gamma, writer, S, &s_acc);
  float* const sM = S.sM; int* const sArg = S.sArg; double* const sZ = S.sZ;
  const int a = s_acc;
  const int row = r0 + a;                                  // the row the last token is drawn from
  const bool resid = a < gamma;                            // correction (max(0,p-q)) or bonus (p)
  const float selM = sM[a];
  const int selArg = sArg[a];
  const double invZ = (sZ[a] > 0.0) ? 1.0 / sZ[a] : 0.0;
  if (writer)
    for (int j = tid; j <= gamma; j += kSaThreads)
      if (j != a) A.out_tok[r0 + j] = (j < a) ? A.draft_tok[g0 + j] : -1;
  if (A.k2 <= 0.f) {   // greedy target: the one-hot (and its residual) sits on the argmax
    if (writer && tid == 0) {
      A.out_tok[row] = selArg;
      if (A.margin != nullptr) A.margin[A.Gamma + i] = 1.0f;
    }
    return;
  }
  const float* lrow = A.logits + (size_t)row * A.V;
  const float* qrow = resid ? sa_q_row(A, g0, a) : nullptr;

  // ---- mass of this CTA's chunk of the selected row
  {
    const int base = c * kSaChunk;
    float l[kSaPerThread], q[kSaPerThread];
    load_chunk<VEC>(lrow, base, A.V, tid, l);
    if (resid) load_chunk<VEC>(qrow, base, A.V, tid, q, 0.f);
    double acc = 0.0;
#pragma unroll
    for (int e = 0; e < kSaPerThread; ++e) acc += elem_mass(l[e], selM, A.k2, invZ, resid, resid ? q[e] : 0.f);
    const double tot = block_sum_f64(acc, s_warp);
    if (tid == 0) {
      A.mass[(size_t)i * A.n_chunk + c] = tot;
      __threadfence();
      const int ticket = atomicAdd(&A.tickets[i], 1);
      s_is_last = (ticket == A.n_chunk - 1) ? 1 : 0;
    }
  }
  __syncthreads();
  if (!s_is_last) return;
  __threadfence();

  // ---- the server's last CTA draws the token
  const double u = (double)A.u_sample[i];
  double* sMass = reinterpret_cast<double*>(smem_raw);           // the decide arrays are dead now
  const bool mass_in_smem = (size_t)A.n_chunk * sizeof(double) <= (size_t)A.smem_bytes;
  if (mass_in_smem)
    for (int cc = tid; cc < A.n_chunk; cc += kSaThreads) sMass[cc] = __ldcg(A.mass + (size_t)i * A.n_chunk + cc);
  __syncthreads();
  if (tid == 0) {
    const double* gm = A.mass + (size_t)i * A.n_chunk;
    auto mass_at = [&](int cc) { return mass_in_smem ? sMass[cc] : __ldcg(gm + cc); };
    double total = 0.0;
    for (int cc = 0; cc < A.n_chunk; ++cc) total += mass_at(cc);
    const double thr = u * total;
    double run = 0.0, before = 0.0;
    int pick = -1, last_pos = -1;
    for (int cc = 0; cc < A.n_chunk; ++cc) {
      const double mc = mass_at(cc);
      if (mc > 0.0) last_pos = cc;
      if (run + mc > thr) { pick = cc; before = run; break; }
      run += mc;
    }
    if (pick < 0 && last_pos >= 0) {   // rounding left no chunk: last chunk that has mass
      pick = last_pos;
      before = 0.0;
      for (int cc = 0; cc < pick; ++cc) before += mass_at(cc);
    }
    s_chunk = pick; s_before = before; s_thr = thr; s_total = total;
    s_tok = INT_MAX; s_last = -1; s_lo = 0.0; s_hi = 0.0;
  }
  __syncthreads();
  if (s_chunk >= 0) {
    scan_chunk<VEC>(lrow, qrow, s_chunk * kSaChunk, A.V, selM, A.k2, invZ, s_before, s_thr,
               &s_tok, &s_last, &s_lo, &s_hi, s_warp);
  } else {
    // max(0, p - q) has no mass at all: draw from p itself, scanning the whole row in order.
    double before = 0.0;   // total of p is 1 by construction of invZ
    const double thr = u;
    if (tid == 0) { s_thr = thr; s_total = 1.0; }
    for (int cc = 0; cc < A.n_chunk; ++cc) {
      __syncthreads();
      if (tid == 0) s_before = before;
      __syncthreads();
      scan_chunk<VEC>(lrow, nullptr, cc * kSaChunk, A.V, selM, A.k2, invZ, s_before, thr,
                 &s_tok, &s_last, &s_lo, &s_hi, s_warp);
      if (s_tok != INT_MAX) break;
      double part = 0.0;
      for (int k = 0; k < kSaThreads / 32; ++k) part += s_warp[k];
      before += part;
    }
  }
  if (tid == 0) {
    int tok = s_tok;
    float marg = 0.f;
    if (tok == INT_MAX) {
      tok = s_last >= 0 ? s_last : selArg;
    } else if (s_total > 0.0) {
      const double x = s_thr - s_lo, y = s_hi - s_thr;
      marg = (float)((x < y ? x : y) / s_total);
    }
    A.out_tok[row] = tok;
    if (A.margin != nullptr) A.margin[A.Gamma + i] = marg;
  }
}


// ------------------------------------------------------------------------------------------------
// sa_finish_cluster: the finish step with one thread-block cluster per server.
//
// CTA k of the cluster owns the k-th slice of the vocabulary.  The draft tokens' scalars are fetched
// while the statistics pass is still running (programmatic dependent launch); after the (redundant,
// cheap) decide step every CTA brings its slice of the selected draft row into shared memory with
// bulk copies, reads the matching logits from global memory, and overwrites the slice with the
// masses max(p - q, 0) (or p for a bonus row).  The CTAs exchange their slice totals through
// distributed shared memory around one cluster barrier; the CTA whose slice holds u * total then
// finds the token in the masses it already has in shared memory: no ticket, no second trip to
// global memory.  Thread t sums one contiguous run of the slice (an odd number of elements, so the
// strided shared-memory reads do not collide).  One slice per CTA lets two clusters share an SM.
constexpr int kFcThreads = 512;
constexpr int kFcCluster = 8;
constexpr int kFcWarps = kFcThreads / 32;
constexpr uint32_t kFcPiece = 16384;               // bytes per bulk copy

inline int fc_slice(int V) { return ((V + kFcCluster - 1) / kFcCluster + 3) / 4 * 4; }

// LOADS = 16-byte loads of logits a thread keeps in flight: 4 lets two clusters share an SM (64
// registers a thread); 10 covers a whole slice of up to 20480 logits in one round trip to L2 and is
// used when the batch is small enough for every CTA to have an SM of its own.
template <int LOADS>
__global__ void __launch_bounds__(kFcThreads, LOADS > 4 ? 1 : 2) sa_finish_cluster(SaFinishArgs A, int slice) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_acc, s_abort, s_found, s_lastpos;
  __shared__ double s_warp[kFcWarps];
  __shared__ double s_cta_mass[2][kFcCluster];     // written by the peers (and by this CTA for itself)
  cluster_arrive_release();                        // phase 0: "my shared memory exists"; waited for before the first remote store
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int rank = (int)cluster_cta_rank(), i = blockIdx.y;
  const uint32_t bar = smem_u32(&s_bar);
  if (tid == 0) {
    mbar_init(bar, 1);
    s_abort = 0; s_found = INT_MAX; s_lastpos = -1;
    fence_barrier_init();
    fence_proxy_async();
  }
  // Before the wait: only data that was complete before the statistics pass started (that kernel
  // releases this one after its own wait): offsets, draft tokens, their logits and draft
  // probabilities, uniforms.  The statistics themselves are read after the wait.
  const bool writer = (rank == 0);
  const int r0 = A.cu_q[i], r1 = A.cu_q[i + 1];
  const int gamma = r1 - r0 - 1;
  bool live = sa_server_ok(i, r0, r1, A.N, A.Tq);            // uniform over the cluster
  float* sx = reinterpret_cast<float*>(smem_raw);            // the slice: first the draft row, then the masses in place
  const SaDecideSmem S = sa_decide_carve(smem_raw + (size_t)slice * 4, live ? gamma : 0);
  if (live) sa_fetch_scalars(A, i, r0, gamma, writer, S, A.stats_from_predecessor ? 1 : 0);
  const double u = (double)A.u_sample[i];
  pdl_wait();
  pdl_launch_dependents();
  if (live && A.stats_from_predecessor) sa_fetch_scalars(A, i, r0, gamma, writer, S, 2);   // the logits are the predecessor's output
  __syncthreads();
  if (!live && writer && tid == 0) {
    set_status(A.d_status, GS_ERR_SHAPE);
    A.accepted[i] = 0; A.n_out[i] = 0;
  }
  int a = 0, row = 0, selArg = 0;
  bool resid = false;
  float selM = 0.f;
  double invZ = 0.0;
  if (live) {
    const int g0 = r0 - i;
    a = sa_decide(A, i, r0, gamma, writer, S, &s_acc);
    row = r0 + a;                                            // the row the last token is drawn from
    resid = a < gamma;                                       // correction (max(0,p-q)) or bonus (p)
    selM = S.sM[a]; selArg = S.sArg[a];
    invZ = (S.sZ[a] > 0.0) ? 1.0 / S.sZ[a] : 0.0;
    if (writer)
      for (int j = tid; j <= gamma; j += kFcThreads)
        if (j != a) A.out_tok[r0 + j] = (j < a) ? A.draft_tok[g0 + j] : -1;
    if (A.k2 <= 0.f) {   // greedy target: the one-hot (and its residual) sits on the argmax
      if (writer && tid == 0) {
        A.out_tok[row] = selArg;
        if (A.margin != nullptr) A.margin[A.Gamma + i] = 1.0f;
      }
      live = false;
    }
  }
  if (!live) {           // the whole cluster takes this path together; close the open barrier phase
    cluster_wait_acquire();
    return;
  }
  const int g0 = r0 - i;
  const int start = rank * slice;
  const int len = max(0, min(slice, A.V - start));           // a multiple of 4 (V is)
  const float4* l4 = reinterpret_cast<const float4*>(A.logits + (size_t)row * A.V + start);
  // ---- this CTA's slice of the draft row -> shared memory (bulk copies, one barrier)
  if (resid && len > 0 && wid == 0) {
    const char* qsrc = reinterpret_cast<const char*>(sa_q_row(A, g0, a) + start);
    const uint32_t bytes = (uint32_t)len * 4u;
    if (lane == 0) mbar_arrive_expect_tx(bar, bytes);
    __syncwarp();
    for (uint32_t off = lane * kFcPiece; off < bytes; off += 32 * kFcPiece)
      bulk_load_1d(smem_u32(sx) + off, qsrc + off, min(kFcPiece, bytes - off), bar);
  }
  // ---- masses in place: x = max(p - q, 0) after a rejection, p for the bonus row.  Logits come
  // straight from global memory (the statistics pass has just read them), four 16-byte loads per
  // thread in flight.  Element masses are fp32 (the exponential is an fp32 approximation in either
  // kernel); every sum over them is fp64.
  const float invZf = (float)invZ, negMk = -selM * A.k2;
  bool q_here = !resid;
  auto fill_masses = [&](bool res) {
    const int n4 = len >> 2;
    for (int f0 = tid; f0 < n4; f0 += LOADS * kFcThreads) {
      float4 l[LOADS];
#pragma unroll
      for (int k = 0; k < LOADS; ++k) {
        const int f = f0 + k * kFcThreads;
        l[k] = (f < n4) ? __ldg(l4 + f) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < LOADS; ++k) {
        l[k].x = fast_exp2(fmaf(l[k].x, A.k2, negMk)) * invZf;
        l[k].y = fast_exp2(fmaf(l[k].y, A.k2, negMk)) * invZf;
        l[k].z = fast_exp2(fmaf(l[k].z, A.k2, negMk)) * invZf;
        l[k].w = fast_exp2(fmaf(l[k].w, A.k2, negMk)) * invZf;
      }
      if (!q_here) {       // first use of the draft row: its copies have landed
        if (!mbar_wait(bar, 0u, &s_abort)) set_status(A.d_status, GS_ERR_TIMEOUT);
        q_here = true;
      }
#pragma unroll
      for (int k = 0; k < LOADS; ++k) {
        const int f = f0 + k * kFcThreads;
        if (f < n4) {
          float4* dst = reinterpret_cast<float4*>(sx) + f;
          if (res) {
            const float4 q = *dst;
            l[k].x = fmaxf(l[k].x - q.x, 0.f); l[k].y = fmaxf(l[k].y - q.y, 0.f);
            l[k].z = fmaxf(l[k].z - q.z, 0.f); l[k].w = fmaxf(l[k].w - q.w, 0.f);
          }
          *dst = l[k];
        }
      }
    }
    if (!q_here) {         // threads without elements still have to see the copies complete
      if (!mbar_wait(bar, 0u, &s_abort)) set_status(A.d_status, GS_ERR_TIMEOUT);
      q_here = true;
    }
    __syncthreads();
  };
  if (len == 0) q_here = true;                               // nothing was requested for an empty slice
  const int E = ((len + kFcThreads - 1) / kFcThreads) | 1;   // elements per thread, odd
  const int e0 = min(len, tid * E), e1 = min(len, e0 + E);

  int tok = -1;
  float marg = 0.f;
  for (int pass = 0; pass < 2; ++pass) {
    fill_masses(resid);
    // ---- mass of the thread's run, then the CTA-wide prefix in thread order
    double tot = 0.0;
    int last_pos = -1;
    for (int e = e0; e < e1; ++e) {
      const float x = sx[e];
      if (x > 0.f) last_pos = e;
      tot += (double)x;
    }
    double incl = tot;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const double t = shfl_up_f64(incl, d);
      if (lane >= d) incl += t;
    }
    const double prev = shfl_up_f64(incl, 1);
    if (lane == 31) s_warp[wid] = incl;
    __syncthreads();
    double woff = 0.0;
    for (int k = 0; k < wid; ++k) woff += s_warp[k];
    const double excl = (lane == 0) ? woff : woff + prev;     // CTA prefix before this thread
    const double G = woff + incl;                             // and including it
    if (pass == 0) cluster_wait_acquire();                    // every peer's shared memory is there
    if (tid == kFcThreads - 1) {
#pragma unroll
      for (int k = 0; k < kFcCluster; ++k)
        st_cluster_f64(map_to_cta(smem_u32(&s_cta_mass[pass][rank]), (uint32_t)k), G);
    }
    cluster_arrive_release();
    cluster_wait_acquire();
    double total = 0.0;
#pragma unroll
    for (int k = 0; k < kFcCluster; ++k) total += s_cta_mass[pass][k];
    if (!(total > 0.0)) {
      if (resid) { resid = false; continue; }       // max(0, p - q) has no mass: draw from p itself
      if (writer && tid == 0) { tok = selArg; }     // no mass at all (cannot happen for finite logits)
      break;
    }
    const double thr = u * total;
    int owner = -1, last_rank = -1;
    double before = 0.0, run = 0.0;
#pragma unroll
    for (int k = 0; k < kFcCluster; ++k) {
      const double mk = s_cta_mass[pass][k];
      if (mk > 0.0) last_rank = k;
      if (owner < 0 && run + mk > thr) { owner = k; before = run; }
      run += mk;
    }
    if (owner >= 0) {
      if (rank == owner) {
        // first thread whose inclusive prefix exceeds the threshold, then first such element
        if (before + G > thr) atomicMin(&s_found, tid);
        __syncthreads();
        if (tid == s_found) {
          double r2 = 0.0, lo = before + excl, hi = lo;
          int pick = -1, pos = -1;
          for (int e = e0; e < e1; ++e) {
            const double x = (double)sx[e];
            if (x > 0.0) {
              pos = e;
              const double c = before + (excl + (r2 + x));
              if (c > thr) { pick = e; lo = before + (excl + r2); hi = c; break; }
              r2 += x;
            }
          }
          if (pick < 0) pick = pos;                 // rounding between the two prefix forms: last element with mass
          else { const double x = thr - lo, y = hi - thr; marg = (float)((x < y ? x : y) / total); }
          tok = (pick >= 0) ? start + pick : selArg;
        }
      }
    } else if (rank == last_rank) {                 // rounding left no slice: the last token that has mass
      if (last_pos >= 0) atomicMax(&s_lastpos, last_pos);
      __syncthreads();
      if (tid == 0) tok = (s_lastpos >= 0) ? start + s_lastpos : selArg;
    }
    break;
  }
  if (tok >= 0) {
    A.out_tok[row] = tok;
    if (A.margin != nullptr) A.margin[A.Gamma + i] = marg;
  }
}

}  // namespace gs

extern "C" gs_status gs_spec_accept_select(int variant) {
  if (variant < 0 || variant > 1) return GS_ERR_INVALID_ARG;
  gs::g_sa_finish_variant = variant;
  return GS_OK;
}

extern "C" size_t gs_spec_accept_workspace(int N, int Tq, int V) {
  if (N <= 0 || Tq <= 0 || V <= 0) return 256;
  return gs::sa_layout(N, Tq, V, nullptr, nullptr);
}

namespace gs {
static gs_status spec_accept_impl(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                  const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                  float temperature, int N, int Tq, int V,
                                  int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                  float* ratio, float* p_tok, float* margin,
                                  double* alpha_hat, double* X, double eta, double beta,
                                  double alpha_min, double alpha_max,
                                  void* ws, size_t ws_bytes, int32_t* d_status, void* stream,
                                  const ChunkStat* pre_stats, int pre_chunks, const float* q_near = nullptr,
                                  int q_near_rows = 0);
}

// The acceptance step of the host-buffer round: q_probs may be host memory that the device reads over
// the bus, with the first q_near_rows draft rows of every server also present at q_near (device memory,
// same layout).  stats == NULL runs the statistics pass.
gs_status gs::spec_accept_near(const float* logits, const float* q_probs, const float* q_near, int q_near_rows,
                               const int32_t* draft_tok, const int32_t* cu_q, const float* u_accept,
                               const float* u_sample, float temperature, int N, int Tq, int V, int32_t* accepted,
                               int32_t* out_tok, int32_t* n_out, float* ratio, float* p_tok, double* alpha_hat,
                               double* X, double eta, double beta, double alpha_min, double alpha_max,
                               const void* stats, int n_chunk, void* ws, size_t ws_bytes, int32_t* d_status,
                               void* stream) {
  return spec_accept_impl(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, temperature, N, Tq, V, accepted, out_tok,
                          n_out, ratio, p_tok, nullptr, alpha_hat, X, eta, beta, alpha_min, alpha_max, ws, ws_bytes, d_status,
                          stream, static_cast<const ChunkStat*>(stats), n_chunk, q_near, q_near_rows);
}


extern "C" gs_status gs_spec_accept(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                    const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                    float temperature, int N, int Tq, int V,
                                    int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                    float* ratio, float* p_tok, float* margin,
                                    double* alpha_hat, double* X, double eta, double beta,
                                    double alpha_min, double alpha_max,
                                    void* ws, size_t ws_bytes, int32_t* d_status, void* stream) {
  return gs::spec_accept_impl(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, temperature, N, Tq, V, accepted,
                              out_tok, n_out, ratio, p_tok, margin, alpha_hat, X, eta, beta, alpha_min, alpha_max,
                              ws, ws_bytes, d_status, stream, nullptr, 0);
}

/* The acceptance step on statistics that gs_lm_head_logits_stats wrote: no pass over the logits. */
extern "C" gs_status gs_spec_accept_prestats(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                             const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                             float temperature, int N, int Tq, int V,
                                             int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                             float* ratio, float* p_tok, float* margin,
                                             double* alpha_hat, double* X, double eta, double beta,
                                             double alpha_min, double alpha_max,
                                             const void* stats, int n_chunk,
                                             void* ws, size_t ws_bytes, int32_t* d_status, void* stream) {
  if (stats == nullptr || n_chunk <= 0) return GS_ERR_INVALID_ARG;
  return gs::spec_accept_impl(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, temperature, N, Tq, V, accepted,
                              out_tok, n_out, ratio, p_tok, margin, alpha_hat, X, eta, beta, alpha_min, alpha_max,
                              ws, ws_bytes, d_status, stream, static_cast<const gs::ChunkStat*>(stats), n_chunk);
}

static gs_status gs::spec_accept_impl(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                      const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                      float temperature, int N, int Tq, int V,
                                      int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                      float* ratio, float* p_tok, float* margin,
                                      double* alpha_hat, double* X, double eta, double beta,
                                      double alpha_min, double alpha_max,
                                      void* ws, size_t ws_bytes, int32_t* d_status, void* stream,
                                      const ChunkStat* pre_stats, int pre_chunks, const float* q_near,
                                      int q_near_rows) {
  using namespace gs;
  if (N < 0 || Tq < 0 || V < 0 || !(temperature >= 0.f)) return GS_ERR_INVALID_ARG;
  if (N == 0) return GS_OK;
  if (Tq < N) return GS_ERR_SHAPE;
  if (V == 0) return GS_ERR_SHAPE;
  const int Gamma = Tq - N;
  if (!logits || !cu_q || !u_sample || !accepted || !out_tok || !n_out) return GS_ERR_INVALID_ARG;
  if (Gamma > 0 && (!q_probs || !draft_tok || !u_accept || !ratio || !p_tok)) return GS_ERR_INVALID_ARG;
  if ((alpha_hat == nullptr) != (X == nullptr)) return GS_ERR_INVALID_ARG;
  if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GS_ERR_WORKSPACE;
  if (ws_bytes < gs_spec_accept_workspace(N, Tq, V)) return GS_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SaWorkspace w;
  sa_layout(N, Tq, V, &w, static_cast<char*>(ws));
  const int n_chunk = (V + kSaChunk - 1) / kSaChunk;
  const float k2 = temperature > 0.f ? kLog2e / temperature : 0.f;
  const bool vec = (V % 4 == 0) && (reinterpret_cast<uintptr_t>(logits) % 16 == 0) &&
                   (q_probs == nullptr || reinterpret_cast<uintptr_t>(q_probs) % 16 == 0) &&
                   (q_near == nullptr || reinterpret_cast<uintptr_t>(q_near) % 16 == 0);

  dim3 g1(n_chunk, Tq);
  if (pre_stats == nullptr &&
      launch_ex(vec ? sa_row_stats<true> : sa_row_stats<false>, g1, dim3(kSaThreads), 0, st, true, 1,
                logits, V, n_chunk, k2, w.stats, w.tickets, N) != cudaSuccess)
    return GS_ERR_CUDA;

  SaFinishArgs A;
  A.logits = logits; A.q_probs = q_probs; A.draft_tok = draft_tok; A.cu_q = cu_q; A.u_accept = u_accept;
  A.u_sample = u_sample;
  A.N = N; A.Tq = Tq; A.V = V; A.n_chunk = n_chunk; A.Gamma = Gamma; A.tau = temperature; A.k2 = k2;
  A.accepted = accepted; A.out_tok = out_tok; A.n_out = n_out;
  A.ratio = ratio; A.p_tok = p_tok; A.margin = margin;
  A.alpha_hat = alpha_hat; A.X = X; A.eta = eta; A.beta = beta; A.alpha_min = alpha_min; A.alpha_max = alpha_max;
  A.stats = w.stats; A.tickets = w.tickets; A.mass = w.mass; A.d_status = d_status;
  A.stats_from_predecessor = 0;
  A.q_near = (q_near != nullptr && q_near_rows > 0) ? q_near : q_probs;
  A.q_near_rows = (q_near != nullptr && q_near_rows > 0) ? q_near_rows : 0;
  if (pre_stats != nullptr) { A.stats = pre_stats; A.n_chunk = pre_chunks; A.stats_from_predecessor = 1; }
  // rows of one server are bounded by Tq - (N-1); size the dynamic shared memory for that
  const size_t max_rows = (size_t)(Tq - N + 1);
  const size_t smem = sa_decide_bytes(max_rows);
  // One cluster per server when the two row slices fit a CTA's shared memory next to the decide arrays.
  const int slice = fc_slice(V);
  const size_t smem_fc = (size_t)slice * 4 + smem;
  if (vec && g_sa_finish_variant != 1 && smem_fc <= 200 * 1024) {
    static PerDeviceOnce attr_set;
    const int slot = device_slot();
    if (attr_set.needed(slot)) {
      if (cudaFuncSetAttribute(sa_finish_cluster<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess ||
          cudaFuncSetAttribute(sa_finish_cluster<10>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
        return GS_ERR_CUDA;
      attr_set.mark(slot);
    }
    A.smem_bytes = (int)smem_fc;
    // every CTA on an SM of its own (with room to spare for the placement of whole clusters)?
    const bool roomy = (long long)N * kFcCluster * 3 <= (long long)sm_count() * 2 && slice <= 10 * kFcThreads * 4;
    if ((roomy ? launch_ex(sa_finish_cluster<10>, dim3(kFcCluster, N), dim3(kFcThreads), smem_fc, st, true, kFcCluster, A, slice)
               : launch_ex(sa_finish_cluster<4>, dim3(kFcCluster, N), dim3(kFcThreads), smem_fc, st, true, kFcCluster, A, slice)) !=
        cudaSuccess) {
      (void)cudaGetLastError();
      return GS_ERR_CUDA;
    }
    count_launches(pre_stats == nullptr ? 2 : 1);
    return launch_status();
  }
  if (pre_stats != nullptr) return GS_ERR_UNSUPPORTED;     // only the cluster kernel takes foreign statistics
  if (smem > 160 * 1024) return GS_ERR_UNSUPPORTED;
  A.smem_bytes = (int)smem;
  if (smem > 40 * 1024) {
    if (cudaFuncSetAttribute(sa_finish<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(sa_finish<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return GS_ERR_CUDA;
  }
  dim3 g2(k2 > 0.f ? n_chunk : 1, N);
  if (launch_ex(vec ? sa_finish<true> : sa_finish<false>, g2, dim3(kSaThreads), smem, st, true, 1, A) != cudaSuccess)
    return GS_ERR_CUDA;
  count_launches(2);
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// gs_spec_accept_static: the same acceptance pass for callers that cannot hand over a workspace.
//
// Some hosts of this library may not allocate device memory at the point where a round runs: a
// serving loop whose memory pool was sized and frozen at start-up, a plug-in that is only lent
// input and output buffers, code running where cudaMalloc would serialise or fail.  For them the
// scratch (chunk statistics, per-server selection, chunk masses) lives in the fixed array below,
// which every GPU that loads the library carries until the process exits.
namespace gs {

constexpr size_t kSaStaticBytes = 2u << 20;   // 2 MiB
static __device__ __align__(256) unsigned char g_sa_static_scratch[kSaStaticBytes];

// In host code the symbol above is only a handle; the device address has to be asked for, once
// per device, with that device current.
static void* sa_static_scratch_ptr(gs_status* err) {
  static void* cached[kMaxDevices] = {};
  const int dev = device_slot();
  if (dev < 0) { *err = GS_ERR_CUDA; return nullptr; }
  if (cached[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_sa_static_scratch) != cudaSuccess || p == nullptr) { *err = GS_ERR_CUDA; return nullptr; }
    cached[dev] = p;
  }
  return cached[dev];
}

}  // namespace gs

extern "C" size_t gs_spec_accept_static_capacity(void) { return gs::kSaStaticBytes; }

extern "C" gs_status gs_spec_accept_static(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                           const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                           float temperature, int N, int Tq, int V,
                                           int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                           float* ratio, float* p_tok, float* margin,
                                           double* alpha_hat, double* X, double eta, double beta,
                                           double alpha_min, double alpha_max,
                                           int32_t* d_status, void* stream) {
  if (N < 0 || Tq < 0 || V < 0) return GS_ERR_INVALID_ARG;
  if (N == 0) return GS_OK;
  if (gs_spec_accept_workspace(N, Tq, V) > gs::kSaStaticBytes) return GS_ERR_WORKSPACE;   // problem too large
  gs_status err = GS_OK;
  void* scratch = gs::sa_static_scratch_ptr(&err);
  if (scratch == nullptr) return err;
  return gs_spec_accept(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, temperature, N, Tq, V,
                        accepted, out_tok, n_out, ratio, p_tok, margin, alpha_hat, X, eta, beta,
                        alpha_min, alpha_max, scratch, gs::kSaStaticBytes, d_status, stream);
}
