// gs_spec_accept: temperature softmax statistics, sequential accept/reject, correction or bonus
// token by inverse CDF, and the estimator updates (Sec. II-A2; Eq. updatealpha, Eq. updateX).
//
// Two launches on one stream:
//   1. sa_row_stats   every logit row is cut into chunks of 8192 floats; one CTA per (chunk,row)
//                     streams its chunk once with 16-byte loads and writes (max, argmax, sum exp).
//   2. sa_finish      one CTA per (chunk, server).  Every CTA of a server first repeats the small
//                     "decide" step (a warp per row merges that row's chunk statistics, evaluates
//                     p(s_j), q(s_j), the ratio; one thread scans for the first rejection), which
//                     selects the one row the last token is drawn from; the CTA then sums the mass
//                     of its chunk of that row (max(0, p - q) after a rejection, p for the bonus
//                     row).  The last CTA of a server to finish (an atomic ticket, nobody waits)
//                     scans the chunk masses in order, finds the chunk that holds u * total and
//                     does an ordered prefix scan inside it.  CTA (0, server) writes the outputs
//                     and the estimator update.
// Only one row per server is read a second time.  All cross-thread sums are fp64 in a fixed
// order, so two runs give identical bits.
#include "common.cuh"

namespace gs {

constexpr int kSaThreads = 256;
constexpr int kSaChunk = 8192;                   // floats per CTA
constexpr int kSaPerThread = kSaChunk / kSaThreads;  // 32
constexpr float kLog2e = 1.4426950408889634f;

struct ChunkStat {   // 16 bytes
  float m;
  int arg;
  double z;
};

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
};

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

template <bool VEC>
__global__ void __launch_bounds__(kSaThreads) sa_finish(SaFinishArgs A) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ int s_acc, s_is_last, s_chunk, s_tok, s_last;
  __shared__ double s_before, s_thr, s_total, s_lo, s_hi;
  __shared__ double s_warp[kSaThreads / 32];
  const int c = blockIdx.x, i = blockIdx.y, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const bool writer = (c == 0);           // one CTA per server owns the outputs
  const int r0 = A.cu_q[i], r1 = A.cu_q[i + 1];
  const int gamma = r1 - r0 - 1;
  if (r0 < 0 || gamma < 0 || r1 > A.Tq) {
    if (writer && tid == 0) {
      set_status(A.d_status, GS_ERR_SHAPE);
      A.accepted[i] = 0; A.n_out[i] = 0;
    }
    return;
  }
  const int g0 = r0 - i;
  // per-row merged statistics, rows j = 0..gamma
  float* sM = reinterpret_cast<float*>(smem_raw);                // [gamma+1]
  int* sArg = reinterpret_cast<int*>(sM + (gamma + 1));          // [gamma+1]
  int* sRej = sArg + (gamma + 1);                                // [gamma+1] 1 = would be rejected
  size_t off = (size_t)(3 * (gamma + 1)) * 4;
  off = (off + 7) / 8 * 8;
  double* sZ = reinterpret_cast<double*>(smem_raw + off);        // [gamma+1]
  double* sRatio = sZ + (gamma + 1);                             // [gamma+1] clipped ratios

  // ---- decide.  First every draft position's scalars are fetched in parallel (token -> logit and
  // draft probability are dependent loads), then a warp per row merges that row's chunk statistics.
  float* sL = reinterpret_cast<float*>(sRatio + (gamma + 1));    // [gamma] logit of the draft token
  float* sQ = sL + (gamma + 1);                                  // [gamma] q of the draft token
  float* sU = sQ + (gamma + 1);                                  // [gamma] uniform
  int* sTok = reinterpret_cast<int*>(sU + (gamma + 1));          // [gamma] token, -1 if out of range
  for (int j = tid; j < gamma; j += kSaThreads) {
    const int s = A.draft_tok[g0 + j];
    const bool in = (s >= 0 && s < A.V);
    sTok[j] = in ? s : -1;
    sL[j] = in ? A.logits[(size_t)(r0 + j) * A.V + s] : 0.f;
    sQ[j] = in ? A.q_probs[(size_t)(g0 + j) * A.V + s] : 0.f;
    sU[j] = A.u_accept[g0 + j];
    if (!in && writer) set_status(A.d_status, GS_ERR_INVALID_ARG);
  }
  __syncthreads();
  const double inv_tau = A.tau > 0.f ? 1.0 / (double)A.tau : 0.0;
  for (int j = wid; j <= gamma; j += kSaThreads / 32) {
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
        if (c0s.m > -INFINITY) z += c0s.z * exp(((double)c0s.m - (double)M) * inv_tau);
        if (c1s.m > -INFINITY) z += c1s.z * exp(((double)c1s.m - (double)M) * inv_tau);
      }
    } else {
      for (int cc = lane; cc < A.n_chunk; cc += 32) argmax_merge(M, arg, st[cc].m, st[cc].arg);
      warp_argmax(M, arg);
      if (A.tau > 0.f)
        for (int cc = lane; cc < A.n_chunk; cc += 32)
          if (st[cc].m > -INFINITY) z += st[cc].z * exp(((double)st[cc].m - (double)M) * inv_tau);
    }
    const double Z = warp_sum_f64(z);
    if (lane == 0) {
      sM[j] = M; sArg[j] = arg; sZ[j] = Z;
      if (j < gamma) {
        const int s = sTok[j];
        double p = 0.0, q = 0.0, rho = 0.0;
        if (s >= 0) {
          const float l = sL[j];
          if (A.tau > 0.f) p = (Z > 0.0) ? exp(((double)l - (double)M) * inv_tau) / Z : 0.0;
          else p = (s == arg) ? 1.0 : 0.0;
          q = (double)sQ[j];
          if (q > 0.0) rho = p / q;
          else rho = (p > 0.0) ? (double)INFINITY : 0.0;
        }
        const double u = (double)sU[j];
        sRej[j] = (u > rho) ? 1 : 0;
        const double clipped = rho < 1.0 ? rho : 1.0;
        sRatio[j] = clipped;
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
      if (sRej[j]) { a = j; break; }
    }
    s_acc = a;
    if (writer) {
      A.accepted[i] = a;
      A.n_out[i] = a + 1;
      if (A.alpha_hat != nullptr && A.X != nullptr) {
        if (gamma > 0) {
          double sum = 0.0;
          for (int j = 0; j < gamma; ++j) sum += sRatio[j];
          const double obs = sum / (double)gamma;
          double ah = (1.0 - A.eta) * A.alpha_hat[i] + A.eta * obs;
          ah = ah < A.alpha_min ? A.alpha_min : ah;
          ah = ah > A.alpha_max ? A.alpha_max : ah;
          A.alpha_hat[i] = ah;
        }
        A.X[i] = (1.0 - A.beta) * A.X[i] + A.beta * (double)(a + 1);
      }
    }
  }
  __syncthreads();
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
  const float* qrow = resid ? A.q_probs + (size_t)(g0 + a) * A.V : nullptr;

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

}  // namespace gs

extern "C" size_t gs_spec_accept_workspace(int N, int Tq, int V) {
  if (N <= 0 || Tq <= 0 || V <= 0) return 256;
  return gs::sa_layout(N, Tq, V, nullptr, nullptr);
}

extern "C" gs_status gs_spec_accept(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                    const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                    float temperature, int N, int Tq, int V,
                                    int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                    float* ratio, float* p_tok, float* margin,
                                    double* alpha_hat, double* X, double eta, double beta,
                                    double alpha_min, double alpha_max,
                                    void* ws, size_t ws_bytes, int32_t* d_status, void* stream) {
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
                   (q_probs == nullptr || reinterpret_cast<uintptr_t>(q_probs) % 16 == 0);

  dim3 g1(n_chunk, Tq);
  if (vec) sa_row_stats<true><<<g1, kSaThreads, 0, st>>>(logits, V, n_chunk, k2, w.stats, w.tickets, N);
  else sa_row_stats<false><<<g1, kSaThreads, 0, st>>>(logits, V, n_chunk, k2, w.stats, w.tickets, N);

  SaFinishArgs A;
  A.logits = logits; A.q_probs = q_probs; A.draft_tok = draft_tok; A.cu_q = cu_q; A.u_accept = u_accept;
  A.u_sample = u_sample;
  A.N = N; A.Tq = Tq; A.V = V; A.n_chunk = n_chunk; A.Gamma = Gamma; A.tau = temperature; A.k2 = k2;
  A.accepted = accepted; A.out_tok = out_tok; A.n_out = n_out;
  A.ratio = ratio; A.p_tok = p_tok; A.margin = margin;
  A.alpha_hat = alpha_hat; A.X = X; A.eta = eta; A.beta = beta; A.alpha_min = alpha_min; A.alpha_max = alpha_max;
  A.stats = w.stats; A.tickets = w.tickets; A.mass = w.mass; A.d_status = d_status;
  // rows of one server are bounded by Tq - (N-1); size the dynamic shared memory for that
  const size_t max_rows = (size_t)(Tq - N + 1);
  const size_t smem = align_up(3 * max_rows * 4, 8) + 2 * max_rows * 8 + 4 * max_rows * 4;
  if (smem > 160 * 1024) return GS_ERR_UNSUPPORTED;
  A.smem_bytes = (int)smem;
  if (smem > 40 * 1024) {
    if (cudaFuncSetAttribute(sa_finish<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(sa_finish<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return GS_ERR_CUDA;
  }
  dim3 g2(k2 > 0.f ? n_chunk : 1, N);
  if (vec) sa_finish<true><<<g2, kSaThreads, smem, st>>>(A);
  else sa_finish<false><<<g2, kSaThreads, smem, st>>>(A);
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
  constexpr int kMaxDevices = 64;
  static void* cached[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { *err = GS_ERR_CUDA; return nullptr; }
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
