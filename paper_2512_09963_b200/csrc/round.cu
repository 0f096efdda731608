// gs_verify_round_host: one whole verification round for a caller whose per-round data lives in
// host memory (what the draft servers sent this round), with the model state resident on the GPU.
// It stages the inputs with cudaMemcpyAsync, enqueues the four steps of the round and copies the
// small results back; nothing here computes.  The draft distributions are by far the largest
// input (Gamma x V floats), and the acceptance pass reads little of them: q(s_j) of every drafted
// token and ONE row per server, the row of its first rejection.  Where the caller's buffer is pinned
// memory that the device can address, the kernels therefore read it where it lies (a few MB cross
// the bus instead of Gamma x V x 4 bytes, which at cfg2 take longer than the whole round on the
// device).  Otherwise the distributions travel on a copy stream of the library's own while attention
// and the LM head run, and an event hands them to the caller's stream before gs_spec_accept.
#include "common.cuh"
#include <algorithm>

namespace gs {

struct RoundLayout {
  size_t Q, H, q_probs, draft_tok, u_accept, u_sample, cu_q, cu_kv;     // staged inputs
  size_t O, logits, accepted, out_tok, n_out, ratio, p_tok, S_next, status;
  size_t ws_attn, ws_head, ws_acc, stats;
  size_t ws_attn_bytes, ws_head_bytes, ws_acc_bytes, stats_bytes;
  size_t total;
};

static size_t esize(gs_dtype dt) { return dt == GS_F32 ? 4 : 2; }

static RoundLayout round_layout(const gs_round_desc& r) {
  RoundLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + (bytes ? bytes : 1), 256); return o; };
  const size_t Tq = (size_t)r.Tq, N = (size_t)r.N, Gamma = Tq - N, V = (size_t)r.V;
  L.Q = take(Tq * r.Hq * r.hd * esize(r.dt));
  L.H = take(Tq * r.d * esize(r.dt));
  L.q_probs = take(Gamma * V * 4);
  L.draft_tok = take(Gamma * 4);
  L.u_accept = take(Gamma * 4);
  L.u_sample = take(N * 4);
  L.cu_q = take((N + 1) * 4);
  L.cu_kv = take((N + 1) * 4);
  L.O = take(Tq * r.Hq * r.hd * esize(r.dt));
  L.logits = take(Tq * V * 4);
  L.accepted = take(N * 4);
  L.out_tok = take(Tq * 4);
  L.n_out = take(N * 4);
  L.ratio = take(Gamma * 4);
  L.p_tok = take(Gamma * 4);
  L.S_next = take(N * 4);
  L.status = take(4);
  L.ws_attn_bytes = gs_verify_attn_workspace(r.N, r.Tq, r.total_kv, r.max_kv_len, r.Hq, r.Hkv, r.hd, r.dt);
  L.ws_head_bytes = gs_lm_head_workspace(r.Tq, r.d, r.V, r.dt);
  L.ws_acc_bytes = gs_spec_accept_workspace(r.N, r.Tq, r.V);
  L.ws_attn = take(L.ws_attn_bytes);
  L.ws_head = take(L.ws_head_bytes);
  L.ws_acc = take(L.ws_acc_bytes);
  L.stats_bytes = gs_lm_head_stats_bytes(r.Tq);
  L.stats = take(L.stats_bytes);
  L.total = off;
  return L;
}

// One copy stream and two events per device, created on first use and kept for the process.
struct RoundSide {
  cudaStream_t copy = nullptr;
  cudaEvent_t begin = nullptr, staged = nullptr, h_ready = nullptr;
  bool ok = false;
};
static RoundSide* round_side() {
  static RoundSide side[gs::kMaxDevices];
  const int dev = gs::device_slot();
  if (dev < 0) return nullptr;
  RoundSide& s = side[dev];
  if (!s.ok) {
    if (cudaStreamCreateWithFlags(&s.copy, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&s.begin, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&s.staged, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&s.h_ready, cudaEventDisableTiming) != cudaSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    s.ok = true;
  }
  return &s;
}

static bool desc_ok(const gs_round_desc* r) {
  return r != nullptr && r->N > 0 && r->Tq >= r->N && r->total_kv > 0 && r->max_kv_len > 0 && r->Hq > 0 &&
         r->Hkv > 0 && r->hd > 0 && r->d > 0 && r->V > 0 && r->C >= 0 && (r->dt == GS_F32 || r->dt == GS_BF16);
}


// 1 = read the draft distributions in place where possible, with the first rows copied meanwhile (default);
// 2 = in place, nothing copied; 0 = always stage them.
static int g_round_in_place = 1;
// Bytes of first draft rows the copy engine brings over beside the in-place reads: about what crosses the
// bus while the LM head streams its weight (a quarter of a millisecond at 40-50 GB/s).
constexpr size_t kRoundNearBytes = 10u << 20;

// First draft rows per server that the copy engine brings over beside the in-place reads.
static int round_near_rows(const gs_round_desc& r) {
  if (g_round_in_place == 2) return 0;
  const size_t layer = (size_t)r.N * (size_t)r.V * 4;               // one position of every server
  return (int)std::min<size_t>(kRoundNearBytes / layer, (size_t)8);
}

// The address under which the device can read a host buffer where it lies, or NULL.
static const float* device_view_of_host(const float* h) {
  if (h == nullptr || !g_round_in_place) return nullptr;
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, h) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
  if (at.type != cudaMemoryTypeHost || at.devicePointer == nullptr) return nullptr;
  return static_cast<const float*>(at.devicePointer);
}

}  // namespace gs

extern "C" gs_status gs_verify_round_configure(int read_in_place) {
  if (read_in_place < 0 || read_in_place > 2) return GS_ERR_INVALID_ARG;
  gs::g_round_in_place = read_in_place;
  return GS_OK;
}

extern "C" int gs_verify_round_reads_in_place(const float* h_q_probs) {
  return gs::device_view_of_host(h_q_probs) != nullptr ? 1 : 0;
}

extern "C" int gs_verify_round_near_rows(const gs_round_desc* r) {
  return gs::desc_ok(r) ? gs::round_near_rows(*r) : 0;
}

extern "C" size_t gs_verify_round_workspace(const gs_round_desc* r) {
  if (!gs::desc_ok(r)) return 0;
  return gs::round_layout(*r).total;
}

extern "C" gs_status gs_verify_round_host(const gs_round_desc* r,
                                          const void* h_Q, const void* h_H, const float* h_q_probs,
                                          const int32_t* h_draft_tok, const float* h_u_accept,
                                          const float* h_u_sample, const int32_t* h_cu_q, const int32_t* h_cu_kv,
                                          const void* d_K, const void* d_V, const void* d_W,
                                          double* d_alpha_hat, double* d_X,
                                          const int32_t* d_s_min, const int32_t* d_s_max,
                                          void* d_ws, size_t ws_bytes,
                                          int32_t* h_accepted, int32_t* h_out_tok, int32_t* h_n_out,
                                          int32_t* h_S_next, int32_t* h_status, void* stream) {
  using namespace gs;
  if (!desc_ok(r)) return GS_ERR_INVALID_ARG;
  const size_t Gamma = (size_t)(r->Tq - r->N);
  if (!h_Q || !h_H || !h_u_sample || !h_cu_q || !h_cu_kv || !d_K || !d_V || !d_W || !d_alpha_hat || !d_X ||
      !h_accepted || !h_out_tok || !h_n_out || !h_S_next || !h_status)
    return GS_ERR_INVALID_ARG;
  if (Gamma > 0 && (!h_q_probs || !h_draft_tok || !h_u_accept)) return GS_ERR_INVALID_ARG;
  if (d_ws == nullptr || (reinterpret_cast<uintptr_t>(d_ws) & 255u) != 0) return GS_ERR_WORKSPACE;
  const RoundLayout L = round_layout(*r);
  if (ws_bytes < L.total) return GS_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(d_ws);
  const size_t Tq = (size_t)r->Tq, N = (size_t)r->N, V = (size_t)r->V, es = esize(r->dt);
  auto h2d_on = [&](cudaStream_t q, size_t off, const void* src, size_t bytes) {
    return bytes == 0 || cudaMemcpyAsync(w + off, src, bytes, cudaMemcpyHostToDevice, q) == cudaSuccess;
  };
  auto h2d = [&](size_t off, const void* src, size_t bytes) { return h2d_on(st, off, src, bytes); };
  auto d2h = [&](void* dst, size_t off, size_t bytes) {
    return cudaMemcpyAsync(dst, w + off, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  };
  // First what attention and the LM head need, on the caller's stream (copies are served in the
  // order they are issued, so the large one must not be queued ahead of these) ...
  bool ok = h2d(L.Q, h_Q, Tq * r->Hq * r->hd * es) && h2d(L.cu_q, h_cu_q, (N + 1) * 4) && h2d(L.cu_kv, h_cu_kv, (N + 1) * 4);
  if (!ok || cudaMemsetAsync(w + L.status, 0, 4, st) != cudaSuccess) return GS_ERR_CUDA;
  RoundSide* side = round_side();
  if (side == nullptr) return GS_ERR_CUDA;
  if (cudaEventRecord(side->begin, st) != cudaSuccess) return GS_ERR_CUDA;
  // The hidden states are the LM head's input only: they cross on the copy stream while attention runs.
  if (cudaStreamWaitEvent(side->copy, side->begin, 0) != cudaSuccess || !h2d_on(side->copy, L.H, h_H, Tq * r->d * es) ||
      cudaEventRecord(side->h_ready, side->copy) != cudaSuccess)
    return GS_ERR_CUDA;
  int32_t* d_status = reinterpret_cast<int32_t*>(w + L.status);
  const int32_t* cu_q = reinterpret_cast<const int32_t*>(w + L.cu_q);
  const int32_t* cu_kv = reinterpret_cast<const int32_t*>(w + L.cu_kv);
  gs_status s = gs_verify_attn(w + L.Q, d_K, d_V, w + L.O, cu_q, cu_kv, r->N, r->Tq, r->total_kv, r->max_kv_len,
                               r->Hq, r->Hkv, r->hd, r->scale, r->dt, w + L.ws_attn, L.ws_attn_bytes, d_status, st);
  if (s != GS_OK) return s;
  if (cudaStreamWaitEvent(st, side->h_ready, 0) != cudaSuccess) return GS_ERR_CUDA;
  // LM head with the softmax statistics in its epilogue where the shape has that kernel, so that the
  // acceptance step does not read the logits a second time; the plain pair of calls otherwise.
  int n_chunk = 0;
  s = GS_ERR_UNSUPPORTED;
  if (gs_lm_head_stats_pays(r->Tq))
    s = gs_lm_head_logits_stats(w + L.H, d_W, reinterpret_cast<float*>(w + L.logits), r->Tq, r->d, r->V, r->dt,
                                r->temperature, w + L.stats, L.stats_bytes, &n_chunk, w + L.ws_head, L.ws_head_bytes,
                                d_status, st);
  const bool have_stats = (s == GS_OK);
  if (s == GS_ERR_UNSUPPORTED)
    s = gs_lm_head_logits(w + L.H, d_W, reinterpret_cast<float*>(w + L.logits), r->Tq, r->d, r->V, r->dt,
                          w + L.ws_head, L.ws_head_bytes, d_status, st);
  if (s != GS_OK) return s;
  // ... then what only the acceptance pass reads, over the copy stream.  It starts once the caller's
  // stream has reached this call (the event recorded above: the previous round may still be reading the
  // staging area).  Enqueued after attention and the LM head, so that the device is already at work while
  // the host issues these copies.
  const float* q_in_place = (Gamma > 0) ? device_view_of_host(h_q_probs) : nullptr;
  ok = h2d_on(side->copy, L.draft_tok, h_draft_tok, Gamma * 4) && h2d_on(side->copy, L.u_accept, h_u_accept, Gamma * 4) &&
       h2d_on(side->copy, L.u_sample, h_u_sample, N * 4);
  // In place: the copy engine still brings the FIRST rows of every server over while attention and the
  // LM head run (a rejection is most likely early), as many positions as cross the bus in about the time
  // the LM head takes whatever the batch; the acceptance kernels read a later row from the host buffer.
  int near_rows = 0;
  if (ok && q_in_place != nullptr) {
    near_rows = round_near_rows(*r);
    for (int i = 0; ok && near_rows > 0 && i < r->N; ++i) {
      // a server with inconsistent offsets gets no rows here (the kernels skip and flag it)
      const long long g0 = (long long)h_cu_q[i] - i, gam = (long long)h_cu_q[i + 1] - h_cu_q[i] - 1;
      if (g0 < 0 || gam <= 0 || g0 + gam > (long long)Gamma) continue;
      const size_t rows = (size_t)std::min<long long>(gam, near_rows);
      ok = h2d_on(side->copy, L.q_probs + (size_t)g0 * V * 4, h_q_probs + (size_t)g0 * V, rows * V * 4);
    }
  } else if (ok) {
    ok = h2d_on(side->copy, L.q_probs, h_q_probs, Gamma * V * 4);
  }
  if (!ok || cudaEventRecord(side->staged, side->copy) != cudaSuccess) return GS_ERR_CUDA;
  if (cudaStreamWaitEvent(st, side->staged, 0) != cudaSuccess) return GS_ERR_CUDA;
  const float* lg = reinterpret_cast<const float*>(w + L.logits);
  const float* qp = (q_in_place != nullptr) ? q_in_place : reinterpret_cast<const float*>(w + L.q_probs);
  const int32_t* dtok = reinterpret_cast<const int32_t*>(w + L.draft_tok);
  const float* ua = reinterpret_cast<const float*>(w + L.u_accept);
  const float* us = reinterpret_cast<const float*>(w + L.u_sample);
  int32_t* o_acc = reinterpret_cast<int32_t*>(w + L.accepted);
  int32_t* o_tok = reinterpret_cast<int32_t*>(w + L.out_tok);
  int32_t* o_n = reinterpret_cast<int32_t*>(w + L.n_out);
  float* o_ratio = reinterpret_cast<float*>(w + L.ratio);
  float* o_p = reinterpret_cast<float*>(w + L.p_tok);
  const float* q_near = reinterpret_cast<const float*>(w + L.q_probs);
  s = GS_ERR_UNSUPPORTED;
  if (have_stats)
    s = spec_accept_near(lg, qp, q_near, near_rows, dtok, cu_q, ua, us, r->temperature, r->N, r->Tq, r->V, o_acc, o_tok,
                         o_n, o_ratio, o_p, d_alpha_hat, d_X, r->eta, r->beta, r->alpha_min, r->alpha_max,
                         w + L.stats, n_chunk, w + L.ws_acc, L.ws_acc_bytes, d_status, st);
  if (s == GS_ERR_UNSUPPORTED)
    s = spec_accept_near(lg, qp, q_near, near_rows, dtok, cu_q, ua, us, r->temperature, r->N, r->Tq, r->V, o_acc, o_tok,
                         o_n, o_ratio, o_p, d_alpha_hat, d_X, r->eta, r->beta, r->alpha_min, r->alpha_max,
                         nullptr, 0, w + L.ws_acc, L.ws_acc_bytes, d_status, st);
  if (s != GS_OK) return s;
  s = gs_schedule(d_X, d_alpha_hat, r->N, r->C, d_s_min, d_s_max, reinterpret_cast<int32_t*>(w + L.S_next),
                  d_status, st);
  if (s != GS_OK) return s;
  ok = d2h(h_accepted, L.accepted, N * 4) && d2h(h_out_tok, L.out_tok, Tq * 4) && d2h(h_n_out, L.n_out, N * 4) &&
       d2h(h_S_next, L.S_next, N * 4) && d2h(h_status, L.status, 4);
  return ok ? GS_OK : GS_ERR_CUDA;
}
