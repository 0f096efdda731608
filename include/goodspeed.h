/*
 * goodspeed.h -- C ABI of the GoodSpeed verification-server hot path for NVIDIA B200 (sm_100a).
 *
 * One verification round of the paper's Algorithm 1 (the verification-server steps:
 * batching, verification, estimator update, GoodSpeed-sched) is four calls:
 *
 *   gs_verify_attn      target attention of every server's gamma_i+1 new positions   (Sec. II-A2)
 *   gs_lm_head_logits   W h of  P_M = softmax(W h)                                   (Sec. II-A1)
 *   gs_spec_accept      softmax, accept/reject, correction/bonus token, estimators   (Sec. II-A2,
 *                                                          Eq. updatealpha, Eq. updateX, Sec. III-C)
 *   gs_schedule         next allocation S(t+1), Eq. goodspeed_sched                  (Sec. III-C)
 *
 * Conventions common to all entry points
 *   - Every tensor pointer is caller-owned DEVICE memory unless a parameter says "host".
 *     The library never allocates, frees or synchronises; scratch comes from a caller
 *     workspace whose size the matching *_workspace() query returns (bytes, 256-aligned base
 *     required).  Workspace contents need not be initialised and are clobbered.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls enqueue work
 *     and return; outputs are valid once the stream has reached that point.
 *   - Return value: GS_OK or a synchronous argument error (nothing was launched).  Errors that
 *     only the device can see (non-monotone offsets, token id outside [0,V)) are written to
 *     *d_status (device int32; sticky: the first non-zero code stays; the caller zeroes it
 *     and reads it after its own synchronisation).  d_status may be NULL.
 *   - Ragged layout.  N servers; server i drafts gamma_i tokens and owns gamma_i+1 verify
 *     positions.  cu_q[N+1] (int32, cu_q[0]=0) are the row offsets of those positions:
 *     rows cu_q[i] .. cu_q[i+1]-1, T_q = cu_q[N].  Arrays with one entry per DRAFT token
 *     (Gamma = T_q - N entries: q_probs rows, draft_tok, u_accept, ratio, p_tok, margin)
 *     place server i at offset cu_q[i]-i.  Row cu_q[i]+j (j = 0..gamma_i) conditions on the
 *     prefix plus draft tokens s_1..s_j, i.e. it is the target distribution p_{j+1}; row
 *     cu_q[i]+gamma_i is the bonus distribution p_{gamma_i+1}.
 */
#ifndef GOODSPEED_H_
#define GOODSPEED_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GS_OK = 0,
  GS_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned pointer */
  GS_ERR_SHAPE = 2,       /* sizes inconsistent with each other or with the offsets */
  GS_ERR_UNSUPPORTED = 3, /* a shape or dtype this build has no kernel for */
  GS_ERR_WORKSPACE = 4,   /* workspace missing or smaller than the query says */
  GS_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
  GS_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out (device status only) */
} gs_status;

typedef enum { GS_F32 = 0, GS_BF16 = 1 } gs_dtype;

const char* gs_status_str(gs_status s);

/* Library/ABI version (major*100 + minor). */
int gs_version(void);

/* Process-wide switch (not thread-safe; default on): whether the library's kernels are launched
 * with the programmatic-dependent-launch attribute.  With it, a kernel's set-up (barrier and
 * tensor-memory allocation, descriptor fetch, cluster rendezvous) overlaps the tail of the kernel
 * before it on the stream; every kernel still waits for its predecessor to finish, with its
 * writes visible, before it touches global memory, so results do not depend on the switch.
 * The paper has no counterpart: this is launch plumbing. */
gs_status gs_set_dependent_launch(int on);

/* --------------------------------------------------------------------------------------------
 * gs_verify_attn -- Sec. II-A2: the target model scores all drafted positions of all servers
 * in one parallel pass.  The paper gives no attention formula; this is scaled-dot-product
 * attention with grouped KV heads, causal among the new positions, full view of the prefix.
 *
 *   Q  [T_q, Hq, hd]            queries of the new positions (rotary etc. already applied)
 *   K,V[total_kv, Hkv, hd]      per-server caches, concatenated; server i owns rows
 *                               cu_kv[i] .. cu_kv[i+1]-1 and its last gamma_i+1 rows are the
 *                               new positions themselves (already appended by the caller)
 *   O  [T_q, Hq, hd]            output, same dtype as Q
 *   New position t (0-based) of server i attends to keys 0 .. L_i+t of that server, with
 *   L_i = (cu_kv[i+1]-cu_kv[i]) - (gamma_i+1).  Query head h reads KV head h / (Hq/Hkv).
 *   dt: GS_F32 (fp32 in/out) or GS_BF16 (bf16 in/out); scores, softmax and accumulation fp32.
 *   max_kv_len: an upper bound on any server's cu_kv[i+1]-cu_kv[i] (sizes the split-KV scratch).
 *   scale: multiplies q.k (pass 1/sqrt(hd)).
 * GS_BF16 with hd = 128 and a group size Hq/Hkv of at most 128 runs on the tensor cores
 * (tcgen05, split over the KV length, partial results merged from the workspace); every other
 * shape runs a plain kernel.
 * Errors: INVALID_ARG (null/negative), SHAPE (Hq % Hkv != 0), UNSUPPORTED (hd > 256, T_q > 65535),
 * WORKSPACE.
 * Device status: GS_ERR_SHAPE if a server has fewer keys than new positions, more keys than
 * max_kv_len, or offsets that decrease; that server's rows are then left unwritten.
 */
size_t gs_verify_attn_workspace(int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv, int hd,
                                gs_dtype dt);
/* Tuning knob of the tensor-core kernel (process-wide, not thread-safe): the number of 128-key tiles
 * one split of a server's KV range covers at most; 0 = automatic (enough splits to give every SM
 * work, but no split shorter than 12 tiles and at most 8 per server).  A large value means no
 * splitting.  Results agree to rounding.  The workspace size depends
 * on it: set it before gs_verify_attn_workspace.  Errors: INVALID_ARG. */
gs_status gs_verify_attn_configure(int tiles_per_split);
/* Kernel choice of the tensor-core path (process-wide, not thread-safe).  0 = automatic: a batch with
 * few (server, block of positions, KV head) groups runs one thread-block cluster of 2, 4 or 8 CTAs per
 * group (each CTA takes a part of the group's keys, the parts are merged through distributed shared
 * memory; the workspace is not touched), every other batch -- and any batch while a split size is
 * forced by gs_verify_attn_configure -- runs persistent CTAs that walk the batch's items and merge
 * KV splits through the workspace.  A batch with no more groups than SMs, but too many for clusters,
 * runs the cluster kernel with one CTA per group.  1 = always the persistent kernel; 2, 4, 8 = always
 * clusters of that size; 3 = always one CTA per group.  Results agree to rounding.  Errors: INVALID_ARG. */
gs_status gs_verify_attn_select(int variant);
gs_status gs_verify_attn(const void* Q, const void* K, const void* V, void* O,
                         const int32_t* cu_q, const int32_t* cu_kv,
                         int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv, int hd,
                         float scale, gs_dtype dt,
                         void* ws, size_t ws_bytes, int32_t* d_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_verify_attn_paged -- the same attention (Sec. II-A2) over caches that grow: Sec. III-A has
 * every round append the verified tokens to each server's prefix, so the caches are kept as pages
 * of a pool and a server's cache grows by whole pages without being moved.
 *
 *   K_pool, V_pool [n_pages * 128, Hkv, hd]   pages of 128 rows (bf16)
 *   block_table    [N, max_pages] int32       page of server i's t-th run of 128 keys (entries beyond
 *                                             the server's length are not read)
 *   cu_kv          [N+1] int32                running sum of the cache LENGTHS (new positions included);
 *                                             key k of server i is row (block_table[i][k/128]*128 + k%128)
 *   everything else as gs_verify_attn; max_kv_len <= max_pages * 128 bounds every length.
 *   Rows of a page beyond the cache length are masked by index but still pass through the tensor
 *   cores with weight zero: they must hold finite numbers (initialise the pool once; stale rows of
 *   earlier use are fine, NaN or Inf bit patterns are not).
 * Tensor-core path only (GS_BF16, hd = 128): other shapes return UNSUPPORTED.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, WORKSPACE.  Device status: GS_ERR_SHAPE as gs_verify_attn,
 * GS_ERR_INVALID_ARG for a block-table entry outside [0, n_pages).
 */
size_t gs_verify_attn_paged_workspace(int N, int Tq, int max_kv_len, int Hq, int Hkv, int hd, gs_dtype dt);
gs_status gs_verify_attn_paged(const void* Q, const void* K_pool, const void* V_pool, void* O,
                               const int32_t* cu_q, const int32_t* cu_kv, const int32_t* block_table,
                               int N, int Tq, int n_pages, int max_pages, int max_kv_len,
                               int Hq, int Hkv, int hd, float scale, gs_dtype dt,
                               void* ws, size_t ws_bytes, int32_t* d_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_lm_head_logits -- Sec. II-A1: logits = W h for every verify position.
 *
 *   H      [T, d]   hidden states, row-major (d contiguous)
 *   W      [d, V]   head weight, row-major (V contiguous)
 *   logits [T, V]   fp32, row-major
 *   logits[t, v] = sum_c H[t, c] * W[c, v], products exact, accumulation fp32.
 *   dt: dtype of H and W.  GS_BF16 runs on the tensor cores (tcgen05, accumulators in tensor
 *   memory) and needs d % 8 == 0, V % 8 == 0 and 16-byte aligned H, W; GS_F32 is a plain FMA
 *   kernel meant for small problems.
 * Errors: INVALID_ARG, UNSUPPORTED (alignment rules above), WORKSPACE, CUDA.
 */
size_t gs_lm_head_workspace(int T, int d, int V, gs_dtype dt);
/* Tuning knobs of the bf16 kernel (process-wide, not thread-safe; 0 = choose automatically):
 * m_tiles = upper bound on the blocks of 128 vocabulary columns a CTA owns per tile (1..9),
 * stages = upper bound on the depth of the shared-memory ring of W, k_rows = rows of W per ring
 * stage (16, 32 or 64).  Results do not depend on them.  Errors: INVALID_ARG. */
gs_status gs_lm_head_configure(int m_tiles, int stages, int k_rows);
/* Kernel choice of the bf16 path (process-wide, not thread-safe): 0 = automatic (CTA pairs
 * where the device can schedule them), 1 = one CTA per tile, 2 = CTA pairs: two SMs share one M = 256 MMA and each loads
 * half of the rows of H, which halves the L2 traffic of H (tile width at most 4 blocks of 256
 * columns; k_rows is ignored).  Results do not depend on the choice.  Errors: INVALID_ARG. */
gs_status gs_lm_head_select(int variant);
gs_status gs_lm_head_logits(const void* H, const void* W, float* logits, int T, int d, int V,
                            gs_dtype dt, void* ws, size_t ws_bytes, int32_t* d_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_lm_head_logits_w4 -- Sec. II-A1 with a 4-bit weight: the paper's larger target model is an
 * AWQ-INT4 checkpoint (Sec. V: Llama3.1-70B-Instruct-AWQ-INT4); it names no storage format, this is
 * the library's own.  The head weight W [d, V] is given as
 *
 *   qweight [d/8, V]     uint32   eight 4-bit codes per word, along d: the code of W[8w + j, v]
 *                                 (j = 0..7) sits in bits [4n, 4n+4) of qweight[w, v] with
 *                                 n = (j >> 1) + 4 (j & 1)  (nibbles 0..3 hold j = 0, 2, 4, 6 and
 *                                 nibbles 4..7 hold j = 1, 3, 5, 7: a shift and one mask then yield
 *                                 two neighbouring k in the two halves of a register)
 *   scales  [d/group, V] bf16     one scale per group of `group` consecutive k and column
 *   zeros   [d/group, V] uint8    the group's zero point, 0..15
 *   W[k, v] = scales[k / group, v] * (code[k, v] - zeros[k / group, v])
 *
 *   H [T, d] bf16, logits [T, V] fp32 as gs_lm_head_logits:
 *   logits[t, v] = sum_k H[t, k] * bf16(W[k, v])   -- every weight is rounded to bf16 once (the one
 *   multiplication by the scale), products exact, accumulation fp32 on the tensor cores.
 * Needs group == 64 or group % 128 == 0, d % 128 == 0, d % group == 0, V % 16 == 0 and 16-byte aligned pointers (UNSUPPORTED
 * otherwise).  No workspace.  More than 256 rows stream the weights once per 256 rows.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.  Device status: GS_ERR_TIMEOUT only.
 */
gs_status gs_lm_head_logits_w4(const void* H, const uint32_t* qweight, const void* scales, const uint8_t* zeros,
                               int group, float* logits, int T, int d, int V, int32_t* d_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_spec_accept -- Sec. II-A2 (acceptance rule, accepted count m, correction / bonus token),
 * with the estimator updates of Sec. III-C fused at its tail (Eq. updatealpha, Eq. updateX).
 *
 *   logits   [T_q, V] fp32     target logits (rows as described at the top)
 *   q_probs  [Gamma, V] fp32   draft distributions q_{i,j}
 *   draft_tok[Gamma] int32     draft tokens s_{i,j}
 *   u_accept [Gamma] fp32      the uniforms r_j of the acceptance test, in (0,1)
 *   u_sample [N] fp32          one uniform per server for the correction / bonus draw
 *   temperature                p_j = softmax(logits_j / temperature); 0 means greedy: p_j is the
 *                              one-hot at the lowest-index argmax
 * Outputs
 *   accepted [N] int32         a_i = number of accepted draft tokens, 0 <= a_i <= gamma_i
 *   out_tok  [T_q] int32       server i's segment: a_i accepted draft tokens, then the
 *                              correction (a_i < gamma_i) or bonus token, then -1 padding
 *   n_out    [N] int32         a_i + 1
 *   ratio    [Gamma] fp32      min(1, p_j(s_j)/q_j(s_j)) for EVERY draft position
 *   p_tok    [Gamma] fp32      p_j(s_j)
 *   margin   [Gamma + N] fp32  nullable.  First Gamma: u_j - p_j(s_j)/q_j(s_j) (signed).  Last N:
 *                              distance of the sampling threshold to the nearer edge of the
 *                              emitted token's CDF interval, in units of the total mass.
 * Rules: s_j is accepted iff u_j <= p_j(s_j)/q_j(s_j); q_j(s_j)=0 accepts iff p_j(s_j)>0;
 * verification stops at the first rejection.  The last token is drawn by inverse CDF in
 * ascending token id, smallest v whose cumulative mass exceeds u_sample * total, from
 * max(0, p - q) at the rejected position, or from p of the bonus row; if max(0, p - q) has no
 * mass the draw falls back to p.
 * Estimators (alpha_hat, X: [N] fp64 in/out, both NULL to skip):
 *   alpha_hat_i <- clamp((1-eta) alpha_hat_i + eta * mean_j ratio_j, alpha_min, alpha_max)
 *                  (unchanged when gamma_i = 0);  X_i <- (1-beta) X_i + beta (a_i + 1).
 * Errors: INVALID_ARG, SHAPE (T_q < N), WORKSPACE.  Device status: GS_ERR_SHAPE for a server whose
 * offsets leave it without a row, or leave a server before or after it without one (decreasing
 * offsets, cu_q[N] > T_q): that server gets accepted = n_out = 0 and nothing else of it is read or
 * written; GS_ERR_INVALID_ARG for a draft token outside [0, V) (it is then rejected).
 */
size_t gs_spec_accept_workspace(int N, int Tq, int V);
/* Kernel choice of the second pass (process-wide, not thread-safe): 0 = automatic: one thread-block
 * cluster per server, slices of the selected row held in shared memory and slice masses exchanged
 * through distributed shared memory, where V % 4 == 0, the rows are 16-byte aligned and one row
 * slice fits a CTA's shared memory; 1 = always the ticket kernel (chunk masses through the
 * workspace, the last CTA of a server draws).  Accept decisions, ratios and estimators do not depend
 * on the choice; the drawn token can differ only when u_sample * total lies within rounding of a
 * CDF step.  Errors: INVALID_ARG. */
gs_status gs_spec_accept_select(int variant);
gs_status gs_spec_accept(const float* logits, const float* q_probs, const int32_t* draft_tok,
                         const int32_t* cu_q, const float* u_accept, const float* u_sample,
                         float temperature, int N, int Tq, int V,
                         int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                         float* ratio, float* p_tok, float* margin,
                         double* alpha_hat, double* X, double eta, double beta,
                         double alpha_min, double alpha_max,
                         void* ws, size_t ws_bytes, int32_t* d_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_lm_head_logits_stats + gs_spec_accept_prestats -- Sec. II-A1 and II-A2 as one computation:
 * P_M = softmax(W h) needs, per verify position, the maximum and the sum of exponentials of the
 * logits.  gs_spec_accept obtains them by reading every logit once more; here the LM head's epilogue
 * writes them while it still holds the logits in tensor memory, and the acceptance step starts from
 * them.
 *
 * gs_lm_head_logits_stats: arguments and results as gs_lm_head_logits, plus
 *   temperature   the softmax temperature the statistics are for (0 = greedy: maxima only)
 *   stats         device buffer of gs_lm_head_stats_bytes(T) bytes, 16-byte aligned; receives
 *                 *n_chunk entries per row (one per CTA of the launch; opaque)
 *   n_chunk       host int, written before the call returns
 *   bf16 on CTA pairs with T <= 512 only; every other case returns GS_ERR_UNSUPPORTED and launches
 *   nothing (call gs_lm_head_logits and gs_spec_accept instead).
 * gs_spec_accept_prestats: arguments and results as gs_spec_accept (same temperature!), plus the
 *   stats buffer and n_chunk.  Needs V % 4 == 0, 16-byte aligned rows and a vocabulary slice that
 *   fits shared memory (the cluster kernel); otherwise GS_ERR_UNSUPPORTED and nothing is launched.
 * Accept decisions and probabilities agree with gs_spec_accept to rounding (the sums of
 * exponentials are grouped differently).
 */
size_t gs_lm_head_stats_bytes(int T);
/* 1 where the statistics epilogue is expected to make the round shorter than the separate statistics
 * pass of gs_spec_accept (up to 256 rows: the extra epilogue work hides under the next tile's MMAs), 0
 * where it is not (more rows: a single accumulator, every epilogue holds up the tensor core). */
int gs_lm_head_stats_pays(int T);
gs_status gs_lm_head_logits_stats(const void* H, const void* W, float* logits, int T, int d, int V,
                                  gs_dtype dt, float temperature, void* stats, size_t stats_bytes,
                                  int* n_chunk, void* ws, size_t ws_bytes, int32_t* d_status, void* stream);
gs_status gs_spec_accept_prestats(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                  const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                  float temperature, int N, int Tq, int V,
                                  int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                  float* ratio, float* p_tok, float* margin,
                                  double* alpha_hat, double* X, double eta, double beta,
                                  double alpha_min, double alpha_max,
                                  const void* stats, int n_chunk,
                                  void* ws, size_t ws_bytes, int32_t* d_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_spec_accept_static -- no counterpart in the paper: a convenience of this library.
 *
 * The same computation, arguments and results as gs_spec_accept, for callers that cannot provide
 * a workspace because they are not allowed to allocate device memory where the round runs (a
 * serving loop with a memory pool frozen at start-up, a plug-in that only borrows its input and
 * output buffers, a context in which an allocation would stall or fail).  The scratch is a fixed
 * array of gs_spec_accept_static_capacity() bytes (2 MiB) inside the library; every GPU that
 * loads the library holds that array until the process ends.  The call itself allocates nothing.
 *   - Limit: gs_spec_accept_workspace(N, Tq, V) must not exceed the capacity (for V = 151936 that
 *     is about 6800 verify positions); larger problems return GS_ERR_WORKSPACE and launch nothing.
 *   - The first call on each device looks the array's device address up (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls share the one array.  Nothing in it has to be cleared between calls (every word a
 *     call reads it has written before), but two calls that overlap on the GPU (different
 *     streams, or different host threads) race on it and give wrong results: keep them ordered.
 * Errors: as gs_spec_accept, plus WORKSPACE for the size limit and CUDA if the address lookup fails.
 */
size_t gs_spec_accept_static_capacity(void);
gs_status gs_spec_accept_static(const float* logits, const float* q_probs, const int32_t* draft_tok,
                                const int32_t* cu_q, const float* u_accept, const float* u_sample,
                                float temperature, int N, int Tq, int V,
                                int32_t* accepted, int32_t* out_tok, int32_t* n_out,
                                float* ratio, float* p_tok, float* margin,
                                double* alpha_hat, double* X, double eta, double beta,
                                double alpha_min, double alpha_max,
                                int32_t* d_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_schedule -- GoodSpeed-sched (Eq. goodspeed_sched, Sec. III-C) with U_i = log:
 *   maximise sum_i (1/X_i) (1 - alpha_hat_i^(S_i+1)) / (1 - alpha_hat_i)
 *   subject to sum_i S_i <= C, s_min_i <= S_i <= s_max_i, S_i integer.
 * Solved exactly by marginal allocation: the gain of raising S_i from s to s+1 is
 * alpha_hat_i^(s+1)/X_i, decreasing in s; start at s_min and give the remaining budget one token
 * at a time to the largest gain (lowest index on ties).  Gains are formed as alpha_hat_i/X_i
 * followed by repeated fp64 multiplication by alpha_hat_i, so results are reproducible bit for bit.
 *
 *   X, alpha_hat [N] fp64 (device);  s_min, s_max [N] int32 nullable (0 and C);  S_out [N] int32.
 * Errors: INVALID_ARG, UNSUPPORTED (N > 1024).  If sum s_min > C the floors are returned as they
 * are and *d_status = GS_ERR_SHAPE.
 */
gs_status gs_schedule(const double* X, const double* alpha_hat, int N, int C,
                      const int32_t* s_min, const int32_t* s_max, int32_t* S_out,
                      int32_t* d_status, void* stream);
/* Kernel choice (process-wide, not thread-safe): 0 = automatic: for N <= 32 (and N*C*8 bytes of
 * shared memory available) every server's gain list is written out once and each server finds by
 * bisection how many of its entries rank among the `budget` largest of all lists in the order
 * (gain descending, server ascending, step ascending), which is the set the greedy hands out;
 * 1 = always the token-by-token greedy.  The allocation does not depend on the choice.
 * Errors: INVALID_ARG. */
gs_status gs_schedule_select(int variant);

/* gs_schedule_host -- the same GoodSpeed-sched allocation (Eq. goodspeed_sched, Sec. III-C) for
 * estimator state in HOST memory: every pointer is a host pointer, no CUDA call is made, the result
 * is in S_out when the call returns.  Same marginal-allocation steps and the same chain of fp64
 * multiplications as gs_schedule, so the two give identical allocations for identical inputs.  Meant
 * for a scheduler that runs beside the GPU or on ranks that have exchanged their estimates; cost
 * O(N * C).  Errors: INVALID_ARG (null/negative), UNSUPPORTED (N > 2^20), SHAPE if sum s_min > C (the
 * floors are then returned as they are). */
gs_status gs_schedule_host(const double* X, const double* alpha_hat, int N, int C,
                           const int32_t* s_min, const int32_t* s_max, int32_t* S_out);

/* --------------------------------------------------------------------------------------------
 * gs_verify_round_host -- Algorithm 1, the verification-server steps of one round (batching,
 * verification, estimator update, GoodSpeed-sched), for a caller whose per-round data is in HOST
 * memory: what the draft servers sent (draft tokens, full draft distributions, Alg. 1 "Send
 * s_i(t), q_{i,j}") plus the hidden states and queries of the new positions.  The KV caches, the
 * head weight and the estimator state stay resident on the device.
 *
 *   h_*      host pointers (pinned memory lets the copies overlap); shapes as in the calls above
 *   d_K,d_V  [total_kv, Hkv, hd], d_W [d, V]: device, resident; d_alpha_hat, d_X [N] fp64 device,
 *            updated in place; d_s_min/d_s_max [N] int32 device, nullable
 *   d_ws     device scratch of gs_verify_round_workspace() bytes, 256-aligned; it also holds the
 *            attention output O and the logits of the round
 *   outputs  h_accepted[N], h_out_tok[T_q], h_n_out[N], h_S_next[N], h_status[1] (device status)
 * The call enqueues host->device copies, gs_verify_attn, gs_lm_head_logits, gs_spec_accept (with
 * the estimator update), gs_schedule and the device->host copies and returns; the host outputs are
 * valid after the caller synchronises `stream`.  Host buffers must stay untouched until then.
 * The hidden states (read only by the LM head) and the draft distributions, tokens and uniforms (read
 * only by the acceptance pass) are copied on a stream of the library's own (one per device, created on
 * the first call together with three events; make that first call outside any stream capture) while
 * attention and the LM head run on `stream`; `stream` waits for them before the call that reads them,
 * and they wait for `stream` to reach this call, so back-to-back rounds on one stream are ordered.  Rounds issued on DIFFERENT streams with the same
 * d_ws race, as they would anyway.
 * Draft distributions in pinned memory that the device can address (cudaHostAlloc, or cudaHostRegister
 * with the mapped flag) are NOT copied: the acceptance pass needs q(s_j) of the drafted tokens and one
 * row per server (the row of its first rejection), and its kernels read those from the host buffer
 * over the bus -- at most N*V*4 + 32*Gamma bytes instead of Gamma*V*4 (see gs_verify_round_configure);
 * the first rows of every server are copied meanwhile (gs_verify_round_near_rows) and read on the device.
 * Errors: as the four calls; CUDA if a copy could not be enqueued.
 */
typedef struct gs_round_desc {
  int N, Tq, total_kv, max_kv_len, Hq, Hkv, hd, d, V, C;
  gs_dtype dt;
  float scale, temperature;
  double eta, beta, alpha_min, alpha_max;
} gs_round_desc;

size_t gs_verify_round_workspace(const gs_round_desc* r);
/* Whether gs_verify_round_host may read the draft distributions where they lie (process-wide, not
 * thread-safe; 1 = yes, with the first rows of every server copied meanwhile: the default; 2 = yes, and
 * nothing of them is copied; 0 = always stage them in the workspace).  Results do not depend on it.
 * Errors: INVALID_ARG. */
gs_status gs_verify_round_configure(int read_in_place);
/* 1 if gs_verify_round_host would read this host buffer of draft distributions in place (it is pinned
 * memory with a device address and in-place reads are on), 0 if it would stage it. */
int gs_verify_round_reads_in_place(const float* h_q_probs);
/* Beside the in-place reads the copy engine still brings the FIRST rows of every server's draft
 * distributions to the device while attention and the LM head run (a rejection is most likely early, and
 * a row that is already there need not cross the bus when the acceptance pass wants it): this many
 * positions per server, as many as about 10 MB hold, at most 8 (0 for an invalid descriptor). */
int gs_verify_round_near_rows(const gs_round_desc* r);
gs_status gs_verify_round_host(const gs_round_desc* r,
                               const void* h_Q, const void* h_H, const float* h_q_probs,
                               const int32_t* h_draft_tok, const float* h_u_accept, const float* h_u_sample,
                               const int32_t* h_cu_q, const int32_t* h_cu_kv,
                               const void* d_K, const void* d_V, const void* d_W,
                               double* d_alpha_hat, double* d_X,
                               const int32_t* d_s_min, const int32_t* d_s_max,
                               void* d_ws, size_t ws_bytes,
                               int32_t* h_accepted, int32_t* h_out_tok, int32_t* h_n_out,
                               int32_t* h_S_next, int32_t* h_status, void* stream);

/* --------------------------------------------------------------------------------------------
 * gs_selftest_wait_timeout -- no counterpart in the paper: a check of the library's failure path.
 * Every device-side wait of this library (on an mbarrier a TMA load, an MMA or another warp
 * completes) is bounded: when it runs out the kernel raises an abort flag, all its roles leave their
 * loops, GS_ERR_TIMEOUT goes to *d_status and the kernel ends normally, so the context stays usable.
 * This call launches one warp that waits, with that same wait routine, for a barrier nothing ever
 * completes, with a limit of limit_us microseconds (1 .. 1 000 000) instead of the production 2 s.
 *   d_status     device int32 (required): receives GS_ERR_TIMEOUT (sticky like every device status)
 *   d_waited_ns  device uint64, nullable: how long the wait lasted
 * Errors: INVALID_ARG.  Nothing faults and nothing waits beyond the limit. */
gs_status gs_selftest_wait_timeout(unsigned int limit_us, int32_t* d_status, unsigned long long* d_waited_ns,
                                   void* stream);

/* Number of CUDA kernels the library has launched so far in this process (host-side counter). */
unsigned long long gs_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* GOODSPEED_H_ */
