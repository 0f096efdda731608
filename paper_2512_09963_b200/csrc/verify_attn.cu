// gs_verify_attn: dispatch between the tensor-core split-KV kernel (bf16, head size 128) and the
// plain kernel (fp32, other head sizes).
#include "common.cuh"
#include "attn_generic.cuh"
#include "attn_tc.cuh"

extern "C" gs_status gs_verify_attn_configure(int tiles_per_split) {
  if (tiles_per_split < 0) return GS_ERR_INVALID_ARG;
  gs::attn_tiles_per_split_override() = tiles_per_split;
  return GS_OK;
}

extern "C" gs_status gs_verify_attn_select(int variant) {
  if (variant != 0 && variant != 1 && variant != 2 && variant != 3 && variant != 4 && variant != 8) return GS_ERR_INVALID_ARG;
  gs::attn_variant_override() = variant;
  return GS_OK;
}

extern "C" size_t gs_verify_attn_workspace(int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv,
                                           int hd, gs_dtype dt) {
  using namespace gs;
  if (N <= 0 || Tq <= 0 || total_kv <= 0 || max_kv_len <= 0 || Hq <= 0 || Hkv <= 0) return 256;
  if (!attn_tc_supported(Hq, Hkv, hd, dt)) return 256;
  return align_up(attn_tc_plan(N, Tq, total_kv, max_kv_len, Hq, Hkv).ws_bytes, 256);
}

extern "C" gs_status gs_verify_attn(const void* Q, const void* K, const void* V, void* O,
                                    const int32_t* cu_q, const int32_t* cu_kv,
                                    int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv, int hd,
                                    float scale, gs_dtype dt,
                                    void* ws, size_t ws_bytes, int32_t* d_status, void* stream) {
  using namespace gs;
  if (N < 0 || Tq < 0 || total_kv < 0 || max_kv_len < 0 || Hq <= 0 || Hkv <= 0 || hd <= 0)
    return GS_ERR_INVALID_ARG;
  if (dt != GS_F32 && dt != GS_BF16) return GS_ERR_INVALID_ARG;
  if (N == 0 || Tq == 0) return GS_OK;
  if (!Q || !K || !V || !O || !cu_q || !cu_kv) return GS_ERR_INVALID_ARG;
  if (Hq % Hkv != 0) return GS_ERR_SHAPE;
  if (hd > 32 * kGenAttnMaxPerLane) return GS_ERR_UNSUPPORTED;
  if (Tq > 65535) return GS_ERR_UNSUPPORTED;
  if (ws == nullptr || ws_bytes < gs_verify_attn_workspace(N, Tq, total_kv, max_kv_len, Hq, Hkv, hd, dt))
    return GS_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dt == GS_F32)
    return launch_attn_generic<float>(Q, K, V, O, cu_q, cu_kv, N, Tq, total_kv, max_kv_len, Hq, Hkv, hd,
                                      scale, d_status, st);
  const bool aligned = (reinterpret_cast<uintptr_t>(Q) % 16 == 0) && (reinterpret_cast<uintptr_t>(K) % 16 == 0) &&
                       (reinterpret_cast<uintptr_t>(V) % 16 == 0) && (reinterpret_cast<uintptr_t>(ws) % 256 == 0);
  if (attn_tc_supported(Hq, Hkv, hd, dt) && aligned && total_kv > 0 && max_kv_len > 0)
    return launch_attn_tc(Q, K, V, O, cu_q, cu_kv, N, Tq, total_kv, max_kv_len, Hq, Hkv, scale, ws, d_status, st);
  return launch_attn_generic<__nv_bfloat16>(Q, K, V, O, cu_q, cu_kv, N, Tq, total_kv, max_kv_len, Hq, Hkv,
                                            hd, scale, d_status, st);
}

// ------------------------------------------------------------------------------------------------
// Paged caches: K and V live in a pool of 128-row pages and every server names its pages in a
// block table, so a cache can grow by whole pages without being moved (Sec. III-A: the verified
// tokens are appended to each server's prefix every round).
extern "C" size_t gs_verify_attn_paged_workspace(int N, int Tq, int max_kv_len, int Hq, int Hkv, int hd, gs_dtype dt) {
  using namespace gs;
  if (N <= 0 || Tq <= 0 || max_kv_len <= 0 || Hq <= 0 || Hkv <= 0) return 256;
  if (!attn_tc_supported(Hq, Hkv, hd, dt)) return 256;
  const long long bound = (long long)N * max_kv_len;
  if (bound > INT_MAX / 2) return 0;
  return align_up(attn_tc_plan(N, Tq, (int)bound, max_kv_len, Hq, Hkv).ws_bytes, 256);
}

extern "C" gs_status gs_verify_attn_paged(const void* Q, const void* K_pool, const void* V_pool, void* O,
                                          const int32_t* cu_q, const int32_t* cu_kv, const int32_t* block_table,
                                          int N, int Tq, int n_pages, int max_pages, int max_kv_len,
                                          int Hq, int Hkv, int hd, float scale, gs_dtype dt,
                                          void* ws, size_t ws_bytes, int32_t* d_status, void* stream) {
  using namespace gs;
  if (N < 0 || Tq < 0 || n_pages < 0 || max_pages < 0 || max_kv_len < 0 || Hq <= 0 || Hkv <= 0 || hd <= 0)
    return GS_ERR_INVALID_ARG;
  if (dt != GS_F32 && dt != GS_BF16) return GS_ERR_INVALID_ARG;
  if (N == 0 || Tq == 0) return GS_OK;
  if (!Q || !K_pool || !V_pool || !O || !cu_q || !cu_kv || !block_table) return GS_ERR_INVALID_ARG;
  if (Hq % Hkv != 0) return GS_ERR_SHAPE;
  if (n_pages == 0 || max_pages == 0 || max_kv_len == 0 || max_kv_len > max_pages * kAtTile) return GS_ERR_SHAPE;
  if (Tq > 65535 || (long long)N * max_kv_len > INT_MAX / 2 || (long long)n_pages * kAtTile > INT_MAX / 2)
    return GS_ERR_UNSUPPORTED;
  const bool aligned = (reinterpret_cast<uintptr_t>(Q) % 16 == 0) && (reinterpret_cast<uintptr_t>(K_pool) % 16 == 0) &&
                       (reinterpret_cast<uintptr_t>(V_pool) % 16 == 0);
  if (!attn_tc_supported(Hq, Hkv, hd, dt) || !aligned) return GS_ERR_UNSUPPORTED;   // tensor-core path only
  if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 ||
      ws_bytes < gs_verify_attn_paged_workspace(N, Tq, max_kv_len, Hq, Hkv, hd, dt))
    return GS_ERR_WORKSPACE;
  return launch_attn_tc(Q, K_pool, V_pool, O, cu_q, cu_kv, N, Tq, N * max_kv_len, max_kv_len, Hq, Hkv, scale, ws,
                        d_status, static_cast<cudaStream_t>(stream), block_table, max_pages, n_pages);
}
