// gs_lm_head_logits: logits = H W (Sec. II-A1).
//
// bf16 path (tcgen05 / tensor memory).  The product is computed transposed, logits^T = W^T H^T:
// the vocabulary dimension is the MMA's M (128 columns of W per MMA, read as an MN-major A
// operand straight from W's [d, V] layout) and the verify positions are the MMA's N (H is the
// K-major B operand).  A CTA owns a tile of up to 9 consecutive 128-column units for ALL
// positions, so W is streamed from HBM exactly once and each k row of a tile is one long
// contiguous run; H (a few MB) is re-read from L2 through its own small ring.  With the
// vocabulary on the TMEM lanes, an epilogue thread holds one vocabulary column and a warp's
// store of one position is 32 consecutive floats of the row-major [T, V] output.
//
//   warp 0     TMA producer: W boxes (kw k rows x 64 v, 128-byte swizzle) into a deep ring of
//              stages, H boxes (n_tile rows x 64 k) into a 3-stage ring
//   warp 1     allocates tensor memory, issues tcgen05.mma (one thread), commits stages back
//   warps 2-5  epilogue: tcgen05.ld the fp32 accumulators, store logits
// Tiles are spread so that every SM gets the same number of them and widths differ by at most
// one unit.  Accumulators are double-buffered in tensor memory when they fit.  Every barrier
// wait is time-bounded.
//
// fp32 inputs use a plain FMA kernel (small problems only).
#include "common.cuh"
#include "attn_generic.cuh"
#include "sm100_ptx.cuh"
#include "lm_head_w4.cuh"

namespace gs {

// ------------------------------------------------------------------ plain kernel (fp32)
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
  count_launches(1);
  return launch_status();
}

// ------------------------------------------------------------------ tcgen05 kernel (bf16)
constexpr int kTcThreads = 192;
constexpr uint32_t kBlockK = 64;            // k depth of one H stage = one 128-byte swizzle row
constexpr uint32_t kTileM = 128;            // vocabulary columns per MMA ("unit")
constexpr uint32_t kMaxSmem = 232448;       // 227 KB
constexpr int kMaxRowsPerLaunch = 512;      // tensor memory has 512 fp32 columns
constexpr int kHStages = 3;

struct HeadTcParams {
  float* logits;
  int32_t* d_status;
  int T, d, V;
  int row0;              // first row of H / logits this launch covers
  int nt, n_tile;        // N tiles and rows of H per N tile
  int n_acc;             // accumulator buffers in tensor memory
  int kw;                // k rows of W per W stage (16, 32 or 64)
  int w_stages, k_blocks;
  int num_tiles;         // tiles of the vocabulary; tile i is `unit_base + (i < unit_rem)` units wide
  int unit_base, unit_rem;
  uint32_t w_stage_bytes, h_stage_bytes, acc_cols, tmem_cols;
};

// Tile i covers units [unit0, unit0 + width) of 128 vocabulary columns each.
GS_DEVINL void head_tile(const HeadTcParams& P, int i, int& unit0, int& width) {
  width = P.unit_base + (i < P.unit_rem ? 1 : 0);
  unit0 = i * P.unit_base + min(i, P.unit_rem);
}

constexpr int kMaxUnits = 9;                // widest tile, in units

// MMAs of one W stage (KW k rows) for a tile WIDTH units wide: every offset is a compile-time
// constant added to the per-stage base.
template <int KW, int NT, int WIDTH>
GS_DEVINL void head_issue_stage(uint32_t d_acc, uint32_t a_hi, uint32_t a_lo_stage, uint32_t b_hi, uint32_t b_lo_sub,
                                uint32_t n_tile, uint32_t n_tile_u, uint32_t idesc, uint32_t fresh) {
  constexpr uint32_t w_box_u = ((uint32_t)KW * 128u) >> 4;
#pragma unroll
  for (int kk = 0; kk < KW / 16; ++kk) {
    const uint32_t accum = (kk == 0) ? (fresh ^ 1u) : 1u;
#pragma unroll
    for (int m = 0; m < WIDTH; ++m) {
      const uint64_t adesc = ((uint64_t)a_hi << 32) | (a_lo_stage + (uint32_t)(m * 2) * w_box_u + (uint32_t)(kk * 128));
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const uint64_t bdesc = ((uint64_t)b_hi << 32) | (b_lo_sub + (uint32_t)j * n_tile_u + (uint32_t)(kk * 2));
        umma_bf16(d_acc + (uint32_t)(m * NT + j) * n_tile, adesc, bdesc, idesc, accum);
      }
    }
  }
}

// KW = k rows of W per ring stage, NT = number of N tiles.  Both are compile-time so that the
// MMA issue loop unrolls completely: every descriptor is then "a per-stage base plus a constant",
// which keeps the single issuing thread ahead of the tensor core even when an MMA is short
// (a 128 x 48 x 16 MMA occupies the tensor core for about 45 cycles).
template <int KW, int NT>
__global__ void __launch_bounds__(kTcThreads, 1)
lm_head_tc_kernel(const __grid_constant__ CUtensorMap tmapW, const __grid_constant__ CUtensorMap tmapH,
                  const HeadTcParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;            // stages need 1024-byte alignment
  uint8_t* sm = smem_raw + (base - raw);
  const uint32_t h_base = base + (uint32_t)P.w_stages * P.w_stage_bytes;
  const uint32_t bars = h_base + (uint32_t)kHStages * P.h_stage_bytes;
  const int WS = P.w_stages;
  auto wfull_bar = [&](int s) { return bars + 8u * (uint32_t)s; };
  auto wempty_bar = [&](int s) { return bars + 8u * (uint32_t)(WS + s); };
  auto hfull_bar = [&](int s) { return bars + 8u * (uint32_t)(2 * WS + s); };
  auto hempty_bar = [&](int s) { return bars + 8u * (uint32_t)(2 * WS + kHStages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * WS + 2 * kHStages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * WS + 2 * kHStages + 2 + a); };
  const uint32_t n_bars = (uint32_t)(2 * WS + 2 * kHStages + 4);
  uint8_t* tail = sm + (bars - base) + 8u * n_bars;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < WS; ++s) { mbar_init(wfull_bar(s), 1); mbar_init(wempty_bar(s), 1); }
    for (int s = 0; s < kHStages; ++s) { mbar_init(hfull_bar(s), 1); mbar_init(hempty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    tma_prefetch_desc(&tmapW);
    tma_prefetch_desc(&tmapH);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), P.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                    // the prologue above overlaps the previous kernel's tail
  pdl_launch_dependents();       // after the wait: what the successor reads before its own wait is complete by now
  const uint32_t tmem_base = *tmem_slot;
  constexpr int subs = (int)kBlockK / KW;               // W stages per H stage
  constexpr uint32_t w_box_bytes = (uint32_t)KW * 128u; // one box: KW k rows x 64 v

  if (warp == 0) {
    // ---------------- TMA producer (loads are issued in the order the MMA warp consumes them);
    // the whole warp walks the loops, one elected lane issues
    uint32_t ws = 0, wph = 0, hs = 0, hph = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x) {
      int unit0, width;
      head_tile(P, tile, unit0, width);
      const int v0 = unit0 * (int)kTileM;
      const int boxes = 2 * width;
      for (int kb = 0; kb < P.k_blocks && ok; ++kb) {
        const int k0 = kb * (int)kBlockK;
        if (!mbar_wait_warp(hempty_bar(hs), hph ^ 1u, abort_flag)) { ok = false; break; }
        if (elect_one()) {
          mbar_arrive_expect_tx(hfull_bar(hs), P.h_stage_bytes);
          for (int j = 0; j < NT; ++j)
            tma_load_2d(h_base + hs * P.h_stage_bytes + (uint32_t)(j * P.n_tile) * 128u, &tmapH, k0,
                        P.row0 + j * P.n_tile, hfull_bar(hs));
        }
        __syncwarp();
        if (++hs == (uint32_t)kHStages) { hs = 0; hph ^= 1u; }
        for (int sub = 0; sub < subs; ++sub) {
          if (!mbar_wait_warp(wempty_bar(ws), wph ^ 1u, abort_flag)) { ok = false; break; }
          if (elect_one()) {
            mbar_arrive_expect_tx(wfull_bar(ws), (uint32_t)boxes * w_box_bytes);
            const uint32_t dst = base + ws * P.w_stage_bytes;
            for (int b = 0; b < boxes; ++b)
              tma_load_2d(dst + (uint32_t)b * w_box_bytes, &tmapW, v0 + b * 64, k0 + sub * KW, wfull_bar(ws));
          }
          __syncwarp();
          if (++ws == (uint32_t)WS) { ws = 0; wph ^= 1u; }
        }
      }
    }
    if (!ok) {
      // Let loads that are still in flight land before the CTA goes away (bounded).
      const uint64_t t0 = global_timer_ns();
      while (global_timer_ns() - t0 < 200000ull) { }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer: the whole warp walks the loops, one elected lane issues
    const uint32_t idesc = idesc_bf16(kTileM, (uint32_t)P.n_tile, /*A (W^T) MN-major*/ true, /*B (H) K-major*/ false);
    // Descriptors differ only in their low word (the start address >> 4).
    //   A (W^T, MN-major): two 64-column boxes KW*128 bytes apart (leading offset), 8-k groups
    //                      1024 bytes apart (stride offset); 16 k further = +2048 bytes.
    //   B (H, K-major):    rows of 128 bytes, 8-row groups 1024 bytes apart; 16 k further = +32 bytes.
    const uint64_t a_desc0 = smem_desc_sw128(base, w_box_bytes, 1024u);
    const uint64_t b_desc0 = smem_desc_sw128(h_base, 16u, 1024u);
    const uint32_t a_hi = (uint32_t)(a_desc0 >> 32), a_lo0 = (uint32_t)a_desc0;
    const uint32_t b_hi = (uint32_t)(b_desc0 >> 32), b_lo0 = (uint32_t)b_desc0;
    const uint32_t w_stage_u = P.w_stage_bytes >> 4, h_stage_u = P.h_stage_bytes >> 4;
    const uint32_t n_tile_u = ((uint32_t)P.n_tile * 128u) >> 4;       // one N tile of H, in 16-byte units
    const uint32_t n_tile = (uint32_t)P.n_tile;
    uint32_t ws = 0, wph = 0, hs = 0, hph = 0;
    int it = 0;
    bool ok = true;
    constexpr int k16_per_stage = KW / 16;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x, ++it) {
      int unit0, width;
      head_tile(P, tile, unit0, width);
      const int acc = it % P.n_acc;
      const uint32_t acc_ph = (uint32_t)(it / P.n_acc) & 1u;
      if (!mbar_wait_warp(tempty_bar(acc), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t d_acc = tmem_base + (uint32_t)acc * P.acc_cols;
      for (int kb = 0; kb < P.k_blocks && ok; ++kb) {
        if (!mbar_wait_warp(hfull_bar(hs), hph, abort_flag)) { ok = false; break; }
        const uint32_t b_lo_stage = b_lo0 + hs * h_stage_u;
#pragma unroll
        for (int sub = 0; sub < subs; ++sub) {
          if (!mbar_wait_warp(wfull_bar(ws), wph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          if (elect_one()) {
            const uint32_t a_lo_stage = a_lo0 + ws * w_stage_u;
            const uint32_t b_lo_sub = b_lo_stage + (uint32_t)(sub * k16_per_stage * 2);
            const uint32_t fresh = (kb == 0 && sub == 0) ? 1u : 0u;    // first MMAs of the tile overwrite
            switch (width) {
              case 1: head_issue_stage<KW, NT, 1>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              case 2: head_issue_stage<KW, NT, 2>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              case 3: head_issue_stage<KW, NT, 3>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              case 4: head_issue_stage<KW, NT, 4>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              case 5: head_issue_stage<KW, NT, 5>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              case 6: head_issue_stage<KW, NT, 6>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              case 7: head_issue_stage<KW, NT, 7>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              case 8: head_issue_stage<KW, NT, 8>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
              default: head_issue_stage<KW, NT, 9>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_sub, n_tile, n_tile_u, idesc, fresh); break;
            }
            umma_commit(wempty_bar(ws));      // frees the W stage once these MMAs have read it
            if (sub == subs - 1) umma_commit(hempty_bar(hs));
          }
          __syncwarp();
          if (++ws == (uint32_t)WS) { ws = 0; wph ^= 1u; }
        }
        if (++hs == (uint32_t)kHStages) { hs = 0; hph ^= 1u; }
      }
      if (ok && elect_one()) umma_commit(tfull_bar(acc));
      __syncwarp();
    }
    if (!ok) {
      // MMAs may still be running: give them (bounded) time before TMEM is freed.
      const uint64_t t0 = global_timer_ns();
      while (global_timer_ns() - t0 < 200000ull) { }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue (warps 2..5): TMEM lane quadrant = warp % 4
    const int q = warp & 3;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x, ++it) {
      int unit0, width;
      head_tile(P, tile, unit0, width);
      const int acc = it % P.n_acc;
      const uint32_t acc_ph = (uint32_t)(it / P.n_acc) & 1u;
      if (!mbar_wait(tfull_bar(acc), acc_ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      for (int m = 0; m < width; ++m) {
        const int v = (unit0 + m) * (int)kTileM + q * 32 + lane;
        for (int j = 0; j < NT; ++j) {
          for (int c0 = 0; c0 < P.n_tile; c0 += 16) {
            const int t_first = j * P.n_tile + c0;
            if (t_first >= P.T) break;                       // warp-uniform
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * P.acc_cols +
                                   (uint32_t)((m * NT + j) * P.n_tile + c0);
            uint32_t r[16];
            tmem_ld16(taddr, r);
            tmem_ld_wait();
            if (v < P.V) {
              float* out = P.logits + (size_t)(P.row0 + t_first) * P.V + v;
#pragma unroll
              for (int c = 0; c < 16; ++c)
                if (t_first + c < P.T) out[(size_t)c * P.V] = __uint_as_float(r[c]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) set_status(P.d_status, GS_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, P.tmem_cols);
  }
}

static int g_head_mt = 0;       // 0 = choose automatically
static int g_head_stages = 0;
static int g_head_kw = 0;
static int g_head_variant = 0;  // 0 = choose automatically, 1 = one CTA per tile, 2 = CTA pairs

inline gs_status launch_lm_head_tc(const void* H, const void* W, float* logits, int T, int d, int V,
                                   int32_t* d_status, cudaStream_t st) {
  using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const HeadTcParams);
  static const KernelFn kernels[3][2] = {
      {lm_head_tc_kernel<16, 1>, lm_head_tc_kernel<16, 2>},
      {lm_head_tc_kernel<32, 1>, lm_head_tc_kernel<32, 2>},
      {lm_head_tc_kernel<64, 1>, lm_head_tc_kernel<64, 2>}};
  static PerDeviceOnce attr_set;
  const int slot = device_slot();
  if (attr_set.needed(slot)) {
    for (int a = 0; a < 3; ++a)
      for (int b = 0; b < 2; ++b)
        if (cudaFuncSetAttribute(kernels[a][b], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem) !=
            cudaSuccess)
          return GS_ERR_CUDA;
    attr_set.mark(slot);
  }
  const int sms = sm_count();
  const int units = (V + (int)kTileM - 1) / (int)kTileM;
  for (int row0 = 0; row0 < T; row0 += kMaxRowsPerLaunch) {
    const int rows = min(kMaxRowsPerLaunch, T - row0);
    HeadTcParams P;
    P.logits = logits; P.d_status = d_status;
    P.T = rows; P.d = d; P.V = V; P.row0 = row0;
    P.nt = (rows + 255) / 256;
    P.n_tile = (((rows + P.nt - 1) / P.nt) + 15) / 16 * 16;
    const int total_n = P.nt * P.n_tile;
    // Widest tile (in units of 128 columns) whose accumulators fit the 512 TMEM columns.
    int max_mt = min(512 / total_n, kMaxUnits);
    if (g_head_mt > 0) max_mt = min(max_mt, g_head_mt);
    if (max_mt < 1) return GS_ERR_UNSUPPORTED;
    // Every SM gets the same number of tiles; tile widths differ by at most one unit.
    const int per_sm = (units + sms - 1) / sms;
    const int tiles_per_sm = (per_sm + max_mt - 1) / max_mt;
    const int num_tiles = min(units, sms * tiles_per_sm);
    P.num_tiles = num_tiles;
    P.unit_base = units / num_tiles;
    P.unit_rem = units % num_tiles;
    const int mt = P.unit_base + (P.unit_rem ? 1 : 0);                // widest tile
    P.acc_cols = (uint32_t)(mt * total_n);
    P.n_acc = (2 * P.acc_cols <= 512) ? 2 : 1;
    uint32_t cols = 32;
    while (cols < (uint32_t)P.n_acc * P.acc_cols) cols <<= 1;
    P.tmem_cols = cols;
    // k rows per W stage: the deepest stage that still leaves a ring of two (measured: fewer,
    // larger TMA boxes and fewer barrier round trips beat a deeper ring of small stages).
    P.h_stage_bytes = (uint32_t)total_n * 128u;
    const uint32_t fixed = 1024u /*alignment*/ + (uint32_t)kHStages * P.h_stage_bytes + 8u * 64u + 64u;
    int kw = g_head_kw;
    if (kw <= 0) {
      kw = 64;
      while (kw > 16 && fixed + 2u * ((uint32_t)mt * 2u * (uint32_t)kw * 128u) > kMaxSmem) kw >>= 1;
    }
    P.kw = kw;
    P.w_stage_bytes = (uint32_t)mt * 2u * (uint32_t)kw * 128u;
    if (fixed + 2 * P.w_stage_bytes > kMaxSmem) return GS_ERR_UNSUPPORTED;
    int stages = (int)((kMaxSmem - fixed) / P.w_stage_bytes);
    if (stages > 24) stages = 24;
    if (g_head_stages > 0 && g_head_stages < stages) stages = g_head_stages;
    if (stages < 2) return GS_ERR_UNSUPPORTED;
    P.w_stages = stages;
    P.k_blocks = (d + (int)kBlockK - 1) / (int)kBlockK;
    CUtensorMap tmapW, tmapH;
    if (!make_tmap_bf16_2d(&tmapW, W, (uint64_t)d, (uint64_t)V, (uint64_t)V, (uint32_t)kw, 64)) return GS_ERR_CUDA;
    if (!make_tmap_bf16_2d(&tmapH, H, (uint64_t)T, (uint64_t)d, (uint64_t)d, (uint32_t)P.n_tile, 64))
      return GS_ERR_CUDA;
    const size_t smem = 1024u + (size_t)stages * P.w_stage_bytes + (size_t)kHStages * P.h_stage_bytes +
                        8u * (2u * (uint32_t)stages + 2u * kHStages + 4u) + 64u;
    const int grid = min(P.num_tiles, sms);
    if (launch_ex(kernels[kw == 16 ? 0 : (kw == 32 ? 1 : 2)][P.nt - 1], dim3(grid), dim3(kTcThreads), smem, st, true, 1,
                  tmapW, tmapH, P) != cudaSuccess) {
      (void)cudaGetLastError();
      return GS_ERR_CUDA;
    }
    count_launches(1);
  }
  return GS_OK;
}

}  // namespace gs

#include "lm_head_pair.cuh"

extern "C" gs_status gs_lm_head_select(int variant) {
  if (variant < 0 || variant > 2) return GS_ERR_INVALID_ARG;
  gs::g_head_variant = variant;
  return GS_OK;
}

extern "C" gs_status gs_lm_head_configure(int m_tiles, int stages, int k_rows) {
  if (m_tiles < 0 || m_tiles > 9 || stages < 0) return GS_ERR_INVALID_ARG;
  if (k_rows != 0 && k_rows != 16 && k_rows != 32 && k_rows != 64) return GS_ERR_INVALID_ARG;
  gs::g_head_mt = m_tiles;
  gs::g_head_stages = stages;
  gs::g_head_kw = k_rows;
  return GS_OK;
}

extern "C" size_t gs_lm_head_workspace(int T, int d, int V, gs_dtype dt) {
  (void)T; (void)d; (void)V; (void)dt;
  return 256;
}

extern "C" gs_status gs_lm_head_logits(const void* H, const void* W, float* logits, int T, int d, int V,
                                       gs_dtype dt, void* ws, size_t ws_bytes, int32_t* d_status,
                                       void* stream) {
  using namespace gs;
  if (T < 0 || d < 0 || V < 0) return GS_ERR_INVALID_ARG;
  if (dt != GS_F32 && dt != GS_BF16) return GS_ERR_INVALID_ARG;
  if (T == 0 || V == 0) return GS_OK;
  if (!H || !W || !logits) return GS_ERR_INVALID_ARG;
  if (ws == nullptr || ws_bytes < gs_lm_head_workspace(T, d, V, dt)) return GS_ERR_WORKSPACE;
  if ((T + kHeadRows - 1) / kHeadRows > 65535) return GS_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dt == GS_F32) return launch_lm_head_plain<float>(H, W, logits, T, d, V, st);
  const bool tma_ok = d > 0 && (d % 8 == 0) && (V % 8 == 0) && (reinterpret_cast<uintptr_t>(H) % 16 == 0) &&
                      (reinterpret_cast<uintptr_t>(W) % 16 == 0);
  if (!tma_ok) return GS_ERR_UNSUPPORTED;
  // CTA pairs by default: a single CTA re-reads H from L2 once per 128 vocabulary columns, a pair
  // half as often, and that traffic is what limits the kernel once there are many rows.  One CTA
  // per tile remains for devices that cannot co-schedule pairs, and as a cross-check.
  if (g_head_variant != 1) {
    const gs_status r = launch_lm_head_pair(H, W, logits, T, d, V, d_status, g_head_mt, g_head_stages, st);
    if (r != GS_ERR_UNSUPPORTED || g_head_variant == 2) return r;
  }
  return launch_lm_head_tc(H, W, logits, T, d, V, d_status, st);
}

// ------------------------------------------------------------------------------------------------
// gs_lm_head_logits_stats: the same product, with the softmax statistics of every row (maximum, its
// lowest index, sum of exponentials at the given temperature, per CTA of the launch) written next to
// the logits by the epilogue.  gs_spec_accept_prestats consumes them, so the acceptance step does
// not have to read every logit once more (Sec. II-A1 and II-A2 are adjacent steps of one computation).
extern "C" size_t gs_lm_head_stats_bytes(int T) {
  if (T <= 0) return 256;
  return gs::align_up((size_t)T * (size_t)gs::sm_count() * sizeof(gs::ChunkStat), 256);
}

/* Whether taking the statistics from the LM-head epilogue is expected to beat the separate statistics
 * pass.  Up to 256 rows the accumulators are double-buffered and the extra epilogue work hides under
 * the next tile's MMAs (measured: the round gets 0.5-3 % shorter); from 257 rows on the accumulator is
 * single and every tile's epilogue, statistics included, holds up the tensor core (measured at 288 rows:
 * LM head +104 us against 32 us saved in the acceptance step). */
extern "C" int gs_lm_head_stats_pays(int T) { return (T > 0 && T <= 256) ? 1 : 0; }

extern "C" gs_status gs_lm_head_logits_stats(const void* H, const void* W, float* logits, int T, int d, int V,
                                             gs_dtype dt, float temperature, void* stats, size_t stats_bytes,
                                             int* n_chunk, void* ws, size_t ws_bytes, int32_t* d_status,
                                             void* stream) {
  using namespace gs;
  if (T < 0 || d < 0 || V < 0 || !(temperature >= 0.f)) return GS_ERR_INVALID_ARG;
  if (dt != GS_F32 && dt != GS_BF16) return GS_ERR_INVALID_ARG;
  if (!H || !W || !logits || !stats || !n_chunk) return GS_ERR_INVALID_ARG;
  if (T == 0 || V == 0) return GS_ERR_UNSUPPORTED;
  if (ws == nullptr || ws_bytes < gs_lm_head_workspace(T, d, V, dt)) return GS_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(stats) & 15u) != 0 || stats_bytes < gs_lm_head_stats_bytes(T)) return GS_ERR_WORKSPACE;
  const bool tma_ok = dt == GS_BF16 && d > 0 && (d % 8 == 0) && (V % 8 == 0) && (reinterpret_cast<uintptr_t>(H) % 16 == 0) &&
                      (reinterpret_cast<uintptr_t>(W) % 16 == 0);
  if (!tma_ok || g_head_variant == 1) return GS_ERR_UNSUPPORTED;
  const float k2 = temperature > 0.f ? 1.4426950408889634f / temperature : 0.f;
  return launch_lm_head_pair(H, W, logits, T, d, V, d_status, g_head_mt, g_head_stages,
                             static_cast<cudaStream_t>(stream), static_cast<ChunkStat*>(stats), k2, sm_count(), n_chunk);
}

// ------------------------------------------------------------------------------------------------
// gs_lm_head_logits_w4: the LM head on 4-bit weights (codes, per-group scales and zero points).
extern "C" gs_status gs_lm_head_logits_w4(const void* H, const uint32_t* qweight, const void* scales,
                                          const uint8_t* zeros, int group, float* logits, int T, int d, int V,
                                          int32_t* d_status, void* stream) {
  using namespace gs;
  if (T < 0 || d < 0 || V < 0 || group <= 0) return GS_ERR_INVALID_ARG;
  if (T == 0 || V == 0) return GS_OK;
  if (!H || !qweight || !scales || !zeros || !logits) return GS_ERR_INVALID_ARG;
  if (d == 0 || d % (int)kW4StageK != 0 || (group != (int)kW4EntryK && group % (int)kW4StageK != 0) || d % group != 0 || V % 16 != 0)
    return GS_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(H) | reinterpret_cast<uintptr_t>(qweight) | reinterpret_cast<uintptr_t>(scales) |
       reinterpret_cast<uintptr_t>(zeros)) % 16 != 0)
    return GS_ERR_UNSUPPORTED;
  return launch_lm_head_w4(H, qweight, scales, zeros, group, logits, T, d, V, d_status, static_cast<cudaStream_t>(stream));
}
