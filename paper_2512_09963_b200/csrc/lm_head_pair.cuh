// LM head on CTA pairs: logits^T = W^T H^T with M = 256 vocabulary columns per MMA, spread over
// the two SMs of a cluster (tcgen05 cta_group::2).
//
// The single-CTA kernel re-reads the whole of H from L2 for every 128 vocabulary columns an SM
// works on.  For many verify positions that traffic, not HBM and not the tensor core, is the
// limit.  A CTA pair shares B: each CTA loads half of the rows of H and its own 128 columns of W,
// and one thread of the even CTA issues MMAs that read both halves.  Per SM the H traffic is
// halved; W is still read exactly once.
//
// Roles per CTA (192 threads): warp 0 lane 0 = TMA producer for this CTA's share, warp 1 lane 0 of
// the even CTA = MMA issuer for the pair, warps 2-5 = epilogue of this CTA's 128 accumulator lanes.
// Barriers: full[s] lives in the even CTA and counts the bytes of both CTAs' loads; empty[s] and
// acc_full[a] exist in both CTAs and are signalled by a commit sent to both; acc_empty[a] lives in
// the even CTA and takes one arrival per epilogue warp of either CTA.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace gs {

constexpr int kPairThreads = 192;
constexpr uint32_t kPairBlockK = 64;        // k depth of a stage = one 128-byte swizzle row
constexpr uint32_t kPairUnit = 256;         // vocabulary columns per MMA of the pair
constexpr uint32_t kPairWUnitBytes = 2u * kPairBlockK * 128u;   // one CTA's W share of a unit: two 64-column boxes
constexpr uint32_t kPairMaxSmem = 232448;
constexpr int kPairMaxUnits = 4;            // widest tile, in units

constexpr int kPairStatRows = 512;          // most rows the epilogue keeps softmax statistics for (two MMAs along the rows)
// Shared memory of the running statistics for a launch with `nt` MMAs along the rows: per epilogue warp
// and row a maximum, its index and a sum.
constexpr uint32_t pair_stat_bytes(int nt) { return 4u * (uint32_t)(nt * 256) * 12u; }

struct HeadPairParams {
  float* logits;
  ChunkStat* stats;      // STATS kernels: [T][gridDim.x], one entry per row and CTA
  float k2;              // log2(e) / temperature (0 = greedy: maxima only)
  int32_t* d_status;
  int T, d, V;
  int row0;              // first row of H / logits this launch covers
  int nt, n_tile;        // MMAs along the rows per unit, rows per MMA (multiple of 16, at most 256)
  int n_acc;             // accumulator buffers in tensor memory
  int stages, k_blocks;
  int num_tiles;         // tiles of the vocabulary; tile i is `unit_base + (i < unit_rem)` units wide
  int unit_base, unit_rem;
  uint32_t h_bytes, stage_bytes, acc_cols, tmem_cols;
};

GS_DEVINL void head_pair_tile(const HeadPairParams& P, int i, int& unit0, int& width) {
  width = P.unit_base + (i < P.unit_rem ? 1 : 0);
  unit0 = i * P.unit_base + min(i, P.unit_rem);
}

// MMAs of one stage (64 k) for a tile WIDTH units wide; every offset is a compile-time constant
// added to the per-stage base.
template <int NT, int WIDTH>
GS_DEVINL void head_pair_issue(uint32_t d_acc, uint32_t a_hi, uint32_t a_lo_stage, uint32_t b_hi, uint32_t b_lo_stage,
                               uint32_t n_tile, uint32_t half_u, uint32_t idesc, uint32_t fresh) {
#pragma unroll
  for (int kk = 0; kk < (int)kPairBlockK / 16; ++kk) {
    const uint32_t accum = (kk == 0) ? (fresh ^ 1u) : 1u;
#pragma unroll
    for (int m = 0; m < WIDTH; ++m) {
      const uint64_t adesc = ((uint64_t)a_hi << 32) | (a_lo_stage + (uint32_t)m * (kPairWUnitBytes >> 4) + (uint32_t)(kk * 128));
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const uint64_t bdesc = ((uint64_t)b_hi << 32) | (b_lo_stage + (uint32_t)j * half_u + (uint32_t)(kk * 2));
        umma_bf16_pair(d_acc + (uint32_t)(m * NT + j) * n_tile, adesc, bdesc, idesc, accum);
      }
    }
  }
}

// Floats to unsigned keys that order the same way (0 is below every key of a real number).
GS_DEVINL uint32_t float_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
GS_DEVINL float key_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// NT = MMAs along the rows per unit; compile-time so that the issue loop unrolls completely.
// STATS: the epilogue also keeps, per row, the softmax statistics of the logits it writes (what the
// acceptance pass would otherwise obtain by reading every logit again): a warp reduces the 32
// columns it holds for 16 rows at a time, one lane per row folds the result into a running entry in
// shared memory, and at the end of the kernel the CTA's four warps are merged into one entry per row.
template <int NT, bool STATS = false>
__global__ void __launch_bounds__(kPairThreads, 1)
lm_head_pair_kernel(const __grid_constant__ CUtensorMap tmapW, const __grid_constant__ CUtensorMap tmapH,
                    const HeadPairParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;            // stages need 1024-byte alignment
  uint8_t* sm = smem_raw + (base - raw);
  const int S = P.stages;
  const uint32_t bars = base + (uint32_t)S * P.stage_bytes;
  auto full_bar = [&](int s) { return bars + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bars + 8u * (uint32_t)(S + s); };
  auto accfull_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * S + a); };
  auto accempty_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * S + 2 + a); };
  uint8_t* tail = sm + (bars - base) + 8u * (uint32_t)(2 * S + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);
  // running statistics: [4 epilogue warps][SR] maxima, indices, sums
  constexpr int SR = NT * 256;
  float* st_m = reinterpret_cast<float*>(tail + 64);
  int* st_a = reinterpret_cast<int*>(st_m + 4 * SR);
  float* st_z = reinterpret_cast<float*>(st_a + 4 * SR);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();                // 0 = even CTA (issues the MMAs)
  if (STATS) {
    for (int i = threadIdx.x; i < 4 * SR; i += kPairThreads) { st_m[i] = -INFINITY; st_a[i] = INT_MAX; st_z[i] = 0.f; }
  }
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(accfull_bar(a), 1); mbar_init(accempty_bar(a), 8); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    tma_prefetch_desc(&tmapW);
    tma_prefetch_desc(&tmapH);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), P.tmem_cols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // the partner's barriers are initialised before anything signals them
  tc_fence_after();
  pdl_wait();                    // the prologue above overlaps the previous kernel's tail
  pdl_launch_dependents();       // after the wait: what the successor reads before its own wait is complete by now
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t h_off = P.stage_bytes - P.h_bytes;        // H share sits at the end of a stage
  const int half = P.n_tile / 2;                           // rows of H per MMA that this CTA holds

  if (warp == 0) {
    // ---------------- TMA producer: this CTA's columns of W and rows of H (whole warp in the loops,
    // one elected lane issues)
    uint32_t st = 0, ph = 0;
    bool ok = true;
    for (int tile = cluster_id; tile < P.num_tiles && ok; tile += n_clusters) {
      int unit0, width;
      head_pair_tile(P, tile, unit0, width);
      const uint32_t tx = 2u * ((uint32_t)width * kPairWUnitBytes + P.h_bytes);    // both CTAs' bytes
      for (int kb = 0; kb < P.k_blocks; ++kb) {
        const int k0 = kb * (int)kPairBlockK;
        if (!mbar_wait_warp(empty_bar(st), ph ^ 1u, abort_flag)) { ok = false; break; }
        if (elect_one()) {
          const uint32_t full0 = map_to_cta(full_bar(st), 0);
          if (rank == 0) mbar_arrive_expect_tx(full_bar(st), tx);
          const uint32_t dst = base + st * P.stage_bytes;
          for (int m = 0; m < width; ++m) {
            const int v = (unit0 + m) * (int)kPairUnit + (int)rank * 128;
            tma_load_2d_pair(dst + (uint32_t)m * kPairWUnitBytes, &tmapW, v, k0, full0);
            tma_load_2d_pair(dst + (uint32_t)m * kPairWUnitBytes + kPairBlockK * 128u, &tmapW, v + 64, k0, full0);
          }
          for (int j = 0; j < NT; ++j)
            tma_load_2d_pair(dst + h_off + (uint32_t)(j * half) * 128u, &tmapH, k0,
                             P.row0 + j * P.n_tile + (int)rank * half, full0);
        }
        __syncwarp();
        if (++st == (uint32_t)S) { st = 0; ph ^= 1u; }
      }
    }
    if (!ok) {
      // Let loads that are still in flight land before the CTA goes away (bounded).
      const uint64_t t0 = global_timer_ns();
      while (global_timer_ns() - t0 < 200000ull) { }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer (even CTA only): the whole warp walks the loops, one elected lane issues
    if (rank == 0) {
      const uint32_t idesc = idesc_bf16(256u, (uint32_t)P.n_tile, /*A (W^T) MN-major*/ true, /*B (H) K-major*/ false);
      //   A (W^T, MN-major): two 64-column boxes 8 KB apart (leading offset), 8-k groups 1024 bytes
      //                      apart (stride offset); 16 k further = +2048 bytes.
      //   B (H, K-major):    rows of 128 bytes, 8-row groups 1024 bytes apart; 16 k further = +32 bytes.
      const uint64_t a_desc0 = smem_desc_sw128(base, kPairBlockK * 128u, 1024u);
      const uint64_t b_desc0 = smem_desc_sw128(base + h_off, 16u, 1024u);
      const uint32_t a_hi = (uint32_t)(a_desc0 >> 32), a_lo0 = (uint32_t)a_desc0;
      const uint32_t b_hi = (uint32_t)(b_desc0 >> 32), b_lo0 = (uint32_t)b_desc0;
      const uint32_t stage_u = P.stage_bytes >> 4;
      const uint32_t half_u = ((uint32_t)half * 128u) >> 4;
      const uint32_t n_tile = (uint32_t)P.n_tile;
      uint32_t st = 0, ph = 0;
      int it = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < P.num_tiles && ok; tile += n_clusters, ++it) {
        int unit0, width;
        head_pair_tile(P, tile, unit0, width);
        const int acc = it % P.n_acc;
        const uint32_t acc_ph = (uint32_t)(it / P.n_acc) & 1u;
        if (!mbar_wait_warp(accempty_bar(acc), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_acc = tmem_base + (uint32_t)acc * P.acc_cols;
        for (int kb = 0; kb < P.k_blocks; ++kb) {
          if (!mbar_wait_warp(full_bar(st), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          if (elect_one()) {
            const uint32_t a_lo_stage = a_lo0 + st * stage_u;
            const uint32_t b_lo_stage = b_lo0 + st * stage_u;
            const uint32_t fresh = (kb == 0) ? 1u : 0u;                 // first MMAs of the tile overwrite
            switch (width) {
              case 1: head_pair_issue<NT, 1>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_stage, n_tile, half_u, idesc, fresh); break;
              case 2: head_pair_issue<NT, 2>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_stage, n_tile, half_u, idesc, fresh); break;
              case 3: head_pair_issue<NT, 3>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_stage, n_tile, half_u, idesc, fresh); break;
              default: head_pair_issue<NT, 4>(d_acc, a_hi, a_lo_stage, b_hi, b_lo_stage, n_tile, half_u, idesc, fresh); break;
            }
            umma_commit_pair(empty_bar(st), 3);       // frees the stage in both CTAs
          }
          __syncwarp();
          if (++st == (uint32_t)S) { st = 0; ph ^= 1u; }
        }
        if (ok && elect_one()) umma_commit_pair(accfull_bar(acc), 3);
        __syncwarp();
      }
      if (!ok) {
        // MMAs may still be running: give them (bounded) time before tensor memory is freed.
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) { }
      }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue (warps 2..5): lane quadrant = warp % 4 of this CTA's 128 lanes
    const int q = warp & 3;
    int it = 0;
    bool ok = true;
    for (int tile = cluster_id; tile < P.num_tiles && ok; tile += n_clusters, ++it) {
      int unit0, width;
      head_pair_tile(P, tile, unit0, width);
      const int acc = it % P.n_acc;
      const uint32_t acc_ph = (uint32_t)(it / P.n_acc) & 1u;
      if (!mbar_wait(accfull_bar(acc), acc_ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      for (int m = 0; m < width; ++m) {
        const int v = (unit0 + m) * (int)kPairUnit + (int)rank * 128 + q * 32 + lane;
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
            if (STATS) {
              // 16 rows x this warp's 32 columns: row maxima by integer reduction on order-preserving
              // keys, lowest column at the maximum by ballot, sums of exponentials by a halving
              // exchange that leaves row c's sum in lanes 2c and 2c+1.
              const bool valid = v < P.V;
              const int c_me = (lane >> 1) & 15;
              float e[16];
              float m_me = -INFINITY;
              int a_me = INT_MAX;
              if (P.k2 > 0.f) {
                // The lane sits in the key's five lowest bits, so one integer reduction yields the row
                // maximum (to 2^-18 relative, from below: all that a reference for the exponentials
                // has to be, as long as every sum uses the same one) and its lowest column.  A vote
                // per row, which the exact index would need, costs more than everything else here.
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                  const float x = __uint_as_float(r[c]);
                  const uint32_t key = valid ? ((float_key(x) & ~31u) | (uint32_t)(31 - lane)) : 0u;
                  const uint32_t mk = __reduce_max_sync(0xffffffffu, key);
                  const float mx = (mk == 0u) ? -INFINITY : key_float(mk & ~31u);
                  e[c] = (valid && mx > -INFINITY) ? fast_exp2((x - mx) * P.k2) : 0.f;
                  if (c == c_me) { m_me = mx; a_me = mk ? (v - lane) + (31 - (int)(mk & 31u)) : INT_MAX; }
                }
              } else {
                // greedy: the exact maximum and its lowest index, no sums
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                  const float x = __uint_as_float(r[c]);
                  const uint32_t key = valid ? float_key(x) : 0u;
                  const uint32_t mk = __reduce_max_sync(0xffffffffu, key);
                  const uint32_t at = __ballot_sync(0xffffffffu, valid && key == mk);
                  e[c] = 0.f;
                  if (c == c_me) { m_me = (mk == 0u) ? -INFINITY : key_float(mk); a_me = at ? (v - lane) + (__ffs(at) - 1) : INT_MAX; }
                }
              }
#pragma unroll
              for (int h = 8; h >= 1; h >>= 1) {           // lanes with bit (2h) set keep the upper half
                const bool up = (lane & (2 * h)) != 0;
#pragma unroll
                for (int i = 0; i < h; ++i) {
                  const float send = up ? e[i] : e[i + h];
                  const float keep = up ? e[i + h] : e[i];
                  e[i] = keep + __shfl_xor_sync(0xffffffffu, send, 2 * h);
                }
              }
              const float z_me = e[0] + __shfl_xor_sync(0xffffffffu, e[0], 1);
              const int row = t_first + c_me;
              if ((lane & 1) == 0 && row < P.T) {
                const int slot = q * SR + row;
                const float m0 = st_m[slot];
                if (m_me > -INFINITY) {
                  const float mn = fmaxf(m0, m_me);
                  const float z0 = (m0 > -INFINITY) ? st_z[slot] * fast_exp2((m0 - mn) * P.k2) : 0.f;
                  st_z[slot] = z0 + z_me * fast_exp2((m_me - mn) * P.k2);
                  if (m_me > m0 || (m_me == m0 && a_me < st_a[slot])) st_a[slot] = a_me;
                  st_m[slot] = mn;
                }
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(map_to_cta(accempty_bar(acc), 0));
    }
  }
  // Nobody leaves while the partner may still signal this CTA's barriers or read its shared memory.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (threadIdx.x == 0 && *abort_flag) set_status(P.d_status, GS_ERR_TIMEOUT);
  if (STATS) {
    // one entry per row for this CTA: its four warps in order (lowest index wins ties)
    for (int row = threadIdx.x; row < P.T; row += kPairThreads) {
      float M = -INFINITY; int arg = INT_MAX;
#pragma unroll
      for (int w = 0; w < 4; ++w) argmax_merge(M, arg, st_m[w * SR + row], st_a[w * SR + row]);
      double z = 0.0;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float mw = st_m[w * SR + row];
        if (mw > -INFINITY) z += (double)st_z[w * SR + row] * (double)fast_exp2((mw - M) * P.k2);
      }
      ChunkStat cs;
      cs.m = M; cs.arg = arg; cs.z = z;
      P.stats[(size_t)(P.row0 + row) * gridDim.x + blockIdx.x] = cs;
    }
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, P.tmem_cols);
  }
}

// ------------------------------------------------------------------ host side
struct HeadPairPlan {
  HeadPairParams P;
  size_t smem;
  int clusters;
  bool ok;
};

// CTA pairs that can be resident at once (one CTA per SM; pairs sit inside one GPC).
template <typename K>
inline int head_pair_max_clusters(K kernel, size_t smem) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * sm_count());
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
  return n;
}

// Plan for `rows` rows (at most 512) starting at row0.  max_units caps the tile width (0 = widest).
inline HeadPairPlan head_pair_plan(int rows, int row0, int d, int V, int clusters_avail, int max_units, int max_stages,
                                   uint32_t reserve = 0) {
  HeadPairPlan pl;
  pl.ok = false;
  HeadPairParams& P = pl.P;
  P.T = rows; P.d = d; P.V = V; P.row0 = row0;
  P.nt = (rows + 255) / 256;
  P.n_tile = (((rows + P.nt - 1) / P.nt) + 15) / 16 * 16;
  const int total_n = P.nt * P.n_tile;
  // Widest tile whose accumulators fit tensor memory twice (the epilogue of one tile then overlaps
  // the MMAs of the next); a single buffer only when one unit needs more than half of it.
  int max_mt = min(max(256 / total_n, 1), kPairMaxUnits);
  if (max_units > 0) max_mt = min(max_mt, max_units);
  if (max_mt < 1 || clusters_avail < 1) return pl;
  P.h_bytes = (uint32_t)(P.nt * (P.n_tile / 2)) * 128u;
  // widest tile that still leaves a ring of three stages
  while (max_mt > 1 && 1024u + 3u * ((uint32_t)max_mt * kPairWUnitBytes + P.h_bytes) + 1024u + reserve > kPairMaxSmem) --max_mt;
  const int units = (V + (int)kPairUnit - 1) / (int)kPairUnit;
  const int per_cluster = (units + clusters_avail - 1) / clusters_avail;
  const int tiles_per_cluster = (per_cluster + max_mt - 1) / max_mt;
  P.num_tiles = min(units, clusters_avail * tiles_per_cluster);
  P.unit_base = units / P.num_tiles;
  P.unit_rem = units % P.num_tiles;
  const int mt = P.unit_base + (P.unit_rem ? 1 : 0);
  P.acc_cols = (uint32_t)(mt * total_n);
  P.n_acc = (2 * P.acc_cols <= 512) ? 2 : 1;
  uint32_t cols = 32;
  while (cols < (uint32_t)P.n_acc * P.acc_cols) cols <<= 1;
  P.tmem_cols = cols;
  P.stage_bytes = (uint32_t)mt * kPairWUnitBytes + P.h_bytes;
  int stages = (int)((kPairMaxSmem - 1024u - 1024u - reserve) / P.stage_bytes);
  if (stages > 16) stages = 16;
  if (max_stages > 0 && max_stages < stages) stages = max_stages;
  if (stages < 2) return pl;
  P.stages = stages;
  P.k_blocks = (d + (int)kPairBlockK - 1) / (int)kPairBlockK;
  pl.smem = 1024u + (size_t)stages * P.stage_bytes + 8u * (2u * (uint32_t)stages + 4u) + 64u + reserve;
  pl.clusters = min(P.num_tiles, clusters_avail);
  pl.ok = true;
  return pl;
}

// stats != NULL: the kernel variant that also writes per-row softmax statistics, [T][*n_chunk] entries
// (one launch only, i.e. T <= 512; otherwise GS_ERR_UNSUPPORTED and nothing is launched).
inline gs_status launch_lm_head_pair(const void* H, const void* W, float* logits, int T, int d, int V,
                                     int32_t* d_status, int max_units, int max_stages, cudaStream_t st,
                                     ChunkStat* stats = nullptr, float k2 = 0.f, int max_chunks = 0, int* n_chunk = nullptr) {
  using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const HeadPairParams);
  static const KernelFn kernels[4] = {lm_head_pair_kernel<1>, lm_head_pair_kernel<2>, lm_head_pair_kernel<1, true>,
                                      lm_head_pair_kernel<2, true>};
  if (stats != nullptr && T > kPairStatRows) return GS_ERR_UNSUPPORTED;
  static int clusters_per_device[kMaxDevices] = {};
  const int slot = device_slot();
  if (slot < 0) return GS_ERR_CUDA;
  int& clusters_avail = clusters_per_device[slot];
  if (clusters_avail <= 0) {
    for (int a = 0; a < 4; ++a) {
      if (cudaFuncSetAttribute(kernels[a], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairMaxSmem) != cudaSuccess)
        return GS_ERR_CUDA;
      if (cudaFuncSetAttribute(kernels[a], cudaFuncAttributeNonPortableClusterSizeAllowed, 0) != cudaSuccess)
        (void)cudaGetLastError();
    }
    clusters_avail = head_pair_max_clusters(kernels[1], kPairMaxSmem);
    if (clusters_avail < 1) { clusters_avail = 0; return GS_ERR_UNSUPPORTED; }
  }
  for (int row0 = 0; row0 < T; row0 += 512) {
    const int rows = min(512, T - row0);
    HeadPairPlan pl = head_pair_plan(rows, row0, d, V, clusters_avail, max_units, max_stages,
                                     stats != nullptr ? pair_stat_bytes((rows + 255) / 256) : 0u);
    if (!pl.ok) return GS_ERR_UNSUPPORTED;
    if (stats != nullptr && 2 * pl.clusters > max_chunks) return GS_ERR_UNSUPPORTED;
    pl.P.logits = logits; pl.P.d_status = d_status; pl.P.stats = stats; pl.P.k2 = k2;
    if (n_chunk != nullptr) *n_chunk = 2 * pl.clusters;
    CUtensorMap tmapW, tmapH;
    if (!make_tmap_bf16_2d(&tmapW, W, (uint64_t)d, (uint64_t)V, (uint64_t)V, kPairBlockK, 64)) return GS_ERR_CUDA;
    if (!make_tmap_bf16_2d(&tmapH, H, (uint64_t)T, (uint64_t)d, (uint64_t)d, (uint32_t)(pl.P.n_tile / 2), 64))
      return GS_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pl.clusters);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = dependent_launch_enabled() ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kernels[(stats != nullptr ? 2 : 0) + pl.P.nt - 1], tmapW, tmapH, pl.P) != cudaSuccess) {
      (void)cudaGetLastError();
      return GS_ERR_CUDA;
    }
    count_launches(1);
  }
  return GS_OK;
}

}  // namespace gs
