// LM head with 4-bit weights: logits = H W with W stored as 4-bit codes plus per-group scales and
// zero points (the paper's larger target is an AWQ-INT4 checkpoint, Sec. V; it gives no format, the
// one used here is defined in goodspeed.h).  The weight stream is a quarter of the bf16 one, which is
// what bounds the LM head for the usual few dozen verify positions.
//
// Same transposed product as the bf16 kernels (logits^T = W^T H^T, vocabulary on the MMA's M), but the
// A operand never exists in shared memory as bf16: the packed words arrive by TMA, dequantising warps
// (one thread per vocabulary column) expand them to bf16 pairs straight into TENSOR MEMORY, and the
// MMAs read A from there (tcgen05.mma with a tensor-memory A operand).  Shared memory carries only the
// packed words (0.5 byte per weight) and H; the expanded weights (2 bytes each) would otherwise cross
// it twice and exceed its bandwidth.
//
//   warp 0       TMA producer: per stage (64 k) H rows, the packed words, scales and zero points of the
//                tile's units
//   warp 1       allocates tensor memory, issues the MMAs (one elected lane), commits slots/stages back
//   warps 2-17   dequantise: four sets of four warps (warp w serves TMEM lane quarter w % 4).  The
//                (k block, unit) pairs of the kernel are numbered in the order the MMAs consume them and
//                dealt to the sets in turn; per pair: 8 words -> 64 weights -> 32 columns of bf16 pairs
//                in tensor memory.  The expanded weights of a whole k block (all units of the tile) form
//                one buffer that is handed to the MMA warp with ONE barrier (a hand-over per pair cost
//                the MMA warp about 480 cycles each: wait, fence, commits)
//   warps 18-21  epilogue: fp32 accumulators -> logits (thread = vocabulary column)
// Every barrier wait is time-bounded.
//
// Measured (B200, d = 5120, V = 151936, 46 rows): 207 us against 247 us for the bf16 weight, i.e. 2.1 TB/s
// of the 4-bit stream (0.32 of the HBM roofline of ITS bytes): not bandwidth-bound yet.  Per k block and
// CTA the MMA warp is busy about 630 cycles (12 MMAs 290, two commits 190, waits and fences 150) and a
// dequantising warp about 1100 per pair (shared-memory loads 180, expansion 390, barrier looks 180 each,
// tensor-memory stores 70), against a period of 1600: the chain weights -> tensor memory -> MMA -> buffer
// free is deeper than the two or three buffers that fit beside the accumulators.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"
#include <cuda_bf16.h>

namespace gs {

constexpr int kW4Sets = 4;                    // sets of four dequantising warps
constexpr int kW4Threads = 32 * (2 + 4 * kW4Sets + 4);
constexpr uint32_t kW4BlockK = 64;            // k per stage
constexpr uint32_t kW4Unit = 128;             // vocabulary columns per MMA
constexpr int kW4MaxWidth = 4;                // units per tile at most
constexpr int kW4MaxBufs = 4;                 // buffers of expanded weights (one k block of a tile each) in tensor memory
constexpr uint32_t kW4SlotCols = 32;          // 64 bf16 = 32 columns per lane
constexpr uint32_t kW4QBytes = 8u * kW4Unit * 4u;   // packed words of one unit and k block: 8 rows x 128 columns
constexpr uint32_t kW4SBytes = kW4Unit * 2u;        // scales of one unit (bf16)
constexpr uint32_t kW4ZBytes = kW4Unit;             // zero points of one unit (uint8)
constexpr uint32_t kW4MaxSmem = 232448;

struct HeadW4Params {
  float* logits;
  int32_t* d_status;
  int T, d, V, group;
  int row0;
  int n_tile;            // rows of H per MMA (T padded to 16)
  int max_width;         // units per tile at most (accumulators are sized for it)
  int n_acc;             // accumulator buffers
  int n_bufs;            // buffers of expanded weights, each max_width x 32 columns
  int stages, k_blocks;
  int num_tiles, unit_base, unit_rem;
  uint32_t h_bytes, stage_bytes, acc_cols, tmem_cols;
};

GS_DEVINL void head_w4_tile(const HeadW4Params& P, int i, int& unit0, int& width) {
  width = P.unit_base + (i < P.unit_rem ? 1 : 0);
  unit0 = i * P.unit_base + min(i, P.unit_rem);
}

// Eight 4-bit codes of one packed word to four bf16 pairs (k, k+1), k = 0, 2, 4, 6 of the word.
// The code of k offset j sits in nibble (j >> 1) + 4 (j & 1), so shifting by 4 i and masking the two
// 16-bit halves yields the codes of j = 2i (low half) and j = 2i + 1 (high half).  OR-ing 0x4300 into a
// half makes the bf16 number 128 + code (exact: bf16 has a unit step there); subtracting 128 + zero is
// exact too, and the one multiplication by the scale rounds once: bf16(scale * (code - zero)).
GS_DEVINL void w4_expand(uint32_t word, __nv_bfloat162 zz, __nv_bfloat162 ss, uint32_t (&out)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t t = ((word >> (4 * i)) & 0x000F000Fu) | 0x43004300u;
    const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(&t);
    const __nv_bfloat162 w = __hmul2(__hsub2(c, zz), ss);
    out[i] = *reinterpret_cast<const uint32_t*>(&w);
  }
}

// MMAs of one k block (64 k) for a tile WIDTH units wide.  WIDTH is a compile-time constant so that the
// loops unroll and every operand address is "a per-k-block base plus a constant": with run-time loops in
// the issuing thread the addresses live in per-thread registers and an MMA costs tens of cycles to issue.
template <int WIDTH>
GS_DEVINL void head_w4_issue(uint32_t d_acc, uint32_t a0, uint32_t b_hi, uint32_t b_lo_stage, uint32_t n_tile,
                             uint32_t idesc, uint32_t fresh) {
#pragma unroll
  for (int kk = 0; kk < (int)kW4BlockK / 16; ++kk) {
    const uint64_t bdesc = ((uint64_t)b_hi << 32) | (b_lo_stage + (uint32_t)(kk * 2));
    const uint32_t accum = (kk == 0) ? (fresh ^ 1u) : 1u;
#pragma unroll
    for (int u = 0; u < WIDTH; ++u)
      umma_bf16_ts(d_acc + (uint32_t)u * n_tile, a0 + (uint32_t)(u * (int)kW4SlotCols + kk * 8), bdesc, idesc, accum);
  }
}

__global__ void __launch_bounds__(kW4Threads, 1)
lm_head_w4_kernel(const __grid_constant__ CUtensorMap tmapQ, const __grid_constant__ CUtensorMap tmapS,
                  const __grid_constant__ CUtensorMap tmapZ, const __grid_constant__ CUtensorMap tmapH,
                  const HeadW4Params P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;            // H tiles need 1024-byte alignment
  uint8_t* sm = smem_raw + (base - raw);
  const int S = P.stages;
  const uint32_t bars = base + (uint32_t)S * P.stage_bytes;
  // barriers: full[S] (TMA bytes), empty[S] (the MMA commit behind a k block: by then the k block's
  // weights have been handed over, i.e. read out of the stage), a_full[bufs] (every dequantising warp,
  // once per k block), a_empty[bufs] (MMA commit), acc_full[2] (MMA commit), acc_empty[2] (4 epilogue warps)
  auto full_bar = [&](int s) { return bars + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bars + 8u * (uint32_t)(S + s); };
  auto afull_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * S + a); };
  auto aempty_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * S + kW4MaxBufs + a); };
  auto accfull_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * S + 2 * kW4MaxBufs + a); };
  auto accempty_bar = [&](int a) { return bars + 8u * (uint32_t)(2 * S + 2 * kW4MaxBufs + 2 + a); };
  uint8_t* tail = sm + (bars - base) + 8u * (uint32_t)(2 * S + 2 * kW4MaxBufs + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < kW4MaxBufs; ++a) { mbar_init(afull_bar(a), 4 * kW4Sets); mbar_init(aempty_bar(a), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(accfull_bar(a), 1); mbar_init(accempty_bar(a), 4); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    tma_prefetch_desc(&tmapQ); tma_prefetch_desc(&tmapS); tma_prefetch_desc(&tmapZ); tma_prefetch_desc(&tmapH);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), P.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                    // the prologue above overlaps the previous kernel's tail
  pdl_launch_dependents();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t n_bufs = (uint32_t)P.n_bufs;
  const uint32_t buf_cols = (uint32_t)P.max_width * kW4SlotCols;
  const uint32_t tmem_A = tmem_base;                                   // n_bufs x max_width x 32 columns
  const uint32_t tmem_acc = tmem_base + n_bufs * buf_cols;             // n_acc x acc_cols
  // stage layout: H | packed words of max_width units | scales | zero points
  const uint32_t q_off = P.h_bytes;
  const uint32_t s_off = q_off + (uint32_t)P.max_width * kW4QBytes;
  const uint32_t z_off = s_off + (uint32_t)P.max_width * kW4SBytes;

  if (warp == 0) {
    // ---------------- TMA producer
    uint32_t st = 0, ph = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x) {
      int unit0, width;
      head_w4_tile(P, tile, unit0, width);
      const uint32_t tx = P.h_bytes + (uint32_t)width * (kW4QBytes + kW4SBytes + kW4ZBytes);
      for (int kb = 0; kb < P.k_blocks; ++kb) {
        if (!mbar_wait_warp(empty_bar(st), ph ^ 1u, abort_flag)) { ok = false; break; }
        if (elect_one()) {
          mbar_arrive_expect_tx(full_bar(st), tx);
          const uint32_t dst = base + st * P.stage_bytes;
          // every CTA walks the k blocks in the same cyclic order but starts somewhere else, so that the
          // CTAs do not all ask L2 for the same lines of H at the same moment
          const int k0 = ((kb + (int)((blockIdx.x * 7u) % (uint32_t)P.k_blocks)) % P.k_blocks) * (int)kW4BlockK;
          const int g = k0 / P.group;
          tma_load_2d(dst, &tmapH, k0, P.row0, full_bar(st));
          for (int u = 0; u < width; ++u) {
            const int v = (unit0 + u) * (int)kW4Unit;
            tma_load_2d(dst + q_off + (uint32_t)u * kW4QBytes, &tmapQ, v, k0 / 8, full_bar(st));
            tma_load_2d(dst + s_off + (uint32_t)u * kW4SBytes, &tmapS, v, g, full_bar(st));
            tma_load_2d(dst + z_off + (uint32_t)u * kW4ZBytes, &tmapZ, v, g, full_bar(st));
          }
        }
        __syncwarp();
        if (++st == (uint32_t)S) { st = 0; ph ^= 1u; }
      }
    }
    if (!ok) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer: the whole warp walks the loops, one elected lane issues.
    // A comes from tensor memory (lane = vocabulary column, 8 columns per 16 k), B = H is K-major in
    // shared memory (rows of 128 bytes, 8-row groups 1024 bytes apart; 16 k further = +32 bytes).
    const uint32_t idesc = idesc_bf16(kW4Unit, (uint32_t)P.n_tile, false, false);
    const uint64_t b_desc0 = smem_desc_sw128(base, 16u, 1024u);
    const uint32_t b_hi = (uint32_t)(b_desc0 >> 32), b_lo0 = (uint32_t)b_desc0;
    const uint32_t stage_u = P.stage_bytes >> 4;
    const uint32_t n_tile = (uint32_t)P.n_tile;
    uint32_t st = 0, ph = 0, buf = 0, bph = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x, ++it) {
      int unit0, width;
      head_w4_tile(P, tile, unit0, width);
      const int acc = it % P.n_acc;
      const uint32_t acc_ph = (uint32_t)(it / P.n_acc) & 1u;
      if (!mbar_wait_warp(accempty_bar(acc), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t d_acc = tmem_acc + (uint32_t)acc * P.acc_cols;
      for (int kb = 0; kb < P.k_blocks && ok; ++kb) {
        if (!mbar_wait_warp(full_bar(st), ph, abort_flag)) { ok = false; break; }     // H of this k block has landed
        if (!mbar_wait_warp(afull_bar(buf), bph, abort_flag)) { ok = false; break; }  // its weights are in tensor memory
        tc_fence_after();
        if (elect_one()) {
          const uint32_t b_lo_stage = b_lo0 + st * stage_u;
          const uint32_t a0 = tmem_A + buf * buf_cols;
          const uint32_t fresh = (kb == 0) ? 1u : 0u;             // the tile's first MMAs overwrite the accumulators
          switch (width) {
            case 1: head_w4_issue<1>(d_acc, a0, b_hi, b_lo_stage, n_tile, idesc, fresh); break;
            case 2: head_w4_issue<2>(d_acc, a0, b_hi, b_lo_stage, n_tile, idesc, fresh); break;
            case 3: head_w4_issue<3>(d_acc, a0, b_hi, b_lo_stage, n_tile, idesc, fresh); break;
            default: head_w4_issue<4>(d_acc, a0, b_hi, b_lo_stage, n_tile, idesc, fresh); break;
          }
          umma_commit(aempty_bar(buf));                           // the buffer may be refilled
          umma_commit(empty_bar(st));                             // H and the packed words of the stage have been read
        }
        __syncwarp();
        if (++buf == n_bufs) { buf = 0; bph ^= 1u; }
        if (++st == (uint32_t)S) { st = 0; ph ^= 1u; }
      }
      if (ok && elect_one()) umma_commit(accfull_bar(acc));
      __syncwarp();
    }
    if (!ok) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    __syncwarp();
  } else if (warp < 2 + 4 * kW4Sets) {
    // ---------------- dequantise: thread = vocabulary column (TMEM lane); set = (warp - 2) / 4
    const int q = warp & 3;
    const uint32_t set = (uint32_t)(warp - 2) >> 2;
    const int col = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    uint32_t st = 0, ph = 0, buf = 0, bph = 0;
    uint32_t seq0 = 0;                         // number of the k block's first (k block, unit) pair
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x) {
      int unit0, width;
      head_w4_tile(P, tile, unit0, width);
      for (int kb = 0; kb < P.k_blocks && ok; ++kb) {
        const uint8_t* stage = sm + st * P.stage_bytes;
        bool mine = false;
        for (int u = 0; u < width; ++u) {
          if ((seq0 + (uint32_t)u) % kW4Sets != set) continue;        // another set's pair
          if (!mine) {
            if (!mbar_wait(full_bar(st), ph, abort_flag)) { ok = false; break; }
          }
          const uint32_t* qw = reinterpret_cast<const uint32_t*>(stage + q_off + (uint32_t)u * kW4QBytes) + col;
          const __nv_bfloat16 sc = *(reinterpret_cast<const __nv_bfloat16*>(stage + s_off + (uint32_t)u * kW4SBytes) + col);
          const uint32_t zp = *(stage + z_off + (uint32_t)u * kW4ZBytes + col);
          const uint32_t zbits = 0x4300u | (zp & 15u);
          const uint32_t zz_u = zbits | (zbits << 16);
          const __nv_bfloat162 zz = *reinterpret_cast<const __nv_bfloat162*>(&zz_u);
          const __nv_bfloat162 ss = __halves2bfloat162(sc, sc);
          uint32_t words[8];
#pragma unroll
          for (int w = 0; w < 8; ++w) words[w] = qw[w * (int)kW4Unit];
          uint32_t lo[16], hi[16];
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            uint32_t o[4];
            w4_expand(words[w], zz, ss, o);
            lo[4 * w] = o[0]; lo[4 * w + 1] = o[1]; lo[4 * w + 2] = o[2]; lo[4 * w + 3] = o[3];
            w4_expand(words[w + 4], zz, ss, o);
            hi[4 * w] = o[0]; hi[4 * w + 1] = o[1]; hi[4 * w + 2] = o[2]; hi[4 * w + 3] = o[3];
          }
          if (!mine) {
            // the buffer's previous contents have been consumed by the MMAs that read them
            if (!mbar_wait(aempty_bar(buf), bph ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after();
            mine = true;
          }
          const uint32_t dst = tmem_A + lane_addr + buf * buf_cols + (uint32_t)u * kW4SlotCols;
          tmem_st16(dst, lo);
          tmem_st16(dst + 16, hi);
        }
        if (!ok) break;
        // Every dequantising warp reports once per k block, with or without a pair of its own -- and only
        // once the buffer has been released for this k block: an arrival made earlier would be counted
        // for the k block that still owns the buffer.
        if (mine) { tmem_st_wait(); tc_fence_before(); }
        else if (!mbar_wait(aempty_bar(buf), bph ^ 1u, abort_flag)) { ok = false; break; }
        __syncwarp();
        if (lane == 0) mbar_arrive(afull_bar(buf));
        seq0 += (uint32_t)width;
        if (++buf == n_bufs) { buf = 0; bph ^= 1u; }
        if (++st == (uint32_t)S) { st = 0; ph ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue (the last four warps): TMEM lane quarter = warp % 4
    const int q = warp & 3;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x, ++it) {
      int unit0, width;
      head_w4_tile(P, tile, unit0, width);
      const int acc = it % P.n_acc;
      const uint32_t acc_ph = (uint32_t)(it / P.n_acc) & 1u;
      if (!mbar_wait(accfull_bar(acc), acc_ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      for (int m = 0; m < width; ++m) {
        const int v = (unit0 + m) * (int)kW4Unit + q * 32 + lane;
        for (int c0 = 0; c0 < P.n_tile; c0 += 16) {
          if (c0 >= P.T) break;                                // warp-uniform
          const uint32_t taddr = tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * P.acc_cols +
                                 (uint32_t)(m * P.n_tile + c0);
          uint32_t r[16];
          tmem_ld16(taddr, r);
          tmem_ld_wait();
          if (v < P.V) {
            float* out = P.logits + (size_t)(P.row0 + c0) * P.V + v;
#pragma unroll
            for (int c = 0; c < 16; ++c)
              if (c0 + c < P.T) out[(size_t)c * P.V] = __uint_as_float(r[c]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(accempty_bar(acc));
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

// ------------------------------------------------------------------ host side
// 2-D tensor map without swizzle (inner box bytes a multiple of 16, no 128-byte limit).
inline bool make_tmap_plain_2d(CUtensorMap* out, CUtensorMapDataType dt, uint32_t esize, const void* base, uint64_t rows,
                               uint64_t cols, uint32_t box_rows, uint32_t box_cols) {
  auto enc = tensor_map_encoder();
  if (enc == nullptr) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * esize};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline gs_status launch_lm_head_w4(const void* H, const uint32_t* qweight, const void* scales, const uint8_t* zeros,
                                   int group, float* logits, int T, int d, int V, int32_t* d_status, cudaStream_t st) {
  static PerDeviceOnce attr_set;
  const int slot = device_slot();
  if (attr_set.needed(slot)) {
    if (cudaFuncSetAttribute(lm_head_w4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kW4MaxSmem) != cudaSuccess)
      return GS_ERR_CUDA;
    attr_set.mark(slot);
  }
  const int sms = sm_count();
  const int units = (V + (int)kW4Unit - 1) / (int)kW4Unit;
  CUtensorMap tmQ, tmS, tmZ;
  if (!make_tmap_plain_2d(&tmQ, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, qweight, (uint64_t)d / 8, (uint64_t)V, 8, kW4Unit) ||
      !make_tmap_plain_2d(&tmS, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, scales, (uint64_t)(d / group), (uint64_t)V, 1, kW4Unit) ||
      !make_tmap_plain_2d(&tmZ, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, zeros, (uint64_t)(d / group), (uint64_t)V, 1, kW4Unit))
    return GS_ERR_CUDA;
  for (int row0 = 0; row0 < T; row0 += 256) {              // more than 256 rows: the weights are streamed once per 256
    const int rows = min(256, T - row0);
    HeadW4Params P;
    P.logits = logits; P.d_status = d_status;
    P.T = rows; P.d = d; P.V = V; P.group = group; P.row0 = row0;
    P.n_tile = (rows + 15) / 16 * 16;
    // widest tile whose accumulators fit tensor memory twice (the epilogue of a tile then overlaps the
    // next tile's MMAs) next to two buffers of expanded weights; one accumulator buffer otherwise
    int width = min(kW4MaxWidth, 512 / (2 * (P.n_tile + (int)kW4SlotCols)));
    P.n_acc = 2;
    if (width < 1) { width = 1; P.n_acc = 1; }
    const int per_cta = (units + sms - 1) / sms;
    const int tiles_per_cta = (per_cta + width - 1) / width;
    P.num_tiles = min(units, sms * tiles_per_cta);
    P.unit_base = units / P.num_tiles;
    P.unit_rem = units % P.num_tiles;
    P.max_width = P.unit_base + (P.unit_rem ? 1 : 0);
    P.acc_cols = (uint32_t)(P.max_width * P.n_tile);
    // the buffers of expanded weights take what the accumulators leave, up to three
    P.n_bufs = min(kW4MaxBufs, (512 - P.n_acc * (int)P.acc_cols) / (P.max_width * (int)kW4SlotCols));
    if (P.n_bufs < 2) return GS_ERR_UNSUPPORTED;
    P.tmem_cols = 512;
    P.h_bytes = (uint32_t)P.n_tile * 128u;
    P.stage_bytes = (uint32_t)align_up(P.h_bytes + (uint32_t)P.max_width * (kW4QBytes + kW4SBytes + kW4ZBytes), 1024);
    int stages = (int)((kW4MaxSmem - 1024u - 1024u) / P.stage_bytes);
    if (stages > 12) stages = 12;
    if (stages < 2) return GS_ERR_UNSUPPORTED;
    P.stages = stages;
    P.k_blocks = d / (int)kW4BlockK;
    const size_t smem = 1024u + (size_t)stages * P.stage_bytes + 8u * (2u * (uint32_t)stages + 2u * kW4MaxBufs + 4u) + 64u;
    CUtensorMap tmH;
    if (!make_tmap_bf16_2d(&tmH, H, (uint64_t)T, (uint64_t)d, (uint64_t)d, (uint32_t)P.n_tile, 64)) return GS_ERR_CUDA;
    const int grid = min(P.num_tiles, sms);
    if (launch_ex(lm_head_w4_kernel, dim3(grid), dim3(kW4Threads), smem, st, true, 1, tmQ, tmS, tmZ, tmH, P) != cudaSuccess) {
      (void)cudaGetLastError();
      return GS_ERR_CUDA;
    }
    count_launches(1);
  }
  return GS_OK;
}

}  // namespace gs
