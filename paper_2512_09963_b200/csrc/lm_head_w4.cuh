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
// A unit = 128 vocabulary columns = one MMA's M; a tile = up to four neighbouring units that share the
// H rows of a stage; every CTA gets the same number of tiles, of widths that differ by at most one.
//
//   warp 0       TMA producer: per stage (128 k) the H rows and, per unit of the tile, the packed words,
//                scales and zero points
//   warps 1-3    MMA issuers (one elected lane each; warp 1 also allocates tensor memory).  Warp m issues
//                the MMAs of the units u with u % 3 == m -- different units are different accumulators, so
//                the three need no order between them -- and commits buffers / stages / accumulators
//                back.  One warp spends about 410 cycles on 8 MMAs whose tensor-pipe time is 272 (640 next
//                to sixteen busy dequantising warps): a single issuer caps the kernel.
//   warps 4-19   dequantise: two sets of eight warps.  The expanded weights pass through ENTRIES in
//                tensor memory, an entry = 64 k of the whole tile (32 columns of bf16 pairs per unit);
//                the entries are numbered in the order the MMAs consume them and alternate between the
//                sets, so that one set fills an entry while the MMAs read the other set's.  Inside a set
//                warp w serves TMEM lane quarter w % 4, and the two warps of a quarter split the entry's
//                k range (4 packed words = 32 k = 16 columns each per unit).
//   warps 20-23  epilogue: fp32 accumulators -> logits (thread = vocabulary column)
// Accumulators are double-buffered where they fit twice next to two entries (the epilogue of a tile then
// overlaps the next tile's MMAs).  Every barrier wait is time-bounded.
//
// What bounds it (B200, measured with stand-alone loops and with copies of the kernel that skip work):
//  * control: each role is one warp of dependent scalar code, about 700-900 cycles per hand-over however
//    little it does.  With 64-k stages and entries of two units the kernel took 160 us even with the
//    expansion, the MMAs and all loads but the packed words removed -- hence stages of 128 k, entries
//    of a whole tile, three MMA issuers;
//  * expansion: 8 codes cost 7 integer instructions (3 shifts, 4 mask-and-or, half rate) and 8 bf16x2
//    instructions, about 26 issue cycles per word and warp with loads and tensor-memory stores: 35-39
//    weights per clock and SM with 16 warps -- 5.26 M weights per SM in about 75 us, a little more than
//    HBM needs for the 4-bit stream (66 us);
//  * the MMAs (M128 N48 K16 from tensor memory: 34 cycles each, N/2 + 10) need 46 us.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"
#include <cuda_bf16.h>

namespace gs {

constexpr uint32_t kW4StageK = 128;           // k per stage
constexpr uint32_t kW4EntryK = 64;            // k per entry of expanded weights
constexpr uint32_t kW4Unit = 128;             // vocabulary columns per MMA
constexpr int kW4MaxWidth = 4;                // units per tile at most
constexpr int kW4MaxBufs = 4;                 // entries of expanded weights in tensor memory at most
constexpr int kW4MmaWarps = 3;
constexpr int kW4DqWarps = 16;                // two sets of eight
constexpr int kW4Threads = 32 * (1 + kW4MmaWarps + kW4DqWarps + 4);
constexpr uint32_t kW4SlotCols = 32;          // 64 bf16 = 32 columns per lane: one unit of one entry
constexpr uint32_t kW4QBytes = (kW4StageK / 8u) * kW4Unit * 4u;   // packed words of one unit and stage: 16 rows x 128 columns
constexpr uint32_t kW4SBytes = 2u * kW4Unit * 2u;   // scales of one unit and stage (bf16; two groups when group = 64)
constexpr uint32_t kW4ZBytes = 2u * kW4Unit;        // zero points of one unit and stage (uint8)
constexpr uint32_t kW4MaxSmem = 232448;

struct HeadW4Params {
  float* logits;
  int32_t* d_status;
  int T, d, V, group;
  int row0;
  int n_tile;            // rows of H per MMA (T padded to 16)
  int max_width;         // units per tile at most (stages, entries and accumulators are sized for it)
  int n_acc;             // accumulator buffers
  int n_bufs;            // entries of expanded weights, each max_width x 32 columns
  int stages, k_stages;  // ring depth; stages per pass over d
  int num_tiles, unit_base, unit_rem;
  uint32_t h_half_bytes, stage_bytes, acc_cols;
};

GS_DEVINL void head_w4_tile(const HeadW4Params& P, int i, int& unit0, int& width) {
  width = P.unit_base + (i < P.unit_rem ? 1 : 0);
  unit0 = i * P.unit_base + min(i, P.unit_rem);
}

// Four packed words (32 k of one vocabulary column) to sixteen bf16 pairs.  The code of k offset j of a
// word sits in nibble (j >> 1) + 4 (j & 1), so shifting by 4 i and masking the two 16-bit halves yields
// the codes of j = 2i (low half) and j = 2i + 1 (high half).  OR-ing 0x4300 into a half makes the bf16
// number 128 + code (exact: bf16 has a unit step there); subtracting 128 + zero is exact too, and the
// one multiplication by the scale rounds once: bf16(scale * (code - zero)).
GS_DEVINL void w4_expand4(const uint32_t (&words)[4], __nv_bfloat162 zz, __nv_bfloat162 ss, uint32_t (&out)[16]) {
#pragma unroll
  for (int w = 0; w < 4; ++w) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      // (x >> 4i) & 0x000F000F | 0x43004300 as one shift and ONE three-input logic instruction
      uint32_t t;
      asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(t) : "r"(words[w] >> (4 * i)), "r"(0x000F000Fu), "r"(0x43004300u));
      const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(&t);
      const __nv_bfloat162 x = __hmul2(__hsub2(c, zz), ss);
      out[4 * w + i] = *reinterpret_cast<const uint32_t*>(&x);
    }
  }
}

// The four MMAs (64 k) of one unit of an entry: unrolled, every operand address "a base plus a constant"
// (with run-time loops in the issuing thread the addresses live in per-thread registers and an MMA
// costs tens of cycles to issue).
GS_DEVINL void head_w4_issue_unit(uint32_t d_acc, uint32_t a0, uint32_t b_hi, uint32_t b_lo, uint32_t idesc, uint32_t fresh) {
#pragma unroll
  for (int kk = 0; kk < (int)kW4EntryK / 16; ++kk) {
    const uint64_t bdesc = ((uint64_t)b_hi << 32) | (b_lo + (uint32_t)(kk * 2));
    umma_bf16_ts(d_acc, a0 + (uint32_t)(kk * 8), bdesc, idesc, (kk == 0) ? (fresh ^ 1u) : 1u);
  }
}

// One warp's share of an entry: for each of the tile's WIDTH units the four packed words of its 32 k,
// expanded and stored to the entry's columns.  WIDTH is a compile-time constant so that all the loads
// are issued up front and the units' instruction streams interleave.  The entry's previous contents
// must have been consumed by the MMAs that read them before the first store: that wait comes after the
// first unit's expansion, which does not need the entry yet.
template <int WIDTH>
GS_DEVINL bool head_w4_expand_entry(const uint32_t* qw0, const __nv_bfloat16* sc0, const uint8_t* zp0, uint32_t dst0,
                                    uint32_t aempty, uint32_t aempty_parity, volatile int* abort_flag) {
  uint32_t words[WIDTH][4];
  __nv_bfloat162 zz[WIDTH], ss[WIDTH];
#pragma unroll
  for (int u = 0; u < WIDTH; ++u) {
#pragma unroll
    for (int w = 0; w < 4; ++w) words[u][w] = qw0[u * (int)(kW4QBytes / 4u) + w * (int)kW4Unit];
    const __nv_bfloat16 sc = sc0[u * (int)(kW4SBytes / 2u)];
    const uint32_t zbits = 0x4300u | ((uint32_t)zp0[u * (int)kW4ZBytes] & 15u);
    const uint32_t zz_u = zbits | (zbits << 16);
    zz[u] = *reinterpret_cast<const __nv_bfloat162*>(&zz_u);
    ss[u] = __halves2bfloat162(sc, sc);
  }
#pragma unroll
  for (int u = 0; u < WIDTH; ++u) {
    uint32_t x[16];
    w4_expand4(words[u], zz[u], ss[u], x);
    if (u == 0) {
      if (!mbar_wait(aempty, aempty_parity, abort_flag)) return false;
      tc_fence_after();
    }
    tmem_st16(dst0 + (uint32_t)u * kW4SlotCols, x);
  }
  return true;
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
  // barriers: full[S] (TMA bytes), empty[S] (one commit per MMA warp behind the stage's second entry: by
  // then the stage's words have been expanded and its H rows read), a_full[bufs] (the eight warps of the
  // set that filled the entry), a_empty[bufs], acc_full[2] (one commit per MMA warp), acc_empty[2] (4
  // epilogue warps)
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
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), kW4MmaWarps); }
    for (int a = 0; a < kW4MaxBufs; ++a) { mbar_init(afull_bar(a), kW4DqWarps / 2); mbar_init(aempty_bar(a), kW4MmaWarps); }
    for (int a = 0; a < 2; ++a) { mbar_init(accfull_bar(a), kW4MmaWarps); mbar_init(accempty_bar(a), 4); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    tma_prefetch_desc(&tmapQ); tma_prefetch_desc(&tmapS); tma_prefetch_desc(&tmapZ); tma_prefetch_desc(&tmapH);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
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
  const uint32_t tmem_A = tmem_base;                                   // n_bufs entries of max_width x 32 columns
  const uint32_t tmem_acc = tmem_base + n_bufs * buf_cols;             // n_acc x acc_cols
  // stage layout: H (two 64-k halves) | packed words of max_width units | scales | zero points
  const uint32_t q_off = 2u * P.h_half_bytes;
  const uint32_t s_off = q_off + (uint32_t)P.max_width * kW4QBytes;
  const uint32_t z_off = s_off + (uint32_t)P.max_width * kW4SBytes;
  const bool two_groups = (P.group == (int)kW4EntryK);                 // a stage spans two groups

  if (warp == 0) {
    // ---------------- TMA producer
    uint32_t st = 0, ph = 0;
    bool ok = true;
    const uint32_t sz_rows = two_groups ? 2u : 1u;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x) {
      int unit0, width;
      head_w4_tile(P, tile, unit0, width);
      const uint32_t tx = 2u * P.h_half_bytes + (uint32_t)width * (kW4QBytes + sz_rows * (kW4Unit * 2u + kW4Unit));
      for (int ks = 0; ks < P.k_stages; ++ks) {
        if (!mbar_wait_warp(empty_bar(st), ph ^ 1u, abort_flag)) { ok = false; break; }
        if (elect_one()) {
          mbar_arrive_expect_tx(full_bar(st), tx);
          const uint32_t dst = base + st * P.stage_bytes;
          const int k0 = ks * (int)kW4StageK;
          const int g = k0 / P.group;
          tma_load_2d(dst, &tmapH, k0, P.row0, full_bar(st));
          tma_load_2d(dst + P.h_half_bytes, &tmapH, k0 + 64, P.row0, full_bar(st));
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
    if (!ok || *abort_flag) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    __syncwarp();
  } else if (warp <= kW4MmaWarps) {
    // ---------------- MMA issuers: the whole warp walks the loops, one elected lane issues (always the
    // same lane: a commit covers the MMAs of the thread that executes it).
    // A comes from tensor memory (lane = vocabulary column, 8 columns per 16 k), B = H is K-major in
    // shared memory (rows of 128 bytes, 8-row groups 1024 bytes apart; 16 k further = +32 bytes; the
    // stage's second 64 k form a second such tile).
    const int mine = warp - 1;
    const uint32_t idesc = idesc_bf16(kW4Unit, (uint32_t)P.n_tile, false, false);
    const uint64_t b_desc0 = smem_desc_sw128(base, 16u, 1024u);
    const uint32_t b_hi = (uint32_t)(b_desc0 >> 32), b_lo0 = (uint32_t)b_desc0;
    const uint32_t stage_u = P.stage_bytes >> 4, half_u = P.h_half_bytes >> 4;
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
      const uint32_t d_tile = tmem_acc + (uint32_t)acc * P.acc_cols;
      const bool any = mine < width;                            // this warp issues MMAs for the tile at all
      for (int ks = 0; ks < P.k_stages && ok; ++ks) {
        if (!mbar_wait_warp(full_bar(st), ph, abort_flag)) { ok = false; break; }     // H of this stage has landed
#pragma unroll
        for (int eh = 0; eh < 2; ++eh) {
          if (!mbar_wait_warp(afull_bar(buf), bph, abort_flag)) { ok = false; break; }  // the entry's weights are in tensor memory
          tc_fence_after();
          if (elect_one()) {
            const uint32_t b_lo = b_lo0 + st * stage_u + (uint32_t)eh * half_u;
            const uint32_t fresh = (ks == 0 && eh == 0) ? 1u : 0u;     // the tile's first MMAs overwrite the accumulators
            const uint32_t a0 = tmem_A + buf * buf_cols;
            if (any) {
              head_w4_issue_unit(d_tile + (uint32_t)mine * n_tile, a0 + (uint32_t)mine * kW4SlotCols, b_hi, b_lo, idesc, fresh);
              if (mine + kW4MmaWarps < width)
                head_w4_issue_unit(d_tile + (uint32_t)(mine + kW4MmaWarps) * n_tile,
                                   a0 + (uint32_t)(mine + kW4MmaWarps) * kW4SlotCols, b_hi, b_lo, idesc, fresh);
              umma_commit(aempty_bar(buf));                           // this warp's share of: the entry may be refilled
              if (eh == 1) umma_commit(empty_bar(st));                // ... and of: the stage has been read
            } else {
              mbar_arrive(aempty_bar(buf));
              if (eh == 1) mbar_arrive(empty_bar(st));
            }
          }
          __syncwarp();
          if (++buf == n_bufs) { buf = 0; bph ^= 1u; }
        }
        if (++st == (uint32_t)S) { st = 0; ph ^= 1u; }
      }
      if (ok && elect_one()) {
        if (any) umma_commit(accfull_bar(acc)); else mbar_arrive(accfull_bar(acc));
      }
      __syncwarp();
    }
    if (!ok || *abort_flag) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    __syncwarp();
  } else if (warp < 1 + kW4MmaWarps + kW4DqWarps) {
    // ---------------- dequantise: thread = vocabulary column (TMEM lane)
    const int idx = (warp - (1 + kW4MmaWarps)) >> 2;          // 0..3
    const uint32_t set = (uint32_t)idx & 1u;                  // entries alternate between the sets
    const int half = idx >> 1;                                // which 32 k of an entry's 64
    const int q = warp & 3;
    const int col = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    uint32_t st = 0, ph = 0;
    uint32_t buf = set % n_bufs, bph = 0, ent = set;          // this set's next entry: number, ring slot, phase
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.num_tiles && ok; tile += gridDim.x) {
      int unit0, width;
      head_w4_tile(P, tile, unit0, width);
      for (int ks = 0; ks < P.k_stages && ok; ++ks) {
        // entry `set` of every stage is this set's (a stage holds two entries)
        const uint8_t* stage = sm + st * P.stage_bytes;
        if (!mbar_wait(full_bar(st), ph, abort_flag)) { ok = false; break; }
        const int wrow = (int)set * 8 + half * 4;               // first of this warp's four rows of packed words
        const int grow = two_groups ? (int)set : 0;             // the entry's group within the stage
        const uint32_t* qw0 = reinterpret_cast<const uint32_t*>(stage + q_off) + wrow * (int)kW4Unit + col;
        const __nv_bfloat16* sc0 = reinterpret_cast<const __nv_bfloat16*>(stage + s_off) + grow * (int)kW4Unit + col;
        const uint8_t* zp0 = stage + z_off + grow * (int)kW4Unit + col;
        const uint32_t dst0 = tmem_A + lane_addr + buf * buf_cols + (uint32_t)half * 16u;
        switch (width) {
          case 1: ok = head_w4_expand_entry<1>(qw0, sc0, zp0, dst0, aempty_bar(buf), bph ^ 1u, abort_flag); break;
          case 2: ok = head_w4_expand_entry<2>(qw0, sc0, zp0, dst0, aempty_bar(buf), bph ^ 1u, abort_flag); break;
          case 3: ok = head_w4_expand_entry<3>(qw0, sc0, zp0, dst0, aempty_bar(buf), bph ^ 1u, abort_flag); break;
          default: ok = head_w4_expand_entry<4>(qw0, sc0, zp0, dst0, aempty_bar(buf), bph ^ 1u, abort_flag); break;
        }
        if (!ok) break;
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(afull_bar(buf));
        // this set's next entry is two further on
        ent += 2u;
        buf += 2u;
        if (buf >= n_bufs) { buf -= n_bufs; bph ^= 1u; }
        if (++st == (uint32_t)S) { st = 0; ph ^= 1u; }
      }
    }
    (void)ent;
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
    tmem_dealloc(tmem_base, 512);
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

// group: 64 (two groups per stage) or a multiple of 128; d a multiple of 128.
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
  const uint32_t sz_rows = (group == (int)kW4EntryK) ? 2u : 1u;
  CUtensorMap tmQ, tmS, tmZ;
  if (!make_tmap_plain_2d(&tmQ, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, qweight, (uint64_t)d / 8, (uint64_t)V, kW4StageK / 8, kW4Unit) ||
      !make_tmap_plain_2d(&tmS, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, scales, (uint64_t)(d / group), (uint64_t)V, sz_rows, kW4Unit) ||
      !make_tmap_plain_2d(&tmZ, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, zeros, (uint64_t)(d / group), (uint64_t)V, sz_rows, kW4Unit))
    return GS_ERR_CUDA;
  for (int row0 = 0; row0 < T; row0 += 256) {              // more than 256 rows: the weights are streamed once per 256
    const int rows = min(256, T - row0);
    HeadW4Params P;
    P.logits = logits; P.d_status = d_status;
    P.T = rows; P.d = d; P.V = V; P.group = group; P.row0 = row0;
    P.n_tile = (rows + 15) / 16 * 16;
    // widest tile whose accumulators fit tensor memory twice (the epilogue of a tile then overlaps the
    // next tile's MMAs) next to two entries of expanded weights; one accumulator buffer otherwise
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
    // the entries of expanded weights take what the accumulators leave
    P.n_bufs = min(kW4MaxBufs, (512 - P.n_acc * (int)P.acc_cols) / (P.max_width * (int)kW4SlotCols));
    if (P.n_bufs < 2) return GS_ERR_UNSUPPORTED;
    P.h_half_bytes = (uint32_t)P.n_tile * 128u;
    P.stage_bytes = (uint32_t)align_up(2u * P.h_half_bytes + (uint32_t)P.max_width * (kW4QBytes + kW4SBytes + kW4ZBytes), 1024);
    int stages = (int)((kW4MaxSmem - 1024u - 1024u) / P.stage_bytes);
    if (stages > 8) stages = 8;
    if (stages < 2) return GS_ERR_UNSUPPORTED;
    P.stages = stages;
    P.k_stages = d / (int)kW4StageK;
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
