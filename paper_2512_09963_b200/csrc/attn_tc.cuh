// Verify attention on the 5th-generation tensor cores (bf16, head size 128).
//
// Work item = (server, block of query positions, KV head, KV split).  The GQA group's queries of
// up to 128/G positions are packed into the 128 rows of one MMA tile (row = position * G + head in
// group), so K and V of a KV head are read once for the whole group and all positions.  Per tile
// of 64 keys:
//     S = Q K^T          tcgen05.mma  M=128, N=64,  K=128   (Q, K from shared memory, S in TMEM)
//     P = 2^(S*c - m)    four softmax warps, one thread per row: tcgen05.ld, causal mask, online
//                        max/sum, bf16 P written to shared memory in the swizzled operand layout
//     O += P V           tcgen05.mma  M=128, N=128, K=64    (V read as an MN-major operand)
// K/V tiles arrive by TMA through a 2-stage ring.  Two CTAs share an SM, so one CTA's softmax
// overlaps the other's MMAs and loads.  An item whose server needs a single KV split normalises and
// stores its rows directly; otherwise it writes an unnormalised partial (m, l, O) to the workspace
// and takes a ticket, and the last split of a (server, position block, KV head) to finish merges
// them (nobody waits).  CTAs are persistent and stride over the items.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "attn_generic.cuh"

namespace gs {

constexpr int kAtThreads = 192;          // warp 0 TMA, warp 1 MMA, warps 2-5 softmax/epilogue
constexpr int kAtTile = 64;              // keys per tile
constexpr int kAtHd = 128;
constexpr int kAtRows = 128;
constexpr int kAtStages = 2;
constexpr uint32_t kAtQBytes = kAtRows * kAtHd * 2;            // 32 KB: two halves of 64 columns
constexpr uint32_t kAtPBytes = kAtRows * kAtTile * 2;          // 16 KB
constexpr uint32_t kAtKvBytes = 2 * kAtTile * kAtHd * 2;       // K + V of one tile: 32 KB
constexpr uint32_t kAtSmem = kAtQBytes + kAtPBytes + kAtStages * kAtKvBytes + 256;
constexpr uint32_t kAtTmemCols = 256;    // S: columns 0..63, O: columns 64..191
constexpr int kAtPartStride = kAtHd + 4; // floats per partial row: O[128], m, l, 2 pad (rows stay 16-byte aligned)
constexpr float kAtLog2e = 1.4426950408889634f;

struct AttnTcParams {
  const int32_t* cu_q;
  const int32_t* cu_kv;
  float* part;              // [items][128][132]
  int* tickets;             // [groups][4] splits of a (server, position block, KV head) done, per 32-row quadrant
  __nv_bfloat16* O;
  int32_t* d_status;
  int N, Tq, total_kv, max_kv_len, Hq, Hkv, G, TB;   // TB = 128 / G query positions per item
  int tiles_per_chunk;      // KV tiles per split (upper bound; splits of a server are balanced)
  int max_items;
  float scale_log2;         // scale * log2(e)
};

struct AttnItem {
  int server, tg, split, g;        // query-position block, KV split, KV head
  int q_row0;                      // first query row (global) of the block
  int n_t;                         // positions in the block
  int kv0, Lkv, L;                 // first key row (global), keys of the server, prefix length
  int tile0, n_tiles;              // tiles [tile0, tile0 + n_tiles) of the server
  int item_base, nsplit, n_used;   // first item of the server, its splits, splits that see any key
  int group;                       // index of (server, position block, KV head) over the whole batch
  int valid;
};

// Splits of a server: its ceil(Lkv/64) tiles are spread over nsplit = ceil(tiles/tiles_per_chunk)
// splits whose sizes differ by at most one tile.
GS_DEVINL int attn_nsplit(int Lkv, int tiles_per_chunk) {
  const int tiles = (Lkv + kAtTile - 1) / kAtTile;
  return max(1, (tiles + tiles_per_chunk - 1) / tiles_per_chunk);
}

// Item `id` in the enumeration  server -> position block -> split -> KV head.
GS_DEVINL AttnItem attn_find_item(const AttnTcParams& P, int id) {
  AttnItem it;
  it.valid = 0;
  int base = 0, gbase = 0;
  for (int i = 0; i < P.N; ++i) {
    const int q0 = P.cu_q[i], n_new = P.cu_q[i + 1] - q0;
    const int k0 = P.cu_kv[i], Lkv = P.cu_kv[i + 1] - k0;
    if (n_new <= 0 || Lkv < n_new || Lkv > P.max_kv_len || k0 < 0 || k0 + Lkv > P.total_kv || q0 < 0 ||
        q0 + n_new > P.Tq)
      continue;   // flagged by the checking kernel
    const int tgs = (n_new + P.TB - 1) / P.TB;
    const int nsplit = attn_nsplit(Lkv, P.tiles_per_chunk);
    const int cnt = tgs * nsplit * P.Hkv;
    if (id < base + cnt) {
      int rem = id - base;
      it.g = rem % P.Hkv; rem /= P.Hkv;
      it.split = rem % nsplit; it.tg = rem / nsplit;
      it.server = i;
      it.item_base = base; it.nsplit = nsplit;
      it.group = gbase + it.tg * P.Hkv + it.g;
      it.q_row0 = q0 + it.tg * P.TB;
      it.n_t = min(P.TB, n_new - it.tg * P.TB);
      it.kv0 = k0; it.Lkv = Lkv; it.L = Lkv - n_new;
      const int tiles = (Lkv + kAtTile - 1) / kAtTile;
      const int tb = tiles / nsplit, tr = tiles % nsplit;
      it.tile0 = it.split * tb + min(it.split, tr);
      it.n_tiles = tb + (it.split < tr ? 1 : 0);
      // keys the block can see end at L + (last position) ; later tiles hold nothing visible
      const int last_key = it.L + it.tg * P.TB + it.n_t - 1;
      const int last_tile = last_key / kAtTile;
      if (it.tile0 + it.n_tiles - 1 > last_tile) it.n_tiles = max(0, last_tile - it.tile0 + 1);
      it.n_used = 0;
      for (int sp = 0; sp < nsplit; ++sp)
        if (sp * tb + min(sp, tr) <= last_tile) it.n_used = sp + 1;
      it.valid = 1;
      return it;
    }
    base += cnt;
    gbase += tgs * P.Hkv;
  }
  return it;
}

__global__ void __launch_bounds__(kAtThreads, 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmapQ, const __grid_constant__ CUtensorMap tmapK,
               const __grid_constant__ CUtensorMap tmapV, const AttnTcParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t q_base = base, p_base = base + kAtQBytes, kv_base = p_base + kAtPBytes;
  const uint32_t bars = kv_base + kAtStages * kAtKvBytes;
  // barriers: 0 q_full, 1 item_done, 2 s_full, 3 p_full, 4 o_full, 5.. kv_full[S], kv_empty[S]
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  uint8_t* tail = smem_raw + (bars - base) + 8 * (5 + 2 * kAtStages);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if ((base & 1023u) != 0) {                     // the operand layouts need a 1024-byte aligned base
    if (threadIdx.x == 0) set_status(P.d_status, GS_ERR_CUDA);
    return;
  }
  if (threadIdx.x == 0) {
    mbar_init(bar(0), 1); mbar_init(bar(1), 4); mbar_init(bar(2), 1); mbar_init(bar(3), 4); mbar_init(bar(4), 1);
    for (int s = 0; s < kAtStages; ++s) { mbar_init(bar(5 + s), 1); mbar_init(bar(5 + kAtStages + s), 1); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    tma_prefetch_desc(&tmapQ); tma_prefetch_desc(&tmapK); tma_prefetch_desc(&tmapV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kAtTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 64u;

  // Every role walks the same item sequence and recomputes the item from the offsets.
  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t st = 0, ph = 0;
      int n_item = 0;
      bool ok = true;
      for (int id = blockIdx.x; id < P.max_items && ok; id += gridDim.x) {
        const AttnItem it = attn_find_item(P, id);
        if (!it.valid) break;
        if (it.n_tiles == 0) continue;
        // Q may be overwritten once the previous item is completely done
        if (n_item > 0 && !mbar_wait(bar(1), (uint32_t)(n_item - 1) & 1u, abort_flag)) { ok = false; break; }
        mbar_arrive_expect_tx(bar(0), kAtQBytes);
        tma_load_3d(q_base, &tmapQ, 0, it.g * P.G, it.q_row0, bar(0));
        tma_load_3d(q_base + kAtQBytes / 2, &tmapQ, 64, it.g * P.G, it.q_row0, bar(0));
        for (int j = 0; j < it.n_tiles; ++j) {
          if (!mbar_wait(bar(5 + kAtStages + st), ph ^ 1u, abort_flag)) { ok = false; break; }
          mbar_arrive_expect_tx(bar(5 + st), kAtKvBytes);
          const uint32_t dst = kv_base + st * kAtKvBytes;
          const int key = it.kv0 + (it.tile0 + j) * kAtTile;
          const int col = it.g * kAtHd;
          tma_load_2d(dst, &tmapK, col, key, bar(5 + st));
          tma_load_2d(dst + 8192u, &tmapK, col + 64, key, bar(5 + st));
          tma_load_2d(dst + 16384u, &tmapV, col, key, bar(5 + st));
          tma_load_2d(dst + 24576u, &tmapV, col + 64, key, bar(5 + st));
          if (++st == kAtStages) { st = 0; ph ^= 1u; }
        }
        ++n_item;
      }
      if (!ok) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(128, kAtTile, false, false);     // S = Q K^T, both K-major
      const uint32_t idesc_o = idesc_bf16(128, kAtHd, false, true);        // O = P V, V is MN-major
      const uint64_t dq = smem_desc_sw128(q_base, 16u, 1024u);
      const uint64_t dp = smem_desc_sw128(p_base, 16u, 1024u);
      const uint64_t dk0 = smem_desc_sw128(kv_base, 16u, 1024u);
      const uint64_t dv0 = smem_desc_sw128(kv_base + 16384u, 8192u, 1024u); // 64-column blocks 8 KB apart
      uint32_t st = 0, ph = 0;
      int n_item = 0, n_tile_total = 0;
      bool ok = true;
      for (int id = blockIdx.x; id < P.max_items && ok; id += gridDim.x) {
        const AttnItem it = attn_find_item(P, id);
        if (!it.valid) break;
        if (it.n_tiles == 0) continue;
        if (!mbar_wait(bar(0), (uint32_t)n_item & 1u, abort_flag)) { ok = false; break; }      // Q landed
        if (n_item > 0 && !mbar_wait(bar(1), (uint32_t)(n_item - 1) & 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        for (int j = 0; j < it.n_tiles; ++j, ++n_tile_total) {
          if (!mbar_wait(bar(5 + st), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t dk = dk0 + (uint64_t)(st * (kAtKvBytes >> 4));
          const uint64_t dv = dv0 + (uint64_t)(st * (kAtKvBytes >> 4));
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {     // 128 head dims = 8 x 16; second half 16 KB (Q) / 8 KB (K) further
            const uint64_t a = dq + (uint64_t)((kk >> 2) * (16384 >> 4) + (kk & 3) * 2);
            const uint64_t b = dk + (uint64_t)((kk >> 2) * (8192 >> 4) + (kk & 3) * 2);
            umma_bf16(tmem_S, a, b, idesc_s, kk > 0 ? 1u : 0u);
          }
          umma_commit(bar(2));                                               // S ready
          if (!mbar_wait(bar(3), (uint32_t)n_tile_total & 1u, abort_flag)) { ok = false; break; }   // P ready
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {     // 64 keys = 4 x 16: P +32 bytes, V +2 groups of 8 keys
            const uint64_t a = dp + (uint64_t)(kk * 2);
            const uint64_t b = dv + (uint64_t)(kk * (2048 >> 4));
            umma_bf16(tmem_O, a, b, idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(bar(5 + kAtStages + st));                              // K/V stage free
          if (++st == kAtStages) { st = 0; ph ^= 1u; }
        }
        if (ok) umma_commit(bar(4));                                         // O complete
        ++n_item;
      }
      if (!ok) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------ softmax + epilogue: thread = row
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    int n_item = 0, n_tile_total = 0;
    bool ok = true;
    for (int id = blockIdx.x; id < P.max_items && ok; id += gridDim.x) {
      const AttnItem it = attn_find_item(P, id);
      if (!it.valid) break;
      if (it.n_tiles == 0) continue;
      const int R = it.n_t * P.G;
      const bool row_ok = r < R;
      const int t = it.tg * P.TB + r / P.G;              // position index inside the server
      const int last_visible = it.L + t;                 // keys 0..L+t
      float m_run = -INFINITY, l_run = 0.f;
      for (int j = 0; j < it.n_tiles; ++j, ++n_tile_total) {
        if (!mbar_wait(bar(2), (uint32_t)n_tile_total & 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        uint32_t sv[64];
        {
          uint32_t (*s4)[16] = reinterpret_cast<uint32_t (*)[16]>(sv);
          tmem_ld16(tmem_S + lane_addr + 0, s4[0]);
          tmem_ld16(tmem_S + lane_addr + 16, s4[1]);
          tmem_ld16(tmem_S + lane_addr + 32, s4[2]);
          tmem_ld16(tmem_S + lane_addr + 48, s4[3]);
          tmem_ld_wait();
        }
        const int key0 = (it.tile0 + j) * kAtTile;       // key index inside the server
        float tmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < 64; ++c) {
          float s = __uint_as_float(sv[c]) * P.scale_log2;
          s = (key0 + c <= last_visible) ? s : -INFINITY;
          sv[c] = __float_as_uint(s);
          tmax = fmaxf(tmax, s);
        }
        // The reference maximum only moves when the tile maximum exceeds it by more than 2^8:
        // P stays below 256, the final O/l is unchanged, and O in TMEM is rescaled rarely.
        const float m_new = (tmax > m_run + 8.f) ? tmax : m_run;
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float corr = (m_run == -INFINITY) ? 0.f : fast_exp2(m_run - m_use);
        // Rescale O when this warp has a row whose reference moved (never for the first tile, whose
        // P V product overwrites O).  All earlier MMAs have completed: S of this tile was
        // committed after them.
        const bool need = row_ok && j > 0 && (m_new > m_run);
        if (__any_sync(0xffffffffu, need)) {
          const float f = need ? corr : 1.f;
#pragma unroll
          for (int c0 = 0; c0 < kAtHd; c0 += 16) {
            uint32_t o[16];
            tmem_ld16(tmem_O + lane_addr + c0, o);
            tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 16; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
            asm volatile(
                "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                ::"r"(tmem_O + lane_addr + c0), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]),
                  "r"(o[6]), "r"(o[7]), "r"(o[8]), "r"(o[9]), "r"(o[10]), "r"(o[11]), "r"(o[12]), "r"(o[13]),
                  "r"(o[14]), "r"(o[15]) : "memory");
          }
          tmem_st_wait();
        }
        float lsum = 0.f;
        const uint32_t prow = p_base + (uint32_t)r * 128u;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {               // 8 keys = 16 bytes per chunk
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float p0 = fast_exp2(__uint_as_float(sv[ch * 8 + 2 * e]) - m_use);
            const float p1 = fast_exp2(__uint_as_float(sv[ch * 8 + 2 * e + 1]) - m_use);
            lsum += p0 + p1;
            __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
            pk[e] = *reinterpret_cast<uint32_t*>(&b);
          }
          const uint32_t addr = prow + (uint32_t)((ch ^ (r & 7)) << 4);   // 128-byte swizzle
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
        }
        l_run = l_run * corr + lsum;
        m_run = m_new;
        fence_proxy_async();          // generic-proxy writes of P -> visible to the tensor core
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(3));
      }
      if (!ok) break;
      // epilogue
      if (!mbar_wait(bar(4), (uint32_t)n_item & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      float o[kAtHd];
#pragma unroll
      for (int c0 = 0; c0 < kAtHd; c0 += 16) {
        uint32_t t16[16];
        tmem_ld16(tmem_O + lane_addr + c0, t16);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 16; ++c) o[c0 + c] = __uint_as_float(t16[c]);
      }
      // TMEM and the Q buffer are free again: the next item may start while this one is stored
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(1));
      __nv_bfloat16* orow = P.O + ((size_t)(it.q_row0 + r / P.G) * P.Hq + it.g * P.G + (r % P.G)) * kAtHd;
      if (it.n_used == 1) {
        // the only split of its group: normalise and store
        if (row_ok) {
          const float inv = 1.f / l_run;
#pragma unroll
          for (int c = 0; c < kAtHd; c += 8) {
            uint4 pk;
            __nv_bfloat162 b0 = __floats2bfloat162_rn(o[c] * inv, o[c + 1] * inv);
            __nv_bfloat162 b1 = __floats2bfloat162_rn(o[c + 2] * inv, o[c + 3] * inv);
            __nv_bfloat162 b2 = __floats2bfloat162_rn(o[c + 4] * inv, o[c + 5] * inv);
            __nv_bfloat162 b3 = __floats2bfloat162_rn(o[c + 6] * inv, o[c + 7] * inv);
            pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
            pk.z = *reinterpret_cast<uint32_t*>(&b2); pk.w = *reinterpret_cast<uint32_t*>(&b3);
            *reinterpret_cast<uint4*>(orow + c) = pk;
          }
        }
      } else {
        // unnormalised partial (O, m, l), then a ticket; the last split of the group merges
        float* out = P.part + ((size_t)id * kAtRows + r) * kAtPartStride;
        if (row_ok) {
#pragma unroll
          for (int c = 0; c < kAtHd; c += 4) *reinterpret_cast<float4*>(out + c) = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
          out[kAtHd] = m_run; out[kAtHd + 1] = l_run;
        }
        // One ticket per (group, 32-row quadrant): the warp that takes the last one finds the other
        // splits' rows of its quadrant complete (their writers fenced before taking theirs).
        __threadfence();
        __syncwarp();
        int tk = 0;
        if (lane == 0) tk = atomicAdd(&P.tickets[it.group * 4 + q], 1);
        tk = __shfl_sync(0xffffffffu, tk, 0);
        const bool last = (tk == it.n_used - 1);
        if (last && row_ok) {
          __threadfence();
          float M = -INFINITY;
          for (int sp = 0; sp < it.n_used; ++sp) {
            const float* p = P.part + ((size_t)(it.item_base + (it.tg * it.nsplit + sp) * P.Hkv + it.g) * kAtRows + r) * kAtPartStride;
            M = fmaxf(M, __ldcg(p + kAtHd));
          }
          float L = 0.f;
#pragma unroll
          for (int c = 0; c < kAtHd; ++c) o[c] = 0.f;
          for (int sp = 0; sp < it.n_used; ++sp) {
            const float* p = P.part + ((size_t)(it.item_base + (it.tg * it.nsplit + sp) * P.Hkv + it.g) * kAtRows + r) * kAtPartStride;
            const float ms = __ldcg(p + kAtHd);
            if (ms == -INFINITY) continue;
            const float w = fast_exp2(ms - M);
            L += __ldcg(p + kAtHd + 1) * w;
#pragma unroll
            for (int c = 0; c < kAtHd; c += 4) {
              const float4 v = __ldcg(reinterpret_cast<const float4*>(p + c));
              o[c] += v.x * w; o[c + 1] += v.y * w; o[c + 2] += v.z * w; o[c + 3] += v.w * w;
            }
          }
          const float inv = 1.f / L;
#pragma unroll
          for (int c = 0; c < kAtHd; c += 8) {
            uint4 pk;
            __nv_bfloat162 b0 = __floats2bfloat162_rn(o[c] * inv, o[c + 1] * inv);
            __nv_bfloat162 b1 = __floats2bfloat162_rn(o[c + 2] * inv, o[c + 3] * inv);
            __nv_bfloat162 b2 = __floats2bfloat162_rn(o[c + 4] * inv, o[c + 5] * inv);
            __nv_bfloat162 b3 = __floats2bfloat162_rn(o[c + 6] * inv, o[c + 7] * inv);
            pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
            pk.z = *reinterpret_cast<uint32_t*>(&b2); pk.w = *reinterpret_cast<uint32_t*>(&b3);
            *reinterpret_cast<uint4*>(orow + c) = pk;
          }
        }
      }
      ++n_item;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) set_status(P.d_status, GS_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kAtTmemCols);
  }
}

// Offsets the device has to vouch for: a server with fewer keys than new positions, more keys than
// max_kv_len, or offsets outside the tensors is skipped by the main kernel and flagged here.
__global__ void attn_check_kernel(const AttnTcParams P) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < P.N; i += gridDim.x * blockDim.x) {
    const int q0 = P.cu_q[i], n_new = P.cu_q[i + 1] - q0;
    const int k0 = P.cu_kv[i], Lkv = P.cu_kv[i + 1] - k0;
    if (n_new <= 0 || Lkv < n_new || Lkv > P.max_kv_len || k0 < 0 || k0 + Lkv > P.total_kv || q0 < 0 ||
        q0 + n_new > P.Tq)
      set_status(P.d_status, GS_ERR_SHAPE);
  }
}

// ------------------------------------------------------------------ host side
struct AttnTcPlan {
  int TB, tiles_per_chunk, max_items, max_groups, grid;
  size_t ticket_bytes, ws_bytes;
};

inline bool attn_tc_supported(int Hq, int Hkv, int hd, gs_dtype dt) {
  if (dt != GS_BF16 || hd != kAtHd || Hkv <= 0 || Hq % Hkv != 0) return false;
  const int G = Hq / Hkv;
  return G >= 1 && G <= 128 && (128 % G) == 0 && (Hkv * hd) % 8 == 0;
}

inline AttnTcPlan attn_tc_plan(int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv) {
  AttnTcPlan pl;
  const int G = Hq / Hkv;
  pl.TB = 128 / G;
  const int slots = 2 * sm_count();
  const int heads_total = max(1, N * Hkv);
  const int tiles_avg = max(1, (total_kv / max(1, N) + kAtTile - 1) / kAtTile);
  const int nsplit_target = max(1, slots / heads_total);
  pl.tiles_per_chunk = max(1, (tiles_avg + nsplit_target - 1) / nsplit_target);
  const int max_tiles = (max_kv_len + kAtTile - 1) / kAtTile;
  const long long blocks = (long long)N + Tq / pl.TB;      // sum over servers of ceil(n_new / TB)
  const long long items = (long long)Hkv * blocks * ((max_tiles + pl.tiles_per_chunk - 1) / pl.tiles_per_chunk);
  pl.max_items = (int)min(items, (long long)INT_MAX / 2);
  pl.grid = min(pl.max_items, slots);
  pl.max_groups = (int)min((long long)Hkv * blocks, (long long)INT_MAX / 2);
  pl.ticket_bytes = align_up((size_t)pl.max_groups * 4 * sizeof(int), 256);
  pl.ws_bytes = pl.ticket_bytes + (size_t)pl.max_items * kAtRows * kAtPartStride * sizeof(float);
  return pl;
}

inline gs_status launch_attn_tc(const void* Q, const void* K, const void* V, void* O, const int32_t* cu_q,
                                const int32_t* cu_kv, int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv,
                                float scale, void* ws, int32_t* d_status, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAtSmem) != cudaSuccess)
      return GS_ERR_CUDA;
    attr_set = true;
  }
  const AttnTcPlan pl = attn_tc_plan(N, Tq, total_kv, max_kv_len, Hq, Hkv);
  AttnTcParams P;
  P.cu_q = cu_q; P.cu_kv = cu_kv; P.d_status = d_status;
  P.tickets = static_cast<int*>(ws);
  P.part = reinterpret_cast<float*>(static_cast<char*>(ws) + pl.ticket_bytes);
  P.O = static_cast<__nv_bfloat16*>(O);
  P.N = N; P.Tq = Tq; P.total_kv = total_kv; P.max_kv_len = max_kv_len; P.Hq = Hq; P.Hkv = Hkv;
  P.G = Hq / Hkv; P.TB = pl.TB; P.tiles_per_chunk = pl.tiles_per_chunk; P.max_items = pl.max_items;
  P.scale_log2 = scale * kAtLog2e;
  auto enc = tensor_map_encoder();
  if (enc == nullptr) return GS_ERR_CUDA;
  CUtensorMap tmQ, tmK, tmV;
  {  // Q [Tq][Hq][hd]: box = 64 columns x G heads x TB positions -> rows (position, head in group)
    cuuint64_t dims[3] = {(cuuint64_t)kAtHd, (cuuint64_t)Hq, (cuuint64_t)Tq};
    cuuint64_t strides[2] = {(cuuint64_t)kAtHd * 2, (cuuint64_t)Hq * kAtHd * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)P.G, (cuuint32_t)P.TB};
    cuuint32_t es[3] = {1, 1, 1};
    if (enc(&tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(Q), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GS_ERR_CUDA;
  }
  // K, V [total_kv][Hkv*hd]: box = 64 columns x 64 keys
  if (!make_tmap_bf16_2d(&tmK, K, (uint64_t)total_kv, (uint64_t)Hkv * kAtHd, (uint64_t)Hkv * kAtHd, kAtTile, 64) ||
      !make_tmap_bf16_2d(&tmV, V, (uint64_t)total_kv, (uint64_t)Hkv * kAtHd, (uint64_t)Hkv * kAtHd, kAtTile, 64))
    return GS_ERR_CUDA;
  if (cudaMemsetAsync(P.tickets, 0, pl.ticket_bytes, st) != cudaSuccess) return GS_ERR_CUDA;
  attn_tc_kernel<<<pl.grid, kAtThreads, kAtSmem, st>>>(tmQ, tmK, tmV, P);
  if (cudaGetLastError() != cudaSuccess) return GS_ERR_CUDA;
  if (d_status != nullptr) attn_check_kernel<<<1, 128, 0, st>>>(P);
  count_launches(d_status != nullptr ? 2 : 1);
  return launch_status();
}

}  // namespace gs
