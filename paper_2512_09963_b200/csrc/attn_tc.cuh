// Verify attention on the 5th-generation tensor cores (bf16, head size 128).
//
// Work item = (server, block of query positions, KV head, KV split).  The GQA group's queries of
// up to 128/G positions are packed into the 128 rows of one MMA tile (row = position * G + head in
// group), so K and V of a KV head are read once for the whole group and all positions.  Per tile
// of 128 keys:
//     S = Q K^T          tcgen05.mma  M=128, N=128, K=128   (Q from tensor memory, K from shared memory)
//     P = 2^(S*c - m)    four softmax warps, one thread per row: tcgen05.ld, causal mask, online
//                        max/sum, bf16 P stored back to tensor memory (tcgen05.st)
//     O += P V           tcgen05.mma  M=128, N=128, K=128   (P from tensor memory, V an MN-major operand)
// Shared memory carries only K and V: with Q and P as shared-memory operands the tensor core's
// operand reads (Q again for every tile) plus the TMA writes exceeded the 128 B/clk of an SM.
// K/V tiles (128 keys) arrive by TMA through a 3-stage ring (one CTA per SM).  S and P are double-buffered and
// the MMA thread issues S of tile j+1 before it waits for P of tile j, so the tensor core, the
// softmax warps and the loads of later tiles overlap.  An item whose server needs a single KV split normalises and
// stores its rows directly; otherwise it writes an unnormalised partial (m, l, O) to the workspace
// and takes a ticket, and the last split of a (server, position block, KV head) to finish merges
// them (nobody waits).  Four more warps do that epilogue, one item behind the softmax warps, so
// stores, tickets and merges overlap the next item's tiles.  CTAs are persistent.  The items are
// enumerated longest cache first; a CTA's first item is the one with its own index, every further one
// is claimed from a global counter when the key producer has asked for the last tile of the one before it (longest
// processing time first, handed out on demand), by a scheduler warp that works out the descriptor once
// and passes it to the other warps through a small queue in shared memory.  The caches may be
// contiguous or pages of a pool named by a block table (a page is one tile).
//
// Small batches (fewer (server, position block, KV head) groups than half the SMs) run the CLUSTER
// instantiation instead: one thread-block cluster of 2, 4 or 8 CTAs per group, CTA k taking the k-th
// part of the group's visible tiles, exactly one item per CTA.  Each CTA leaves its unnormalised
// (O, m, l) rows in its own shared memory (the K/V ring is free by then), the cluster meets at one
// barrier, and the CTAs that hold a part share the rows out and merge them through distributed shared
// memory: no workspace, no tickets, no clearing kernel, and a set-up that finds the CTA's one item with a
// single round of loads.  Batches with more groups than that but no more than SMs run the same
// instantiation with "clusters" of one CTA (one item per CTA, nothing to merge).
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "attn_generic.cuh"
#include <type_traits>

namespace gs {

constexpr int kAtThreads = 384;          // warp 0 TMA (keys), warp 1 MMA, warps 2-5 softmax, warps 6-9 epilogue, warp 10 TMA (values), warp 11 item scheduler
constexpr int kAtTile = 128;             // keys per tile
constexpr int kAtHd = 128;
constexpr int kAtRows = 128;
constexpr int kAtStages = 3;
constexpr uint32_t kAtKvBytes = 2 * kAtTile * kAtHd * 2;       // K + V of one tile: 64 KB
constexpr int kAtMinSplitTiles = 12;     // smallest split the automatic plan makes (tiles of 128 keys)
constexpr int kAtMaxCached = 1023;       // servers whose offsets are cached in shared memory
constexpr int kAtQueue = 8;              // item descriptors in flight between the scheduler warp and the slowest role
constexpr int kAtQueueReaders = 11;      // warps that read every descriptor (all but the scheduler)
constexpr uint32_t kAtItemCacheBytes = 640;  // >= kAtQueue * sizeof(AttnItem)
constexpr uint32_t kAtBarBytes = 512;    // mbarriers and three words behind them
constexpr int kAtSortMax = 256;          // batches of at most this many servers are walked longest cache first
constexpr uint32_t kAtSortBytes = 3 * kAtSortMax * 4;
constexpr uint32_t kAtSmem = kAtStages * kAtKvBytes + kAtBarBytes + 1024 + 4 * (kAtMaxCached + 1) * 4 + kAtItemCacheBytes +
                             kAtSortBytes;     // 214.5 KB: one CTA per SM
// Tensor memory (512 columns): S two buffers 0..127 / 128..255 (P, as bf16 pairs, overwrites the first
// 64 columns of its S buffer once the thread has read its scores), O 256..383, Q (bf16 pairs) 384..447.
// Q and P are A operands read from tensor memory, so shared memory carries only K and V.
constexpr uint32_t kAtTmemCols = 512;
constexpr uint32_t kAtColS = 0, kAtColO = 256, kAtColQ = 384;
constexpr uint32_t kAtHalfBytes = kAtTile * 128u;              // one 64-column half of a K or V tile
constexpr int kAtPartStride = kAtHd + 4; // floats per partial row: O[128], m, l, 2 pad (rows stay 16-byte aligned)
constexpr float kAtLog2e = 1.4426950408889634f;

struct AttnTcParams {
  const int32_t* cu_q;
  const int32_t* cu_kv;
  const int32_t* block_table;   // paged caches: [N][max_pages] page of every 128-key tile of a server; NULL = contiguous
  int max_pages, n_pages;
  float* part;              // [items][128][132]
  int* tickets;             // [groups] splits of a (server, position block, KV head) that are done
  int* next_item;           // items claimed beyond every CTA's first (persistent kernel)
  __nv_bfloat16* O;
  const __nv_bfloat16* Q;
  int32_t* d_status;
  int N, Tq, total_kv, max_kv_len, Hq, Hkv, G, TB;   // TB = 128 / G query positions per item
  int tiles_per_chunk;      // KV tiles per split (upper bound; splits of a server are balanced)
  int min_split_tiles;      // a server is split only into parts of at least this many tiles
  int max_items;
  int cluster;              // CLUSTER kernel: CTAs per group (2, 4 or 8); 0 for the persistent kernel
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
  int id;                          // index in the enumeration (persistent kernel: names the partial rows' place)
  int valid;
};

// Splits of a server: its ceil(Lkv/128) tiles are spread over nsplit = ceil(tiles/tiles_per_chunk)
// splits whose sizes differ by at most one tile -- but never so many that a split falls below
// min_split_tiles: a split costs a partial result, a ticket and a merge (several microseconds of
// dependent round trips), which a handful of tiles at about 1.3 us each does not buy back.
GS_DEVINL int attn_nsplit(int Lkv, int tiles_per_chunk, int min_split_tiles) {
  const int tiles = (Lkv + kAtTile - 1) / kAtTile;
  return max(1, min((tiles + tiles_per_chunk - 1) / tiles_per_chunk, tiles / min_split_tiles));
}

// Items of one server (0 when its offsets are inconsistent: such servers are skipped everywhere
// and flagged by CTA 0) and its (position block, KV head) groups.
GS_DEVINL bool attn_server_ok(const AttnTcParams& P, int q0, int n_new, int k0, int Lkv) {
  if (P.block_table != nullptr && Lkv > P.max_pages * kAtTile) return false;
  return !(n_new <= 0 || Lkv < n_new || Lkv > P.max_kv_len || k0 < 0 || k0 + Lkv > P.total_kv || q0 < 0 ||
           q0 + n_new > P.Tq);
}
GS_DEVINL void attn_server_counts(const AttnTcParams& P, int q0, int n_new, int k0, int Lkv, int& items, int& groups) {
  items = 0; groups = 0;
  if (!attn_server_ok(P, q0, n_new, k0, Lkv)) return;
  const int tgs = (n_new + P.TB - 1) / P.TB;
  groups = tgs * P.Hkv;
  items = groups * attn_nsplit(Lkv, P.tiles_per_chunk, P.min_split_tiles);
}

// Item `id` of server i, whose first item is `base` and first group `gbase`, in the enumeration
// position block -> split -> KV head.
GS_DEVINL AttnItem attn_item_of_server(const AttnTcParams& P, int i, int q0, int n_new, int k0, int Lkv, int base,
                                       int gbase, int id) {
  AttnItem it;
  const int nsplit = attn_nsplit(Lkv, P.tiles_per_chunk, P.min_split_tiles);
  int rem = id - base;
  it.g = rem % P.Hkv; rem /= P.Hkv;
  it.split = rem % nsplit; it.tg = rem / nsplit;
  it.server = i; it.id = id;
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

// Item `id` in the enumeration  server -> position block -> split -> KV head, the servers taken in
// the order s_order gives (longest cache first; NULL = as they come).  With the prefix counts of that
// walk in shared memory (s_base[0..N], s_gbase[0..N-1]) the server is found by bisection; without
// them (more servers than the cache holds) by a walk over the offsets.
GS_DEVINL AttnItem attn_find_item(const AttnTcParams& P, const int32_t* cu_q, const int32_t* cu_kv,
                                  const int32_t* s_base, const int32_t* s_gbase, const int32_t* s_order, int id) {
  AttnItem it;
  it.valid = 0;
  if (s_base != nullptr) {
    if (id >= s_base[P.N]) return it;
    int lo = 0, hi = P.N;                      // the largest i with s_base[i] <= id
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_base[mid] <= id) lo = mid; else hi = mid;
    }
    const int i = (s_order != nullptr) ? s_order[lo] : lo;          // position in the walk -> server
    const int q0 = cu_q[i], k0 = cu_kv[i];
    return attn_item_of_server(P, i, q0, cu_q[i + 1] - q0, k0, cu_kv[i + 1] - k0, s_base[lo], s_gbase[lo], id);
  }
  int base = 0, gbase = 0;
  for (int i = 0; i < P.N; ++i) {
    const int q0 = cu_q[i], n_new = cu_q[i + 1] - q0;
    const int k0 = cu_kv[i], Lkv = cu_kv[i + 1] - k0;
    int cnt, grp;
    attn_server_counts(P, q0, n_new, k0, Lkv, cnt, grp);
    if (id < base + cnt) return attn_item_of_server(P, i, q0, n_new, k0, Lkv, base, gbase, id);
    base += cnt;
    gbase += grp;
  }
  return it;
}

static_assert(sizeof(AttnItem) * kAtQueue <= kAtItemCacheBytes, "item queue too small");

// CLUSTER kernel: part `split` of group `grp` of server i, whose first group is `gbase` (groups are
// numbered server -> position block -> KV head).  Only the tiles that hold a key the block can see are
// shared out, as evenly as possible; the first n_used = min(cluster, visible tiles) parts get one.
GS_DEVINL AttnItem attn_cluster_item(const AttnTcParams& P, int i, int q0, int n_new, int k0, int Lkv, int gbase,
                                     int grp, int split) {
  AttnItem it;
  const int rem = grp - gbase;
  it.g = rem % P.Hkv; it.tg = rem / P.Hkv; it.split = split; it.server = i;
  it.item_base = 0; it.nsplit = P.cluster; it.group = grp; it.id = 0;
  it.q_row0 = q0 + it.tg * P.TB;
  it.n_t = min(P.TB, n_new - it.tg * P.TB);
  it.kv0 = k0; it.Lkv = Lkv; it.L = Lkv - n_new;
  const int last_key = it.L + it.tg * P.TB + it.n_t - 1;
  const int vis = last_key / kAtTile + 1;
  const int tb = vis / P.cluster, tr = vis % P.cluster;
  it.tile0 = split * tb + min(split, tr);
  it.n_tiles = tb + (split < tr ? 1 : 0);
  it.n_used = min(P.cluster, vis);
  it.valid = 1;
  return it;
}

// Whole warp: finds the server that owns group `grp` (32 servers per step: one round of loads, a
// shuffle scan of the servers' group counts, a vote) and writes the CTA's item.
GS_DEVINL void attn_cluster_find_item(const AttnTcParams& P, int grp, int split, int lane, AttnItem* out) {
  int carry = 0;
  bool found = false;
  for (int c = 0; c < P.N && !found; c += 32) {
    const int i = c + lane;
    int q0 = 0, n_new = 0, k0 = 0, Lkv = 0, groups = 0;
    if (i < P.N) {
      q0 = P.cu_q[i]; k0 = P.cu_kv[i];
      n_new = P.cu_q[i + 1] - q0; Lkv = P.cu_kv[i + 1] - k0;
      if (attn_server_ok(P, q0, n_new, k0, Lkv)) groups = ((n_new + P.TB - 1) / P.TB) * P.Hkv;
    }
    int inc = groups;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += a;
    }
    const int excl = carry + inc - groups;
    const bool mine = groups > 0 && grp >= excl && grp < excl + groups;
    if (__ballot_sync(0xffffffffu, mine) != 0u) {
      if (mine) *out = attn_cluster_item(P, i, q0, n_new, k0, Lkv, excl, grp, split);
      found = true;
    }
    carry += __shfl_sync(0xffffffffu, inc, 31);
  }
  if (!found && lane == 0) out->valid = 0;
}

GS_DEVINL float4 ld_cluster_f32x4(uint32_t cluster_addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr) : "memory");
  return v;
}
GS_DEVINL float2 ld_cluster_f32x2(uint32_t cluster_addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(cluster_addr) : "memory");
  return v;
}

// CLUSTER kernel, after the first cluster barrier: this CTA's share of the merge of a group's parts.
// The n_used CTAs that hold a part share the rows out: CTA k merges rows k, k + n_used, ...; its warp w
// the w-th, (w + 10)-th ... of those; lane c4 owns 4 of the 128 head dims, so a row of one part is one
// 512-byte access to that CTA's shared memory.  Every warp fetches all its rows (at most UN), arrives
// at the second cluster barrier (its reads of the peers are done), then does the arithmetic and the
// stores.  (Inlined on purpose: as a real call its stack frame lives in local memory, which is cold,
// and the merge took 8 us longer.)
template <int KMAX, int UN>
GS_DEVINL void attn_cluster_merge(int R, int n_used, int G, int Hq, __nv_bfloat16* O, int q_row0, int g,
                                                int rank, int warp, int lane, const uint8_t* smem_raw) {
  constexpr int kWarps = kAtThreads / 32;
  const uint32_t stage = smem_u32(smem_raw);
  float4 v[UN][KMAX];
  float2 ml[UN][KMAX];
#pragma unroll
  for (int u = 0; u < UN; ++u) {
    const int row = rank + n_used * (warp + kWarps * u);
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      v[u][k] = make_float4(0.f, 0.f, 0.f, 0.f);
      ml[u][k] = make_float2(-INFINITY, 0.f);
      if (row < R && k < n_used) {          // warp-uniform
        if (k == rank) {                       // this CTA's own part: plain shared-memory loads
          const float* mine = reinterpret_cast<const float*>(smem_raw) + (size_t)row * kAtPartStride;
          v[u][k] = *reinterpret_cast<const float4*>(mine + lane * 4);
          ml[u][k] = *reinterpret_cast<const float2*>(mine + kAtHd);
        } else {
          const uint32_t a = map_to_cta(stage, (uint32_t)k) + (uint32_t)row * (kAtPartStride * 4u);
          v[u][k] = ld_cluster_f32x4(a + (uint32_t)lane * 16u);
          ml[u][k] = ld_cluster_f32x2(a + kAtHd * 4u);
        }
      }
    }
  }
  cluster_arrive_release();
#pragma unroll
  for (int u = 0; u < UN; ++u) {
    const int row = rank + n_used * (warp + kWarps * u);
    if (row < R) {
      float M = -INFINITY;
#pragma unroll
      for (int k = 0; k < KMAX; ++k) if (k < n_used) M = fmaxf(M, ml[u][k].x);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float L = 0.f;
#pragma unroll
      for (int k = 0; k < KMAX; ++k) {
        if (k < n_used && ml[u][k].x > -INFINITY) {
          const float wk = fast_exp2(ml[u][k].x - M);
          L += ml[u][k].y * wk;
          acc.x += v[u][k].x * wk; acc.y += v[u][k].y * wk; acc.z += v[u][k].z * wk; acc.w += v[u][k].w * wk;
        }
      }
      const float inv = 1.f / L;
      __nv_bfloat162 b0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
      __nv_bfloat162 b1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
      __nv_bfloat16* orow2 = O + ((size_t)(q_row0 + row / G) * Hq + g * G + (row % G)) * kAtHd;
      *reinterpret_cast<uint2*>(orow2 + lane * 4) = pk;
    }
  }
}

// 2^x on the FMA pipe (x <= 127): floor by the 1.5*2^23 trick, a cubic for 2^f on [0,1] (relative
// error 9e-5, far below bf16 resolution) and an integer add to the exponent.  One softmax thread
// needs 128 exponentials per tile and the special-function unit delivers 4 per clock per SM
// quarter, so every fourth exponential is evaluated here instead.
GS_DEVINL float poly_exp2(float x) {
  x = fmaxf(x, -126.f);
  const float t = (x - 0.5f) + 12582912.f;
  const float n = t - 12582912.f;                       // floor(x) (x itself on exact integers + 0.5 ties)
  const float f = x - n;
  const float p = fmaf(f, fmaf(f, fmaf(f, 0.07706156f, 0.22765097f), 0.69511545f), 1.0f);
  const int e = __float_as_int(t) - 0x4B400000;         // floor(x) as an integer
  return __int_as_float(__float_as_int(p) + (e << 23));
}

// Two non-negative floats to a packed bf16 pair (round half up on the dropped bits) with integer
// ops only: the conversion instruction shares the special-function pipe with the exponentials.
GS_DEVINL uint32_t pack_bf16_pos(float lo, float hi) {
  return __byte_perm(__float_as_uint(lo) + 0x8000u, __float_as_uint(hi) + 0x8000u, 0x7632);
}

// Clears the tickets and the item counter.  The attention kernel is launched behind it as its programmatic dependent: it
// starts at once (this kernel only began after everything earlier on the stream had finished, so the
// inputs are complete) and waits for this grid only where it first touches a ticket.
__global__ void attn_zero_kernel(int* p, int n) {
  pdl_launch_dependents();
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) p[i] = 0;
}

template <bool CLUSTER>
__global__ void __launch_bounds__(kAtThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmapK, const __grid_constant__ CUtensorMap tmapV,
               const AttnTcParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t kv_base = base;
  const uint32_t bars = kv_base + kAtStages * kAtKvBytes;
  // barriers: 0 q_full, 1 item_done, 2-3 s_full[2], 4-5 p_full[2], 6 o_full, 7 pv_done,
  //           8.. kv_full[S], kv_empty[S], then epi_a, epi_b (the 128 epilogue threads meet twice
  //           per item that took a ticket), stats_full (row maxima and sums of an item handed from
  //           the softmax warps to the epilogue warps), o_drained (O of an item read out of tensor
  //           memory: the next item's first product may overwrite it)
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  constexpr int kSFull = 2, kPFull = 4, kOFull = 6, kPvDone = 7, kKvFull = 8, kKvEmpty = 8 + kAtStages;
  constexpr int kEpiA = 8 + 2 * kAtStages, kEpiB = kEpiA + 1, kStatsFull = kEpiA + 2, kODrained = kEpiA + 3;
  // kv_full[s] / kv_empty[s] belong to the K half of a stage only; the V half has barriers of its own
  // (v_full[S], v_empty[S]) and a producer warp of its own.  A tile's keys are needed one softmax before
  // its values and are done with as soon as its scores exist, so the K halves turn over faster than the V
  // halves: more bytes in flight per SM than with whole stages that wait for the tile's second product.
  constexpr int kVFull = kODrained + 1, kVEmpty = kVFull + kAtStages;
  // q_full[Q] / q_empty[Q]: the item queue's slots (written by the scheduler warp, read by every other
  // warp); q_taken: the key producer has started on an item, the scheduler may claim the next
  constexpr int kQFull = kVEmpty + kAtStages, kQEmpty = kQFull + kAtQueue, kQTaken = kQEmpty + kAtQueue;
  static_assert(8 * (kQTaken + 1) + 12 <= (int)kAtBarBytes, "barrier area too small");
  uint8_t* tail = smem_raw + (bars - base) + 8 * (kQTaken + 1);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);
  volatile int* s_last = reinterpret_cast<volatile int*>(tail + 8);
  // The offsets are read by every role for every item: keep them in shared memory when they fit.
  float* s_ml = reinterpret_cast<float*>(smem_raw + kAtStages * kAtKvBytes + kAtBarBytes);     // [128][2] row maximum, row sum
  int32_t* s_cu = reinterpret_cast<int32_t*>(smem_raw + kAtStages * kAtKvBytes + kAtBarBytes + 1024);
  const bool cached = !CLUSTER && P.N <= kAtMaxCached;
  const int32_t* cu_q = cached ? s_cu : P.cu_q;
  const int32_t* cu_kv = cached ? s_cu + (P.N + 1) : P.cu_kv;
  // first item and first group of every server (exclusive prefix sums; entry N = number of items)
  int32_t* s_base_w = s_cu + 2 * (kAtMaxCached + 1);
  int32_t* s_gbase_w = s_base_w + (kAtMaxCached + 1);
  const int32_t* s_base = cached ? s_base_w : nullptr;
  const int32_t* s_gbase = cached ? s_gbase_w : nullptr;
  // walk order (position -> server) and, while it is being built, the counts by server
  int32_t* s_order_w = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(s_gbase_w + (kAtMaxCached + 1)) + kAtItemCacheBytes);
  int32_t* s_tmp_cnt = s_order_w + kAtSortMax;
  int32_t* s_tmp_grp = s_tmp_cnt + kAtSortMax;
  const bool sorted = !CLUSTER && P.N <= kAtSortMax;
  const int32_t* s_order = sorted ? s_order_w : nullptr;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // The next kernel on the stream may set itself up on idle SMs right away (it still waits for this
  // grid to finish before it touches global memory).
  pdl_launch_dependents();
  const bool misaligned = (base & 1023u) != 0;   // the operand layouts need a 1024-byte aligned base
  if (misaligned) {
    if (threadIdx.x == 0) set_status(P.d_status, GS_ERR_CUDA);
    if (!CLUSTER) return;                        // a cluster's CTAs all go on to the cluster barriers, without an item
  }
  if (threadIdx.x == 0) {
    mbar_init(bar(0), 4); mbar_init(bar(1), 4);
    mbar_init(bar(kSFull), 1); mbar_init(bar(kSFull + 1), 1);
    mbar_init(bar(kPFull), 4); mbar_init(bar(kPFull + 1), 4);
    mbar_init(bar(kOFull), 1); mbar_init(bar(kPvDone), 1);
    for (int s = 0; s < kAtStages; ++s) {
      mbar_init(bar(kKvFull + s), 1); mbar_init(bar(kKvEmpty + s), 1);
      mbar_init(bar(kVFull + s), 1); mbar_init(bar(kVEmpty + s), 1);
    }
    mbar_init(bar(kEpiA), 128); mbar_init(bar(kEpiB), 128);
    mbar_init(bar(kStatsFull), 4); mbar_init(bar(kODrained), 4);
    for (int s = 0; s < kAtQueue; ++s) { mbar_init(bar(kQFull + s), 1); mbar_init(bar(kQEmpty + s), kAtQueueReaders); }
    mbar_init(bar(kQTaken), 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    tma_prefetch_desc(&tmapK); tma_prefetch_desc(&tmapV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kAtTmemCols);
    tmem_relinquish();
  }
  // The barrier and tensor-memory set-up above overlaps the tail of whatever runs before this kernel
  // on the stream; global memory is touched only after that work has finished.
  pdl_wait();
  AttnItem* s_items = reinterpret_cast<AttnItem*>(s_gbase_w + (kAtMaxCached + 1));
  // K (or V) of tile j of an item into ring stage st (one elected lane of the producer warp).
  auto tile_row = [&](const AttnItem& it, int j) -> int {
    // contiguous caches: the server's rows follow one another; paged caches: tile = page
    return (P.block_table == nullptr) ? it.kv0 + (it.tile0 + j) * kAtTile
                                      : P.block_table[(size_t)it.server * P.max_pages + it.tile0 + j] * kAtTile;
  };
  auto issue_k = [&](const AttnItem& it, int j, uint32_t st) {
    mbar_arrive_expect_tx(bar(kKvFull + st), kAtKvBytes / 2);
    const uint32_t dst = kv_base + st * kAtKvBytes;
    const int key = tile_row(it, j), col = it.g * kAtHd;
    tma_load_2d(dst, &tmapK, col, key, bar(kKvFull + st));
    tma_load_2d(dst + kAtHalfBytes, &tmapK, col + 64, key, bar(kKvFull + st));
  };
  auto issue_v = [&](const AttnItem& it, int j, uint32_t st) {
    mbar_arrive_expect_tx(bar(kVFull + st), kAtKvBytes / 2);
    const uint32_t dst = kv_base + st * kAtKvBytes + 2 * kAtHalfBytes;
    const int key = tile_row(it, j), col = it.g * kAtHd;
    tma_load_2d(dst, &tmapV, col, key, bar(kVFull + st));
    tma_load_2d(dst + kAtHalfBytes, &tmapV, col + 64, key, bar(kVFull + st));
  };
  int pre_issued = 0;          // CLUSTER: 1 once the producer warp has started the first tile's loads, before the CTA's first barrier
  if (CLUSTER && warp == 0) {
    // Exactly one item per CTA: part (blockIdx.x % cluster) of group (blockIdx.x / cluster), found with
    // one round of loads.  The same warp initialised the barriers (its lane 0, above), so it starts the
    // loads of the first tile's keys at once, without waiting for the other warps (only the first:
    // measured, asking for three tiles at once delays the one the first scores wait for).
    __syncwarp();
    if (misaligned) { if (lane == 0) s_items[0].valid = 0; }
    else attn_cluster_find_item(P, (int)blockIdx.x / P.cluster, (int)blockIdx.x % P.cluster, lane, &s_items[0]);
    __syncwarp();
    const AttnItem it = s_items[0];
    if (it.valid) {
      pre_issued = min(it.n_tiles, 1);
      if (elect_one())
        for (int j = 0; j < pre_issued; ++j) issue_k(it, j, (uint32_t)j);
      __syncwarp();
    }
  }
  if (warp != 1 && cached) {
    const int t = (warp == 0) ? (int)threadIdx.x : (int)threadIdx.x - 32;      // every thread but the allocating warp's
    for (int i = t; i <= P.N; i += kAtThreads - 32) {
      const int q0 = P.cu_q[i], k0 = P.cu_kv[i];
      s_cu[i] = q0; s_cu[P.N + 1 + i] = k0;
      int cnt = 0, grp = 0;
      if (i < P.N) attn_server_counts(P, q0, P.cu_q[i + 1] - q0, k0, P.cu_kv[i + 1] - k0, cnt, grp);
      if (sorted) { if (i < P.N) { s_tmp_cnt[i] = cnt; s_tmp_grp[i] = grp; } }
      else { s_base_w[i] = cnt; s_gbase_w[i] = grp; }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (CLUSTER && !misaligned && !s_items[0].valid) {
    // A group beyond the batch's real number (the grid is sized for a bound): the same holds for every
    // CTA of this cluster, so all of them leave here, before any cluster barrier.  Such clusters are the
    // last in launch order; the sooner they are gone, the sooner the grid is.
    if (warp == 1) tmem_dealloc(*tmem_slot, kAtTmemCols);
    return;
  }
  if (sorted) {
    // Longest cache first: the CTAs' first items are then the largest ones and the short ones fill
    // in behind them, which evens out a ragged batch (cfg3: 79 -> 64 us).  Rank = servers with a
    // longer cache (or an equal one and a lower index); the counts move to their place in the walk.
    for (int i = threadIdx.x; i < P.N; i += kAtThreads) {
      const int Li = s_cu[P.N + 2 + i] - s_cu[P.N + 1 + i];
      int rank = 0;
      for (int j = 0; j < P.N; ++j) {
        const int Lj = s_cu[P.N + 2 + j] - s_cu[P.N + 1 + j];
        rank += (Lj > Li || (Lj == Li && j < i)) ? 1 : 0;
      }
      s_order_w[rank] = i;
      s_base_w[rank] = s_tmp_cnt[i]; s_gbase_w[rank] = s_tmp_grp[i];
    }
    __syncthreads();
  }
  if (cached && warp == 11) {
    // counts -> exclusive prefix sums, 32 servers per step (the scheduler warp: it goes straight on to
    // the CTA's first item)
    int carry = 0, gcarry = 0;
    for (int c = 0; c <= P.N; c += 32) {
      const int i = c + lane;
      const int v = (i < P.N) ? s_base_w[i] : 0, gv = (i < P.N) ? s_gbase_w[i] : 0;
      int inc = v, ginc = gv;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, inc, d), b = __shfl_up_sync(0xffffffffu, ginc, d);
        if (lane >= d) { inc += a; ginc += b; }
      }
      if (i <= P.N) { s_base_w[i] = carry + inc - v; s_gbase_w[i] = gcarry + ginc - gv; }
      carry += __shfl_sync(0xffffffffu, inc, 31);
      gcarry += __shfl_sync(0xffffffffu, ginc, 31);
    }
  }
  // One item descriptor, worked out by one lane and published in slot k mod kAtQueue (scheduler warp).
  auto publish_item = [&](int k, long long id) -> int {
    int valid = 0;
    if (lane == 0) {
      AttnItem it;
      it.valid = 0;
      if (id < P.max_items) it = attn_find_item(P, cu_q, cu_kv, s_base, s_gbase, s_order, (int)id);
      s_items[k % kAtQueue] = it;
      valid = it.valid;
      mbar_arrive(bar(kQFull + k % kAtQueue));
    }
    return __shfl_sync(0xffffffffu, valid, 0);
  };
  int sched_live = 0;
  if (!CLUSTER) {
    // The CTA's first item is the one with its own index.  It is published before the barrier the other
    // warps sleep at: warps that polled the queue instead would take issue slots from the lane that works
    // the descriptor out (measured: 2 us later first loads).
    if (warp == 11) {
      __syncwarp();
      sched_live = publish_item(0, (long long)blockIdx.x);
    }
    __syncthreads();
  }
  // The k-th item of this CTA (whole warp; false: there is none, or a wait ran out).  CLUSTER: the one
  // item found above.  Otherwise the scheduler warp's k-th descriptor, from slot k mod kAtQueue of the
  // queue; the slot goes back to the scheduler once every warp has read it.  The descriptor that ends
  // the sequence (valid = 0) is read by everybody as well.
  auto take_item = [&](int k, AttnItem& it) -> bool {
    if (CLUSTER) {
      if (k > 0) return false;
      it = s_items[0];
      return it.valid != 0;
    }
    const int slot = k % kAtQueue;
    if (!mbar_wait_warp(bar(kQFull + slot), (uint32_t)(k / kAtQueue) & 1u, abort_flag)) return false;
    it = s_items[slot];
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(kQEmpty + slot));
    return it.valid != 0;
  };
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_S = tmem_base + kAtColS, tmem_O = tmem_base + kAtColO;     // S buffer b at tmem_S + 128 b
  const uint32_t tmem_Q = tmem_base + kAtColQ;

  // Every role walks the same item sequence and recomputes the item from the offsets.
  if (blockIdx.x == 0 && warp == 9) {
    // offsets only the device can vouch for: such servers are skipped everywhere and flagged here, by a
    // warp that has nothing to do until the first item ends
    for (int i = lane; i < P.N; i += 32) {
      const int q0 = P.cu_q[i], n_new = P.cu_q[i + 1] - q0;
      const int k0 = P.cu_kv[i], Lkv = P.cu_kv[i + 1] - k0;
      if (!attn_server_ok(P, q0, n_new, k0, Lkv)) {
        set_status(P.d_status, GS_ERR_SHAPE);
      } else if (P.block_table != nullptr) {
        // every tile of the server must name a page of the pool (a bad entry would only read the
        // tensor map's fill value, but the result would be meaningless)
        for (int t = 0; t < (Lkv + kAtTile - 1) / kAtTile; ++t) {
          const int pg = P.block_table[(size_t)i * P.max_pages + t];
          if (pg < 0 || pg >= P.n_pages) set_status(P.d_status, GS_ERR_INVALID_ARG);
        }
      }
    }
    __syncwarp();
  }
  if (warp == 0 || warp == 10) {
    // ------------------------------------------------ TMA producers: warp 0 the keys, warp 10 the values
    // (whole warp in the loops, one elected lane issues)
    {
      const bool keys = (warp == 0);
      const int first = keys ? pre_issued : 0;      // CLUSTER: the first tile's keys are already on their way (stage 0)
      const int b_empty = keys ? kKvEmpty : kVEmpty;
      uint32_t st = (uint32_t)first % kAtStages, ph = (first == kAtStages) ? 1u : 0u;
      bool ok = true;
      AttnItem it;
      for (int k_item = 0; ok && take_item(k_item, it); ++k_item) {
        for (int j = first; j < it.n_tiles; ++j) {
          if (!mbar_wait_warp(bar(b_empty + st), ph ^ 1u, abort_flag)) { ok = false; break; }
          if (elect_one()) {
            if (keys) issue_k(it, j, st); else issue_v(it, j, st);
          }
          __syncwarp();
          if (++st == kAtStages) { st = 0; ph ^= 1u; }
        }
        // every key tile of the item is on its way: time to claim the next item
        if (!CLUSTER && keys && lane == 0) mbar_arrive(bar(kQTaken));
      }
      if (!ok || *abort_flag) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer: the whole warp walks the loops (loop
    // state and descriptors stay warp-uniform), one elected lane issues
    const uint32_t idesc_s = idesc_bf16(128, kAtTile, false, false);     // S = Q K^T, both K-major
    const uint32_t idesc_o = idesc_bf16(128, kAtHd, false, true);        // O = P V, V is MN-major
    const uint64_t dk0 = smem_desc_sw128(kv_base, 16u, 1024u);
    const uint64_t dv0 = smem_desc_sw128(kv_base + 2 * kAtHalfBytes, kAtHalfBytes, 1024u); // 64-column blocks one half apart
    // Two cursors walk the K/V ring: S = Q K^T runs one tile ahead of O += P V, so the tensor core
    // computes the next tile's scores while the softmax warps work on the current tile.
    uint32_t st_s = 0, ph_s = 0, st_v = 0, ph_v = 0;
    int n_item = 0, n_tile_total = 0;
    bool ok = true;
    auto issue_S = [&](uint32_t stage, int n) {
      if (elect_one()) {
        const uint64_t dk = dk0 + (uint64_t)(stage * (kAtKvBytes >> 4));
        const uint32_t d = tmem_S + (uint32_t)(n & 1) * 128u;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {     // 128 head dims = 8 x 16: Q +8 TMEM columns, K +32 bytes / second half 8 KB further
          const uint64_t b = dk + (uint64_t)((kk >> 2) * (kAtHalfBytes >> 4) + (kk & 3) * 2);
          umma_bf16_ts(d, tmem_Q + (uint32_t)(kk * 8), b, idesc_s, kk > 0 ? 1u : 0u);
        }
        umma_commit(bar(kSFull + (n & 1)));                                  // S of tile n ready
        umma_commit(bar(kKvEmpty + stage));                                  // and the tile's keys are done with
      }
      __syncwarp();
    };
    AttnItem it;
    for (int k_item = 0; ok && take_item(k_item, it); ++k_item) {
      if (it.n_tiles == 0) continue;
      // Q of this item sits in tensor memory (written by the softmax warps after they have
      // drained O of the previous item)
      if (!mbar_wait_warp(bar(0), (uint32_t)n_item & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      if (!mbar_wait_warp(bar(kKvFull + st_s), ph_s, abort_flag)) { ok = false; break; }
      tc_fence_after();
      issue_S(st_s, n_tile_total);
      if (++st_s == kAtStages) { st_s = 0; ph_s ^= 1u; }
      for (int j = 0; j < it.n_tiles; ++j, ++n_tile_total) {
        const int n = n_tile_total;
        if (j + 1 < it.n_tiles) {
          // The S buffer of tile n+1 was last read for tile n-1, whose P has been consumed below.
          if (!mbar_wait_warp(bar(kKvFull + st_s), ph_s, abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_S(st_s, n + 1);
          if (++st_s == kAtStages) { st_s = 0; ph_s ^= 1u; }
        }
        if (!mbar_wait_warp(bar(kPFull + (n & 1)), (uint32_t)(n >> 1) & 1u, abort_flag)) { ok = false; break; }   // P ready
        if (j == 0 && n_item > 0) {      // the first product overwrites O: the previous item's O must have been read out
          if (!mbar_wait_warp(bar(kODrained), (uint32_t)(n_item - 1) & 1u, abort_flag)) { ok = false; break; }
        }
        if (!mbar_wait_warp(bar(kVFull + st_v), ph_v, abort_flag)) { ok = false; break; }     // the tile's values have landed
        tc_fence_after();
        if (elect_one()) {
          const uint64_t dv = dv0 + (uint64_t)(st_v * (kAtKvBytes >> 4));
          const uint32_t pn = tmem_S + (uint32_t)(n & 1) * 128u;       // P sits where the scores were
#pragma unroll
          for (int kk = 0; kk < kAtTile / 16; ++kk) {     // 16 keys per step: P +8 TMEM columns, V +2 groups of 8 keys
            const uint64_t b = dv + (uint64_t)(kk * (2048 >> 4));
            umma_bf16_ts(tmem_O, pn + (uint32_t)(kk * 8), b, idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(bar(kVEmpty + st_v));                                  // the tile's values are done with
          umma_commit(bar(kPvDone));                                         // O holds tiles <= n
          if (j + 1 == it.n_tiles) umma_commit(bar(kOFull));                 // O complete
        }
        __syncwarp();
        if (++st_v == kAtStages) { st_v = 0; ph_v ^= 1u; }
      }
      ++n_item;
    }
    if (!ok || *abort_flag) { const uint64_t t0 = global_timer_ns(); while (global_timer_ns() - t0 < 200000ull) { } }
    __syncwarp();
  } else if (warp < 6) {
    // ------------------------------------------------ softmax: thread = row
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    int n_item = 0, n_tile_total = 0;
    bool ok = true;
    AttnItem it;
    for (int k_item = 0; ok && take_item(k_item, it); ++k_item) {
      if (it.n_tiles == 0) continue;
      const int R = it.n_t * P.G;
      const bool row_ok = r < R;
      const int t = it.tg * P.TB + r / P.G;              // position index inside the server
      const int last_visible = it.L + t;                 // keys 0..L+t
      // This thread's query row goes to tensor memory as packed bf16 pairs (the A operand of
      // S = Q K^T).  The previous item's S products, the only readers of Q, finished before its
      // last tile of scores was handed to this thread.
      {
        const uint4* qrow = reinterpret_cast<const uint4*>(
            P.Q + ((size_t)(it.q_row0 + r / P.G) * P.Hq + it.g * P.G + (r % P.G)) * kAtHd);
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 16) {            // 16 columns = 32 head dims = 4 x 16 bytes
          uint32_t w[16];
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint4 x = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok) x = __ldg(qrow + c0 / 4 + v4);
            w[4 * v4] = x.x; w[4 * v4 + 1] = x.y; w[4 * v4 + 2] = x.z; w[4 * v4 + 3] = x.w;
          }
          tmem_st16(tmem_Q + lane_addr + c0, w);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(0));
      }
      float m_run = -INFINITY, l_run = 0.f;     // reference maximum (scaled, log2 units) and running sum
      const int first_visible_end = it.L + it.tg * P.TB;      // last key the block's FIRST position sees
      for (int j = 0; j < it.n_tiles; ++j, ++n_tile_total) {
        const int n = n_tile_total;
        if (!mbar_wait(bar(kSFull + (n & 1)), (uint32_t)(n >> 1) & 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        // The tile is walked twice in chunks of 32 columns (rolled loops: one softmax warp per
        // scheduler executes straight from the instruction cache, and a fully unrolled 128-column
        // body does not fit it): first the row maximum, then exponentials and P.
        const uint32_t s_src = tmem_S + (uint32_t)(n & 1) * 128u + lane_addr;
        const int key0 = (it.tile0 + j) * kAtTile;       // key index inside the server
        // Only tiles that reach past what the block's first position sees need the causal mask.
        const bool masked = key0 + kAtTile - 1 > first_visible_end;
        float tm[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) tm[c] = -INFINITY;
#pragma unroll 1
        for (int c4 = 0; c4 < kAtTile / 32; ++c4) {
          float sv[32];
          uint32_t (*s4)[16] = reinterpret_cast<uint32_t (*)[16]>(sv);
          tmem_ld16(s_src + 32 * c4, s4[0]);
          tmem_ld16(s_src + 32 * c4 + 16, s4[1]);
          tmem_ld_wait();
          if (masked) {
#pragma unroll
            for (int c = 0; c < 32; ++c) sv[c] = (key0 + 32 * c4 + c <= last_visible) ? sv[c] : -INFINITY;
          }
#pragma unroll
          for (int c = 0; c < 32; ++c) tm[c & 7] = fmaxf(tm[c & 7], sv[c]);
        }
        float tmax = fmaxf(fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3])), fmaxf(fmaxf(tm[4], tm[5]), fmaxf(tm[6], tm[7])));
        tmax *= P.scale_log2;                            // the scale is positive
        // The reference maximum only moves when the tile maximum exceeds it by more than 2^8:
        // P stays below 256, the final O/l is unchanged, and O in TMEM is rescaled rarely.
        const float m_new = (tmax > m_run + 8.f) ? tmax : m_run;
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float corr = (m_run == -INFINITY) ? 0.f : fast_exp2(m_run - m_use);
        // Rescale O when this warp has a row whose reference moved (never for the first tile, whose
        // P V product overwrites O).  S runs a tile ahead, so the product of the previous tile
        // may still be in flight: wait for it first.  The next product waits for this tile's P.
        const bool need = row_ok && j > 0 && (m_new > m_run);
        if (__any_sync(0xffffffffu, need)) {
          if (!mbar_wait(bar(kPvDone), (uint32_t)(n - 1) & 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
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
        float ls[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        const float neg_m = -m_use;
        // P (bf16 pairs, 16 columns per chunk) overwrites score columns this thread has already read.
#pragma unroll 1
        for (int c4 = 0; c4 < kAtTile / 32; ++c4) {
          float sv[32];
          uint32_t (*s4)[16] = reinterpret_cast<uint32_t (*)[16]>(sv);
          tmem_ld16(s_src + 32 * c4, s4[0]);
          tmem_ld16(s_src + 32 * c4 + 16, s4[1]);
          tmem_ld_wait();
          if (masked) {
#pragma unroll
            for (int c = 0; c < 32; ++c) sv[c] = (key0 + 32 * c4 + c <= last_visible) ? sv[c] : -INFINITY;
          }
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float x0 = fmaf(sv[2 * e], P.scale_log2, neg_m);
            const float x1 = fmaf(sv[2 * e + 1], P.scale_log2, neg_m);
            const float p0 = fast_exp2(x0);
            const float p1 = (e & 1) ? poly_exp2(x1) : fast_exp2(x1);       // every fourth on the FMA pipe
            ls[e & 7] += p0 + p1;
            pk[e] = pack_bf16_pos(p0, p1);
          }
          tmem_st16(s_src + 16 * c4, pk);
        }
        tmem_st_wait();
        l_run = l_run * corr + (((ls[0] + ls[1]) + (ls[2] + ls[3])) + ((ls[4] + ls[5]) + (ls[6] + ls[7])));
        m_run = m_new;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kPFull + (n & 1)));
      }
      if (!ok) break;
      // Hand the row statistics to the epilogue warps and go on with the next item.  An item of one
      // or two tiles can end before the epilogue has picked up the previous item's statistics: wait
      // until it has (it reads them before it reports O as read out).
      if (n_item > 0 && !mbar_wait(bar(kODrained), (uint32_t)(n_item - 1) & 1u, abort_flag)) { ok = false; break; }
      s_ml[2 * r] = m_run; s_ml[2 * r + 1] = l_run;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kStatsFull));
      ++n_item;
    }
  } else if (warp < 10) {
    // ------------------------------------------------ epilogue: thread = row; runs one item behind
    // the softmax warps, so partial stores, tickets and merges overlap the next item's tiles
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    int n_item = 0, n_ticket = 0;
    bool ok = true;
    AttnItem it;
    for (int k_item = 0; ok && take_item(k_item, it); ++k_item) {
      if (it.n_tiles == 0) continue;
      const int R = it.n_t * P.G;
      const bool row_ok = r < R;
      if (!mbar_wait(bar(kStatsFull), (uint32_t)n_item & 1u, abort_flag)) { ok = false; break; }
      const float m_run = s_ml[2 * r], l_run = s_ml[2 * r + 1];
      if (!mbar_wait(bar(kOFull), (uint32_t)n_item & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      __nv_bfloat16* orow = P.O + ((size_t)(it.q_row0 + r / P.G) * P.Hq + it.g * P.G + (r % P.G)) * kAtHd;
      // partial rows go to the workspace, or (CLUSTER) to this CTA's own shared memory: every tile of
      // the item has been consumed by now, so the K/V ring is free
      float* out = CLUSTER ? reinterpret_cast<float*>(smem_raw) + (size_t)r * kAtPartStride
                           : P.part + ((size_t)it.id * kAtRows + r) * kAtPartStride;
      const bool single = (it.n_used == 1);            // the only split of its group: normalise and store
      const float inv1 = single ? 1.f / l_run : 1.f;
#pragma unroll
      for (int c0 = 0; c0 < kAtHd; c0 += 16) {
        uint32_t t16[16];
        tmem_ld16(tmem_O + lane_addr + c0, t16);
        tmem_ld_wait();
        if (row_ok) {
          if (single) {
#pragma unroll
            for (int c = 0; c < 16; c += 8) {
              uint4 pk;
              __nv_bfloat162 b0 = __floats2bfloat162_rn(__uint_as_float(t16[c]) * inv1, __uint_as_float(t16[c + 1]) * inv1);
              __nv_bfloat162 b1 = __floats2bfloat162_rn(__uint_as_float(t16[c + 2]) * inv1, __uint_as_float(t16[c + 3]) * inv1);
              __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(t16[c + 4]) * inv1, __uint_as_float(t16[c + 5]) * inv1);
              __nv_bfloat162 b3 = __floats2bfloat162_rn(__uint_as_float(t16[c + 6]) * inv1, __uint_as_float(t16[c + 7]) * inv1);
              pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
              pk.z = *reinterpret_cast<uint32_t*>(&b2); pk.w = *reinterpret_cast<uint32_t*>(&b3);
              *reinterpret_cast<uint4*>(orow + c0 + c) = pk;
            }
          } else {
#pragma unroll
            for (int c = 0; c < 16; c += 4)
              *reinterpret_cast<float4*>(out + c0 + c) = make_float4(__uint_as_float(t16[c]), __uint_as_float(t16[c + 1]),
                                                                     __uint_as_float(t16[c + 2]), __uint_as_float(t16[c + 3]));
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kODrained));          // the statistics were read before this point too
      if (!single && row_ok) { out[kAtHd] = m_run; out[kAtHd + 1] = l_run; }
      if (!CLUSTER && !single) {
        // One ticket per group: the CTA that takes the last one finds the other splits' rows
        // complete (their writers fenced before taking theirs) and merges them.  The tickets were
        // cleared by the kernel this one was launched behind: make sure that has finished.
        // The 128 epilogue threads meet on mbarriers with the usual bounded wait.
        pdl_wait();
        __threadfence();
        mbar_arrive(bar(kEpiA));
        if (!mbar_wait(bar(kEpiA), (uint32_t)n_ticket & 1u, abort_flag)) { ok = false; break; }
        if (r == 0) *s_last = (atomicAdd(&P.tickets[it.group], 1) == it.n_used - 1) ? 1 : 0;
        mbar_arrive(bar(kEpiB));
        if (!mbar_wait(bar(kEpiB), (uint32_t)n_ticket & 1u, abort_flag)) { ok = false; break; }
        ++n_ticket;
        if (*s_last != 0) {
          __threadfence();
          // Warp q merges rows q, q+4, ...; lanes across the 128 head dims (lane c4 owns 4 dims), so
          // every load is a coalesced 512-byte row of one split.
          const size_t split_stride = (size_t)P.Hkv * kAtRows * kAtPartStride;       // next split, same head
          const float* p0 = P.part + ((size_t)(it.item_base + it.tg * it.nsplit * P.Hkv + it.g) * kAtRows) * kAtPartStride;
          auto merge_rows = [&](auto kmax_c, auto unroll_c) {
            constexpr int KMAX = decltype(kmax_c)::value, UN = decltype(unroll_c)::value;
            for (int row0 = q; row0 < R; row0 += 4 * UN) {
              float4 v[UN][KMAX];
              float ms[UN][KMAX], ls[UN][KMAX];
#pragma unroll
              for (int u = 0; u < UN; ++u) {
                const int row = min(row0 + 4 * u, R - 1);
#pragma unroll
                for (int k = 0; k < KMAX; ++k) {
                  const float* p = p0 + (size_t)min(k, it.n_used - 1) * split_stride + (size_t)row * kAtPartStride;
                  v[u][k] = __ldcg(reinterpret_cast<const float4*>(p) + lane);
                  ms[u][k] = __ldcg(p + kAtHd);
                  ls[u][k] = __ldcg(p + kAtHd + 1);
                }
              }
#pragma unroll
              for (int u = 0; u < UN; ++u) {
                const int row = row0 + 4 * u;
                if (row >= R) break;
                float M = -INFINITY;
#pragma unroll
                for (int k = 0; k < KMAX; ++k) if (k < it.n_used) M = fmaxf(M, ms[u][k]);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                float L = 0.f;
#pragma unroll
                for (int k = 0; k < KMAX; ++k) {
                  if (k < it.n_used && ms[u][k] > -INFINITY) {
                    const float wk = fast_exp2(ms[u][k] - M);
                    L += ls[u][k] * wk;
                    acc.x += v[u][k].x * wk; acc.y += v[u][k].y * wk; acc.z += v[u][k].z * wk; acc.w += v[u][k].w * wk;
                  }
                }
                const float inv = 1.f / L;
                __nv_bfloat162 b0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
                __nv_bfloat162 b1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
                __nv_bfloat16* orow2 = P.O + ((size_t)(it.q_row0 + row / P.G) * P.Hq + it.g * P.G + (row % P.G)) * kAtHd;
                *reinterpret_cast<uint2*>(orow2 + lane * 4) = pk;
              }
            }
          };
          if (it.n_used <= 2) {                    // 32 rows per round trip to L2
            merge_rows(std::integral_constant<int, 2>{}, std::integral_constant<int, 8>{});
          } else if (it.n_used <= 4) {
            merge_rows(std::integral_constant<int, 4>{}, std::integral_constant<int, 4>{});
          } else if (it.n_used <= 8) {
            merge_rows(std::integral_constant<int, 8>{}, std::integral_constant<int, 2>{});
          } else {
            for (int row = q; row < R; row += 4) {
              float M = -INFINITY;
              for (int sp = 0; sp < it.n_used; ++sp)
                M = fmaxf(M, __ldcg(p0 + sp * split_stride + (size_t)row * kAtPartStride + kAtHd));
              float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
              float L = 0.f;
              for (int sp = 0; sp < it.n_used; ++sp) {
                const float* p = p0 + sp * split_stride + (size_t)row * kAtPartStride;
                const float msp = __ldcg(p + kAtHd);
                if (msp == -INFINITY) continue;
                const float wk = fast_exp2(msp - M);
                L += __ldcg(p + kAtHd + 1) * wk;
                const float4 vv = __ldcg(reinterpret_cast<const float4*>(p) + lane);
                acc.x += vv.x * wk; acc.y += vv.y * wk; acc.z += vv.z * wk; acc.w += vv.w * wk;
              }
              const float inv = 1.f / L;
              __nv_bfloat162 b0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
              __nv_bfloat162 b1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
              uint2 pk;
              pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
              __nv_bfloat16* orow2 = P.O + ((size_t)(it.q_row0 + row / P.G) * P.Hq + it.g * P.G + (row % P.G)) * kAtHd;
              *reinterpret_cast<uint2*>(orow2 + lane * 4) = pk;
            }
          }
        }
      }
      ++n_item;
    }
  } else if (warp == 11 && !CLUSTER) {
    // ------------------------------------------------ item scheduler: descriptor k goes to slot k mod
    // kAtQueue once every warp has read the descriptor that was there.  The first item (the CTA's own
    // index) was published during the set-up; item k >= 1 is claimed from the global counter when the key producer has asked for the
    // last tile of item k - 1, not earlier: the items come longest first, and a CTA that reserved
    // several ahead would sit on work that an idle CTA could do.  The ring still holds that item's last
    // tiles then, which covers the time the descriptor takes (a bisection and a dozen integer divisions).
    for (int k = 1; sched_live; ++k) {
      const int slot = k % kAtQueue;
      if (k >= kAtQueue && !mbar_wait_warp(bar(kQEmpty + slot), (uint32_t)(k / kAtQueue - 1) & 1u, abort_flag)) break;
      if (!mbar_wait_warp(bar(kQTaken), (uint32_t)(k - 1) & 1u, abort_flag)) break;
      long long id = 0;
      if (lane == 0) id = (long long)gridDim.x + atomicAdd(P.next_item, 1);
      sched_live = publish_item(k, id);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CLUSTER) {
    // Every CTA of the cluster arrives here (every wait above is bounded), with its part of the group
    // in its shared memory.  CTA 0 merges the parts that saw keys and stores the rows; the others
    // stay until it has read them.
    cluster_arrive_release();
    cluster_wait_acquire();
    const AttnItem it = s_items[0];
    const int rank = (int)cluster_cta_rank();
    const bool merging = it.valid && it.n_used > 1 && rank < it.n_used;      // uniform over the CTA
    if (merging) {
      // rows of a CTA: at most 128 / n_used; of a warp: a tenth of that, rounded up
      const int R = it.n_t * P.G;
      if (it.n_used <= 2) attn_cluster_merge<2, 7>(R, it.n_used, P.G, P.Hq, P.O, it.q_row0, it.g, rank, warp, lane, smem_raw);
      else if (it.n_used <= 4) attn_cluster_merge<4, 5>(R, it.n_used, P.G, P.Hq, P.O, it.q_row0, it.g, rank, warp, lane, smem_raw);
      else attn_cluster_merge<8, 3>(R, it.n_used, P.G, P.Hq, P.O, it.q_row0, it.g, rank, warp, lane, smem_raw);
    } else {
      cluster_arrive_release();
    }
    cluster_wait_acquire();
  }
  if (threadIdx.x == 0 && *abort_flag) set_status(P.d_status, GS_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kAtTmemCols);
  }
}

// ------------------------------------------------------------------ host side
// KV tiles per split forced by gs_verify_attn_configure (0 = automatic).
inline int& attn_tiles_per_split_override() {
  static int v = 0;
  return v;
}

// Kernel choice forced by gs_verify_attn_select: 0 = automatic, 1 = the persistent kernel, 2 / 4 / 8 =
// the CLUSTER kernel with that many CTAs per group, 3 = the CLUSTER kernel with one CTA per group.
inline int& attn_variant_override() {
  static int v = 0;
  return v;
}

struct AttnTcPlan {
  int TB, tiles_per_chunk, min_split_tiles, max_items, max_groups, grid;
  int cluster;              // CTAs per group of the CLUSTER kernel, 0 = the persistent kernel
  size_t ticket_bytes, ws_bytes;
};

// Both kernels need more dynamic shared memory than the default limit: raised once per device.
inline bool attn_set_attributes() {
  static PerDeviceOnce attr_set;
  const int slot = device_slot();
  if (attr_set.needed(slot)) {
    if (cudaFuncSetAttribute(attn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAtSmem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAtSmem) != cudaSuccess) {
      (void)cudaGetLastError();
      return false;
    }
    attr_set.mark(slot);
  }
  return true;
}

// Clusters of `cs` attention CTAs (one CTA per SM) the device can hold at once; cached per device.
inline int attn_max_clusters(int cs) {
  static int cached[kMaxDevices][4] = {};
  const int slot = device_slot();
  const int idx = cs == 2 ? 0 : cs == 4 ? 1 : 2;
  if (slot >= 0 && cached[slot][idx] != 0) return max(cached[slot][idx], 0);
  if (!attn_set_attributes()) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(cs * sm_count()));
  cfg.blockDim = dim3(kAtThreads);
  cfg.dynamicSmemBytes = kAtSmem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<true>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
  if (slot >= 0) cached[slot][idx] = n > 0 ? n : -1;
  return n;
}

inline bool attn_tc_supported(int Hq, int Hkv, int hd, gs_dtype dt) {
  if (dt != GS_BF16 || hd != kAtHd || Hkv <= 0 || Hq % Hkv != 0) return false;
  const int G = Hq / Hkv;
  return G >= 1 && G <= 128 && (Hkv * hd) % 8 == 0;     // floor(128 / G) positions per tile; leftover rows are masked
}

inline AttnTcPlan attn_tc_plan(int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv) {
  AttnTcPlan pl;
  const int G = Hq / Hkv;
  pl.TB = 128 / G;
  const int slots = sm_count();                        // one CTA per SM
  const int heads_total = max(1, N * Hkv);
  const int tiles_avg = max(1, (total_kv / max(1, N) + kAtTile - 1) / kAtTile);
  const int nsplit_target = max(1, slots / heads_total);
  pl.tiles_per_chunk = max(1, (tiles_avg + nsplit_target - 1) / nsplit_target);
  pl.min_split_tiles = kAtMinSplitTiles;
  // at most eight splits per group: the merge handles up to eight partial results per round trip
  pl.tiles_per_chunk = max(pl.tiles_per_chunk, ((max_kv_len + kAtTile - 1) / kAtTile + 7) / 8);
  if (attn_tiles_per_split_override() > 0) {
    pl.tiles_per_chunk = attn_tiles_per_split_override();
    pl.min_split_tiles = 1;
  }
  const int max_tiles = (max_kv_len + kAtTile - 1) / kAtTile;
  const long long blocks = (long long)N + Tq / pl.TB;      // sum over servers of ceil(n_new / TB)
  const int max_nsplit = max(1, min((max_tiles + pl.tiles_per_chunk - 1) / pl.tiles_per_chunk, max_tiles / pl.min_split_tiles));
  const long long items = (long long)Hkv * blocks * max_nsplit;
  pl.max_items = (int)min(items, (long long)INT_MAX / 2);
  pl.grid = min(pl.max_items, slots);
  pl.max_groups = (int)min((long long)Hkv * blocks, (long long)INT_MAX / 2);
  pl.ticket_bytes = align_up(((size_t)pl.max_groups + 1) * sizeof(int), 256);      // and the item counter behind them
  pl.ws_bytes = pl.ticket_bytes + (size_t)pl.max_items * kAtRows * kAtPartStride * sizeof(float);
  // Few groups (a small batch): one cluster per group, as wide as still lets every cluster of the
  // expected number of groups be resident at once, and no wider than leaves a part two tiles.
  pl.cluster = 0;
  const int forced = attn_variant_override();
  if (forced == 2 || forced == 4 || forced == 8) {
    pl.cluster = forced;
  } else if (forced == 3) {
    pl.cluster = 1;
  } else if (forced == 0 && attn_tiles_per_split_override() == 0) {
    const int avg_new = (Tq + max(1, N) - 1) / max(1, N);
    const long long groups_est = (long long)N * Hkv * ((avg_new + pl.TB - 1) / pl.TB);
    for (int cs = 8; cs >= 2 && pl.cluster == 0; cs >>= 1)
      if (tiles_avg >= 2 * cs && groups_est * cs <= (long long)attn_max_clusters(cs) * cs) pl.cluster = cs;
    // no more groups than SMs: still one item per CTA, so the same kernel with "clusters" of one CTA
    // (its short set-up, no ticket-clearing launch) instead of the persistent one
    if (pl.cluster == 0 && groups_est <= slots) pl.cluster = 1;
  }
  return pl;
}

// block_table == NULL: K, V are [total_kv] rows, server i at cu_kv[i].  Otherwise K, V are pools of
// n_pages pages of 128 rows, block_table[i][t] is the page of server i's t-th tile, and cu_kv only
// carries the lengths (total_kv is then the bound on cu_kv[N] the plan was made for).
inline gs_status launch_attn_tc(const void* Q, const void* K, const void* V, void* O, const int32_t* cu_q,
                                const int32_t* cu_kv, int N, int Tq, int total_kv, int max_kv_len, int Hq, int Hkv,
                                float scale, void* ws, int32_t* d_status, cudaStream_t st,
                                const int32_t* block_table = nullptr, int max_pages = 0, int n_pages = 0) {
  if (!attn_set_attributes()) return GS_ERR_CUDA;
  const AttnTcPlan pl = attn_tc_plan(N, Tq, total_kv, max_kv_len, Hq, Hkv);
  AttnTcParams P;
  P.cu_q = cu_q; P.cu_kv = cu_kv; P.d_status = d_status;
  P.block_table = block_table; P.max_pages = max_pages; P.n_pages = n_pages;
  P.tickets = static_cast<int*>(ws);
  P.next_item = P.tickets + pl.max_groups;
  P.part = reinterpret_cast<float*>(static_cast<char*>(ws) + pl.ticket_bytes);
  P.O = static_cast<__nv_bfloat16*>(O);
  P.Q = static_cast<const __nv_bfloat16*>(Q);
  P.N = N; P.Tq = Tq; P.total_kv = total_kv; P.max_kv_len = max_kv_len; P.Hq = Hq; P.Hkv = Hkv;
  P.G = Hq / Hkv; P.TB = pl.TB; P.tiles_per_chunk = pl.tiles_per_chunk; P.min_split_tiles = pl.min_split_tiles;
  P.max_items = pl.max_items;
  P.cluster = 0;
  P.scale_log2 = scale * kAtLog2e;
  auto enc = tensor_map_encoder();
  if (enc == nullptr) return GS_ERR_CUDA;
  CUtensorMap tmK, tmV;
  // K, V [rows][Hkv*hd]: box = 64 columns x 128 keys
  const uint64_t kv_rows = block_table == nullptr ? (uint64_t)total_kv : (uint64_t)n_pages * kAtTile;
  if (!make_tmap_bf16_2d(&tmK, K, kv_rows, (uint64_t)Hkv * kAtHd, (uint64_t)Hkv * kAtHd, kAtTile, 64) ||
      !make_tmap_bf16_2d(&tmV, V, kv_rows, (uint64_t)Hkv * kAtHd, (uint64_t)Hkv * kAtHd, kAtTile, 64))
    return GS_ERR_CUDA;
  if (pl.cluster > 0 && (long long)pl.max_groups * pl.cluster < (long long)INT_MAX / 2) {
    // one cluster per (server, position block, KV head) group, one item per CTA; groups beyond the
    // batch's real number (the host only knows a bound) find no item and leave at once
    P.cluster = pl.cluster;
    P.max_items = pl.max_groups * pl.cluster;
    if (launch_ex(attn_tc_kernel<true>, dim3((unsigned)P.max_items), dim3(kAtThreads), kAtSmem, st, true, pl.cluster, tmK, tmV,
                  P) != cudaSuccess) {
      (void)cudaGetLastError();
      return GS_ERR_CUDA;
    }
    count_launches(1);
    return launch_status();
  }
  const int n_ticket = (int)(pl.ticket_bytes / sizeof(int));
  attn_zero_kernel<<<(n_ticket + 1023) / 1024 > 64 ? 64 : (n_ticket + 1023) / 1024, 1024, 0, st>>>(P.tickets, n_ticket);
  if (cudaGetLastError() != cudaSuccess) return GS_ERR_CUDA;
  if (launch_ex(attn_tc_kernel<false>, dim3(pl.grid), dim3(kAtThreads), kAtSmem, st, true, 1, tmK, tmV, P) != cudaSuccess) {
    (void)cudaGetLastError();
    return GS_ERR_CUDA;
  }
  count_launches(2);
  return launch_status();
}

}  // namespace gs
