// The CTA-pair variant of the wavefront attention (Sec. 3.1 "W-shaped
// block-causal attention"; Sec. 3.2 Eq. 5): four Q tiles of one request and KV
// head ("a quad") run on a cluster of two CTAs that share every K/V tile.
//
// Why: the one-CTA kernel is bound by shared-memory bandwidth (an SS MMA reads
// its A and B operands from shared memory at the full 128 B/clk of an SM, and
// the TMA fills go through the same port).  With tcgen05 cta_group::2 one MMA
// spans both CTAs (M = 256: 128 rows in each CTA's tensor memory) and each CTA
// holds, fills and feeds only HALF of the B operand: 64 of the 128 keys of a K
// tile for S = Q K^T, 64 of the 128 columns of a V tile for O += P V.  Per
// (Q tile, key tile) 80 KB instead of 128 KB go through a CTA's shared memory.
// Every copy is an ordinary per-CTA TMA load of this GPU's own memory.
//
// Roles in each CTA (384 threads):
//   warp 0      producer: this CTA's two Q tiles, its half of every K and V tile
//               (3-stage rings); in the first CTA it also draws the work items
//               and publishes them to both CTAs
//   warp 1      first CTA only: issues every MMA of the pair and the commits,
//               which arrive on the barriers of both CTAs (one commit per CTA)
//   warps 4-7   softmax + epilogue of this CTA's tile A, 8-11 of its tile B
//               (one thread per query row; as in the one-CTA kernel)
// Streams: A = (tile A of CTA 0, tile A of CTA 1), B likewise; the MMA warp
// ping-pongs between the two streams as the one-CTA kernel does between its
// two tiles.  A stream runs over the key tiles its longer tile can see; the
// shorter tile's softmax hands in P = 0 for the rest.
// Barriers that collect from both CTAs (Q / K / V landed, P written) live in the
// first CTA: the second CTA's copies complete on them and its softmax threads
// arrive on them remotely.  Every wait is bounded; a CTA whose partner stopped
// gives up by itself.
#include <cudaTypedefs.h>

#include "attn_common.cuh"

namespace fb {

// a wait of the whole warp, one outcome, ordered against the other CTA's writes
__device__ __forceinline__ bool pair_wait(uint64_t* bar, uint32_t parity, volatile int* abort, long long limit) {
  return __all_sync(0xffffffffu, mbar_wait_cluster(bar, parity, abort, limit));
}

constexpr int kPairStages = 3;
constexpr int kPairQBytes = 32768;      // one Q tile, 128 rows x 128 bf16
constexpr int kPairKvBytes = 16384;     // half a K tile (64 keys x 128) or half a V tile (128 keys x 64)
constexpr int kPairSmem = 2 * kPairQBytes + 2 * kPairStages * kPairKvBytes + 8192;
static_assert(kPairSmem > 116 * 1024, "one CTA per SM: each allocates all 512 tensor-memory columns");

// One work item of the pair kernel as CTA `rank` sees it: its own unit record of the quad, and
// what it needs of the partner's (how far each stream runs).
struct PairGeom {
  AttnUnit me;
  int jb, chunk;
  int nMeA, nMeB;         // key tiles this CTA's tiles A / B see in this item
  int nSA, nSB;           // key tiles stream A / B runs over: the larger of the two CTAs' counts
  int nAll;
  int winSA, winSB;       // window reach of the streams (the larger of the two tiles')
};

__device__ __forceinline__ void read_unit(const AttnUnit* up, AttnUnit& u) {
  const int4* q = reinterpret_cast<const int4*>(up);
  const int4 a = q[0], b = q[1], c = q[2], d = q[3];
  u.req = a.x; u.kvh = a.y; u.slotA = a.z; u.slotB = a.w;
  u.t0A = b.x; u.t0B = b.y; u.n_tiles = b.z; u.n_chunks = b.w;
  u.nvisA = c.x; u.nvisB = c.y; u.part_base = c.z; u.prefix_len = c.w;
  u.npt = d.x; u.win_row0 = d.y; u.winA = d.z; u.winB = d.w;
}

__device__ __forceinline__ bool load_pair_item(const AttnParams& p, int idx, uint32_t rank, PairGeom& g) {
  const int4 it = *reinterpret_cast<const int4*>(&p.items[idx]);
  AttnUnit other;
  read_unit(&p.units[it.x + (int)rank], g.me);
  read_unit(&p.units[it.x + 1 - (int)rank], other);
  g.chunk = it.y; g.jb = it.z;
  const int je = it.w;
  g.nMeA = max(0, min(je, g.me.nvisA) - g.jb);
  g.nMeB = max(0, min(je, g.me.nvisB) - g.jb);
  g.nSA = max(g.nMeA, max(0, min(je, other.nvisA) - g.jb));
  g.nSB = max(g.nMeB, max(0, min(je, other.nvisB) - g.jb));
  g.nAll = max(g.nSA, g.nSB);
  g.winSA = max(g.me.winA, other.winA);
  g.winSB = max(g.me.winB, other.winB);
  return g.nAll > 0;
}

// keys of local tile j that a tile with window reach `win` may see (<= 0: none)
__device__ __forceinline__ int pair_limit(const PairGeom& g, int j, int win, int resident) {
  const int gj = g.jb + j;
  const int lim = gj < g.me.npt ? g.me.prefix_len + (resident ? win : 0) - gj * kTileN : win - (gj - g.me.npt) * kTileN;
  return min(lim, kTileN);
}

__global__ void __launch_bounds__(kAttnThreads, 1)
wavefront_attn_pair_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKwinHalf,
                           const __grid_constant__ CUtensorMap tmVwin, const __grid_constant__ CUtensorMap tmKpool,
                           const __grid_constant__ CUtensorMap tmVpool, const AttnParams p) {
  constexpr int D = 128;
  constexpr int NST = kPairStages;
  extern __shared__ uint8_t smem_raw[];
  // both CTAs of the pair must lay their shared memory out identically: the MMA descriptors name
  // offsets that are applied in each CTA
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                               // [2] tiles A, B of this CTA
  uint8_t* sK = sQ + 2 * kPairQBytes;               // [NST] this CTA's 64 keys of the tile: two 8 KB halves of d
  uint8_t* sV = sK + NST * kPairKvBytes;            // [NST] this CTA's 64 columns of d, 128 keys
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + NST * kPairKvBytes);
  uint64_t* q_full = bars + 0;          // first CTA: the four Q tiles of the pair have landed
  uint64_t* q_empty = bars + 1;         // both: the last Q K^T of the item has run
  uint64_t* k_full = bars + 2;          // [NST] first CTA: both halves landed
  uint64_t* k_empty = bars + 5;         // [NST] both
  uint64_t* v_full = bars + 8;          // [NST] first CTA
  uint64_t* v_empty = bars + 11;        // [NST] both
  uint64_t* s_full = bars + 14;         // [2] both: S of stream X is in tensor memory
  uint64_t* p_full = bars + 16;         // [2] first CTA: P of stream X written by the 8 softmax warps of both CTAs
  uint64_t* o_full = bars + 18;         // [2] both: the last P V of stream X has run
  uint64_t* item_full = bars + 20;      // [2] both: next work item published
  uint64_t* item_empty = bars + 22;     // [2] first CTA: ... and read by the 18 other consumers of both CTAs
  uint64_t* drain = bars + 24;          // give-up path
  volatile int* s_item = reinterpret_cast<volatile int*>(bars + 25);   // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
  volatile int* abortf = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const bool first = rank == 0;
  const long long LIM = p.wait_cycles;

  if (tid == 0) {
    *abortf = 0;
    mbar_init(q_full, 1); mbar_init(q_empty, 1);
    for (int i = 0; i < NST; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 8); mbar_init(&o_full[i], 1);
      mbar_init(&item_full[i], 1); mbar_init(&item_empty[i], 18);
    }
    mbar_init(drain, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmKwinHalf); tma_prefetch_desc(&tmVwin);
    tma_prefetch_desc(&tmKpool); tma_prefetch_desc(&tmVpool);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();              // both CTAs' barriers are initialised before either signals the other's
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();
  const int n_items = p.hdr->n_items;

  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
  if (warp == 0) {
    // ------------------------------------------------------------ producer
    const bool leader = elect_one();
    const uint32_t qf = mapa_u32(q_full, 0);
    int q_uses = 0, kfill = 0, vfill = 0;
    bool ok = true;
    for (int k = 0; ok; ++k) {
      int idx = 0;
      if (first) {
        if (k >= 2 && !warp_wait(&item_empty[k & 1], ((k >> 1) - 1) & 1, abortf, LIM)) { ok = false; break; }
        if (lane == 0) idx = atomicAdd(&p.hdr->ticket, 1);
        idx = uni(idx);
        if (idx >= n_items) idx = -1;
        if (lane == 0) {
          s_item[k & 1] = idx;
          st_cluster_u32(mapa_u32(const_cast<int*>(&s_item[k & 1]), 1), (uint32_t)idx);
          mbar_arrive(&item_full[k & 1]);
          mbar_arrive_cluster(mapa_u32(&item_full[k & 1], 1));
        }
        __syncwarp();
      } else {
        if (!__all_sync(0xffffffffu, mbar_wait_cluster(&item_full[k & 1], (k >> 1) & 1, abortf, LIM))) { ok = false; break; }
        idx = s_item[k & 1];
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(mapa_u32(&item_empty[k & 1], 0));
      }
      if (idx < 0) break;
      PairGeom g;
      if (!load_pair_item(p, idx, rank, g)) continue;
      const AttnUnit& me = g.me;
      const int req = uni(me.req), kvh = uni(me.kvh & 0xffff);
      const int jb = uni(g.jb), n = uni(g.nAll), npt = uni(me.npt), P = uni(me.prefix_len);
      const int win_row0 = uni(me.win_row0);
      const int win_max = uni(max(g.winSA, g.winSB));
      // the four Q tiles of the pair: each CTA loads its own two
      if (q_uses > 0 && !warp_wait(q_empty, (q_uses - 1) & 1, abortf, LIM)) { ok = false; break; }
      ++q_uses;
      if (leader) {
        if (first) mbar_arrive_expect_tx(q_full, 4 * kPairQBytes);
        const int rowA = me.slotA * p.bl + me.t0A, rowB = me.slotB * p.bl + me.t0B;
        for (int h = 0; h < 2; ++h) {
          tma_load_3d_pair(sQ + h * 16384, &tmQ, qf, h * 64, kvh * p.group, rowA);
          tma_load_3d_pair(sQ + kPairQBytes + h * 16384, &tmQ, qf, h * 64, kvh * p.group, rowB);
        }
      }
      __syncwarp();
      // key tile j of the item: this CTA's half of K (64 keys, all of d) or of V (all keys, 64 of d)
      auto load_kv = [&](int j, bool isV) -> bool {
        const int fill = isV ? vfill : kfill;
        const int st = fill % NST;
        uint64_t* empty = isV ? &v_empty[st] : &k_empty[st];
        uint64_t* full = isV ? &v_full[st] : &k_full[st];
        uint8_t* dst = (isV ? sV : sK) + st * kPairKvBytes;
        const int gj = jb + j;
        const bool paged = gj < npt;
        // pages of the tile that hold a key some tile of the item can see
        const int npg = (gj * kTileN + kPage < P + (p.resident ? win_max : 0)) ? 2 : 1;
        int page[2] = {0, 0};
        if (paged) {
#pragma unroll
          for (int pg = 0; pg < 2; ++pg) {
            const int pidx = gj * 2 + (pg < npg ? pg : 0);     // the second page may not exist: the first stands in
            int v = pidx < p.max_pages_per_req ? __ldg(&p.page_table[(size_t)req * p.max_pages_per_req + pidx]) : -1;
            if (v < 0 || v >= p.num_pages) { if (leader) atomicOr(p.status, FB_ST_BAD_PAGE); v = 0; }
            page[pg] = v;
          }
        }
        if (fill >= NST && !warp_wait(empty, ((fill / NST) - 1) & 1, abortf, LIM)) return false;
        const uint32_t fb_ = mapa_u32(full, 0);
        if (leader) {
          if (!isV) {
            // K: always both halves of the pair (Q K^T always spans 128 keys), 16 KB from each CTA
            if (first) mbar_arrive_expect_tx(full, 2 * kPairKvBytes);
            if (paged) {
              const int y = (page[rank] * p.n_kv_heads + kvh) * kPage;
              for (int h = 0; h < 2; ++h) tma_load_2d_pair(dst + h * 8192, &tmKpool, fb_, h * 64, y);
            } else {
              const int row0 = win_row0 + (gj - npt) * kTileN + 64 * (int)rank;
              for (int h = 0; h < 2; ++h) tma_load_3d_pair(dst + h * 8192, &tmKwinHalf, fb_, h * 64, kvh, row0);
            }
          } else {
            // V: this CTA's 64 columns of d for the keys of the pages in use
            if (paged) {
              if (first) mbar_arrive_expect_tx(full, 2 * npg * 8192);
              for (int pg = 0; pg < npg; ++pg) {
                const int y = (page[pg] * p.n_kv_heads + kvh) * kPage;
                tma_load_2d_pair(dst + pg * 8192, &tmVpool, fb_, 64 * (int)rank, y);
              }
            } else {
              if (first) mbar_arrive_expect_tx(full, 2 * kPairKvBytes);
              const int row0 = win_row0 + (gj - npt) * kTileN;
              tma_load_3d_pair(dst, &tmVwin, fb_, 64 * (int)rank, kvh, row0);
            }
          }
        }
        __syncwarp();
        if (isV) ++vfill; else ++kfill;
        return true;
      };
      if (!load_kv(0, false)) { ok = false; break; }
      for (int j = 0; j < n; ++j) {
        if (j + 1 < n && !load_kv(j + 1, false)) { ok = false; break; }
        if (!load_kv(j, true)) { ok = false; break; }
      }
    }
  } else if (warp == 1 && first) {
    // ---------------------------------------------------------- MMA issuer
    const bool leader = elect_one();
    int q_cnt = 0, cntPA = 0, cntPB = 0, kuse = 0, vuse = 0;
    bool ok = true;
    const uint32_t idesc_qk = umma_idesc_bf16(256, kTileN, 0, 0);
    const uint32_t idesc_pv = umma_idesc_bf16(256, D, 0, 1);
    const uint64_t dQ0 = smem_desc_sw128(smem_u32(sQ), 16, 1024);
    const uint64_t dK0 = smem_desc_sw128(smem_u32(sK), 16, 1024);
    const uint64_t dV0 = smem_desc_sw128(smem_u32(sV), 16384, 1024);
    // S_X = [Q_X of CTA 0; Q_X of CTA 1] K^T over all 128 keys (64 from each CTA's stage `st`)
    auto issue_qk = [&](const int X, int st) {
      const uint64_t qa = dQ0 + (uint32_t)((X * kPairQBytes) >> 4), kb = dK0 + (uint32_t)((st * kPairKvBytes) >> 4);
      const uint32_t d = tmem + X * 128;
      if (leader) {
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t aoff = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;     // Q: 128 rows per half of d
          const uint32_t boff = ((ks >> 2) * 8192 + (ks & 3) * 32) >> 4;      // K: 64 rows per half of d
          umma_ss_pair(d, qa + aoff, kb + boff, idesc_qk, ks > 0 ? 1u : 0u);
        }
        umma_commit_pair(&s_full[X], true);
      }
      __syncwarp();
    };
    // O_X (+)= P_X V over the first nks 16-key steps
    auto issue_pv = [&](const int X, int st, int nks, bool acc) {
      const uint64_t vb = dV0 + (uint32_t)((st * kPairKvBytes) >> 4);
      const uint32_t d = tmem + 256 + X * 128, a = tmem + X * 128;
      if (leader) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          if (ks < nks) umma_ts_pair(d, a + ks * 8, vb + (uint32_t)((ks * 2048) >> 4), idesc_pv, (acc || ks > 0) ? 1u : 0u);
      }
      __syncwarp();
    };
    auto commit = [&](uint64_t* bar) { if (leader) umma_commit_pair(bar, true); __syncwarp(); };
    for (int k = 0; ok; ++k) {
      if (!warp_wait(&item_full[k & 1], (k >> 1) & 1, abortf, LIM)) { ok = false; break; }
      const int idx = s_item[k & 1];
      __syncwarp();
      if (lane == 0) mbar_arrive(&item_empty[k & 1]);
      if (idx < 0) break;
      PairGeom g;
      if (!load_pair_item(p, idx, rank, g)) continue;
      const int nA = uni(g.nSA), nB = uni(g.nSB), n = uni(g.nAll);
      const int winSA = uni(g.winSA), winSB = uni(g.winSB);
      if (!pair_wait(q_full, q_cnt & 1, abortf, LIM)) { ok = false; break; }
      ++q_cnt;
      int st = kuse % NST;
      if (!pair_wait(&k_full[st], (kuse / NST) & 1, abortf, LIM)) { ok = false; break; }
      ++kuse;
      tc_fence_after();
      if (nA > 0) issue_qk(0, st);
      if (nB > 0) issue_qk(1, st);
      commit(&k_empty[st]);
      if (n == 1) commit(q_empty);
      for (int j = 0; j < n; ++j) {
        const int sv = vuse % NST;
        if (!pair_wait(&v_full[sv], (vuse / NST) & 1, abortf, LIM)) { ok = false; break; }
        ++vuse;
        const int st1 = kuse % NST;
        if (j + 1 < n) {
          if (!pair_wait(&k_full[st1], (kuse / NST) & 1, abortf, LIM)) { ok = false; break; }
          ++kuse;
        }
        if (j < nA) {
          const int nks = round16(pair_limit(g, j, winSA, p.resident)) >> 4;
          if (!pair_wait(&p_full[0], cntPA & 1, abortf, LIM)) { ok = false; break; }
          ++cntPA;
          tc_fence_after();
          issue_pv(0, sv, nks, j > 0);
        }
        if (j + 1 < nA) { tc_fence_after(); issue_qk(0, st1); }
        if (j < nB) {
          const int nks = round16(pair_limit(g, j, winSB, p.resident)) >> 4;
          if (!pair_wait(&p_full[1], cntPB & 1, abortf, LIM)) { ok = false; break; }
          ++cntPB;
          tc_fence_after();
          issue_pv(1, sv, nks, j > 0);
        }
        commit(&v_empty[sv]);
        if (j + 1 < nB) { tc_fence_after(); issue_qk(1, st1); }
        if (j + 1 < n) {
          commit(&k_empty[st1]);
          if (j + 2 == n) commit(q_empty);
        }
      }
      if (!ok) break;
      if (nA > 0) commit(&o_full[0]);
      if (nB > 0) commit(&o_full[1]);
    }
  }
  } else {
    // ------------------------------------------------- softmax + epilogue
    // As in the one-CTA kernel: four warps per Q tile, one thread per query row, every wait taken
    // by the whole warp with one outcome.  Differences: P is handed to the MMA warp of the first
    // CTA (a remote arrival from the second), and a tile that sees fewer key tiles than its
    // stream hands in zeros for the rest.
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    const int X = (warp - 4) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const uint32_t tS = tmem + lane_base + X * 128;
    const uint32_t tO = tmem + lane_base + 256 + X * 128;
    const uint32_t pf = mapa_u32(&p_full[X], 0);
    const float sl2 = p.scale_log2;
    int cntS = 0, cntO = 0;
    bool ok = true;
    for (int k = 0; ok; ++k) {
      if (!__all_sync(0xffffffffu, mbar_wait_cluster(&item_full[k & 1], (k >> 1) & 1, abortf, LIM))) { ok = false; break; }
      const int idx = s_item[k & 1];
      __syncwarp();
      if (lane == 0) { if (first) mbar_arrive(&item_empty[k & 1]); else mbar_arrive_cluster(mapa_u32(&item_empty[k & 1], 0)); }
      if (idx < 0) break;
      PairGeom g;
      if (!load_pair_item(p, idx, rank, g)) continue;
      const AttnUnit& me = g.me;
      const int nMine = X == 0 ? g.nMeA : g.nMeB, nStream = X == 0 ? g.nSA : g.nSB;
      if (nStream == 0) continue;
      const int winX = X == 0 ? me.winA : me.winB;
      float m_ref = -INFINITY, l = 0.f;
      for (int j = 0; j < nStream; ++j) {
        if (!warp_wait(&s_full[X], cntS & 1, abortf, LIM)) { ok = false; break; }
        ++cntS;
        tc_fence_after();
        uint32_t pk[64];
        if (j >= nMine) {
          // nothing of this key tile is visible to this Q tile: P = 0 keeps O unchanged
#pragma unroll
          for (int i = 0; i < 64; ++i) pk[i] = 0u;
        } else {
        const int limit = pair_limit(g, j, winX, p.resident);
        if (j == 0) {
          float m8[8];
#pragma unroll
          for (int t = 0; t < 8; ++t) m8[t] = -INFINITY;
          uint32_t sa[64], sb[64];
          tmem_ld32(tS, sa); tmem_ld32(tS + 32, sa + 32);
          tmem_ld_wait();
          tmem_ld32(tS + 64, sb); tmem_ld32(tS + 96, sb + 32);
#pragma unroll
          for (int i = 0; i < 64; i += 16)
#pragma unroll
            for (int t = 0; t < 8; ++t)
              m8[t] = max3(m8[t], i + t < limit ? __uint_as_float(sa[i + t]) : -INFINITY,
                           i + 8 + t < limit ? __uint_as_float(sa[i + 8 + t]) : -INFINITY);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 64; i += 16)
#pragma unroll
            for (int t = 0; t < 8; ++t)
              m8[t] = max3(m8[t], 64 + i + t < limit ? __uint_as_float(sb[i + t]) : -INFINITY,
                           64 + i + 8 + t < limit ? __uint_as_float(sb[i + 8 + t]) : -INFINITY);
          m_ref = fmaxf(fmaxf(fmaxf(m8[0], m8[1]), fmaxf(m8[2], m8[3])), fmaxf(fmaxf(m8[4], m8[5]), fmaxf(m8[6], m8[7])));
        }
        float tile_sum = 0.f;
#pragma unroll 1
        for (int attempt = 0; attempt < 2; ++attempt) {
          const float mb = m_ref * sl2;
          float2 acc2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
          const float2 sl2v = make_float2(sl2, sl2), nmb = make_float2(-mb, -mb);
          uint32_t sc[2][32];
          tmem_ld32(tS, sc[0]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t* sr = sc[c & 1];
            tmem_ld_wait();
            if (c < 3) tmem_ld32(tS + 32 * (c + 1), sc[(c + 1) & 1]);
            if (limit >= 32 * c + 32) {
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1])), sl2v, nmb);
                float2 pv;
                if (((i >> 1) & 3) < kPolyOf4) pv = exp2_poly2(x);
                else pv = make_float2(ex2_approx(x.x), ex2_approx(x.y));
                acc2[(i >> 1) & 1] = __fadd2_rn(acc2[(i >> 1) & 1], pv);
                pk[16 * c + (i >> 1)] = pack_bf16x2(pv.x, pv.y);
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const bool v0 = 32 * c + i < limit, v1 = 32 * c + i + 1 < limit;
                const float x0 = fmaf(__uint_as_float(sr[i]), sl2, -mb), x1 = fmaf(__uint_as_float(sr[i + 1]), sl2, -mb);
                const float p0 = v0 ? ex2_approx(x0) : 0.f, p1 = v1 ? ex2_approx(x1) : 0.f;
                acc2[0].x += p0 + p1;
                pk[16 * c + (i >> 1)] = pack_bf16x2(p0, p1);
              }
            }
          }
          tile_sum = (acc2[0].x + acc2[0].y) + (acc2[1].x + acc2[1].y);
          // the reference is re-based when the tile's exponentials sum to more than 2^8 (a bound on
          // every element at no per-element cost); the largest exponent is then found by one more
          // pass over S, taken by the whole warp
          const bool grow = attempt == 0 && !(tile_sum <= kGrowSum);
          if (!__any_sync(0xffffffffu, grow)) break;
          float xmax = -INFINITY;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t sr[32];
            tmem_ld32(tS + 32 * c, sr);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (32 * c + i < limit) xmax = fmaxf(xmax, fmaf(__uint_as_float(sr[i]), sl2, -mb));
          }
          const float alpha = grow ? ex2_approx(-xmax) : 1.0f;
          if (grow) { m_ref += xmax / sl2; l *= alpha; }
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            tmem_st32(tO + c * 32, o);
          }
          tmem_st_wait();
        }
        l += tile_sum;
        }
        tmem_st32(tS, pk); tmem_st32(tS + 32, pk + 32);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();          // one arrival per warp: a remote arrival per thread would queue up 128 deep
        if (lane == 0) { if (first) mbar_arrive(&p_full[X]); else mbar_arrive_cluster_relaxed(pf); }
      }
      if (!ok) break;
      if (!warp_wait(&o_full[X], cntO & 1, abortf, LIM)) { ok = false; break; }
      ++cntO;
      tc_fence_after();
      if (nMine > 0) {
        const int slot = X == 0 ? me.slotA : me.slotB, t0 = X == 0 ? me.t0A : me.t0B;
        const int kvh = me.kvh & 0xffff;
        if (me.n_chunks <= 1) {
          const int grow_ = slot * p.bl + t0 + row / p.group;
          const int head = kvh * p.group + row % p.group;
          uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)grow_ * p.n_q_heads + head) * D);
          const float inv = 1.0f / l;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              uint32_t v[8];
#pragma unroll
              for (int kk = 0; kk < 8; ++kk)
                v[kk] = pack_bf16x2(__uint_as_float(o[16 * i + 2 * kk]) * inv, __uint_as_float(o[16 * i + 2 * kk + 1]) * inv);
              st_global_v8(dst + c * 4 + 2 * i, v);
            }
          }
        } else {
          const size_t prow = ((size_t)(me.part_base + g.chunk) * 2 + X) * kTileM + row;
          p.part_ml[prow * 2 + 0] = m_ref * sl2;
          p.part_ml[prow * 2 + 1] = l;
          uint4* dst = reinterpret_cast<uint4*>(p.part_o + prow * D);
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 4; ++i) st_global_v8(dst + c * 8 + 2 * i, o + 8 * i);
          }
        }
      }
      tc_fence_before();
    }
  }
  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abortf) {
    // give-up path, as in the one-CTA kernel: everything the MMA warp issued is complete before
    // tensor memory goes back, copies in flight land while the CTA sleeps
    if (tid == 0) atomicOr(p.status, FB_ST_DEV_TIMEOUT);
    if (warp == 1 && first) {
      if (elect_one()) umma_commit_pair(drain, false);
      __syncwarp();
      for (int i = 0; i < 4096 && !mbar_test(drain, 0); ++i) __nanosleep(200);
    }
    for (int i = 0; i < 64; ++i) __nanosleep(10000);
    __syncthreads();
  }
  // neither CTA may leave while the other can still signal its barriers or read its shared memory
  cluster_sync_all();
  if (warp == 1) { tc_fence_after(); tmem_dealloc_pair(tmem, 512); }
}

// ------------------------------------------------------------------- host
int attn_pair_device_setup(fb_ctx* ctx) {
  return cuda_err(ctx, cudaFuncSetAttribute(wavefront_attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kPairSmem), "smem attr");
}

int launch_attn_pair(fb_ctx* ctx, const int32_t* page_table, void* out, void* ws, int32_t* status,
                     cudaStream_t stream) {
  AttnParams p;
  fill_attn_params(ctx, p, page_table, out, ws, status, 1);
  const int grid = (ctx->num_sms / 2) * 2;
  if (int e = cuda_err(ctx, launch_pdl_cluster(wavefront_attn_pair_kernel, grid, kAttnThreads, (size_t)kPairSmem, stream, 2,
                                               ctx->tm_q, ctx->tm_kwin_half, ctx->tm_vwin, ctx->tm_kpool, ctx->tm_vpool, p),
                       "wavefront_attn_pair_kernel launch"))
    return e;
  return launch_attn_combine(ctx, p, 1, stream);
}

}  // namespace fb
