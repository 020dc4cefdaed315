// fb_wavefront_attn: W-shaped block-causal GQA attention over the packed
// wavefronts (Sec. 3.1 "W-shaped block-causal attention"; Sec. 3.2 Eq. 5).
//
// Persistent, warp-specialised tcgen05 kernel, one CTA per SM:
//   warps 0, 2  TMA producers: Q tiles, K/V tiles of the paged prefix (page-table
//               lookups) and of the window tensors, 2-stage K and V rings, one
//               stage of each per warp
//   warp 1      MMA issuer: S = Q K^T and O += P V with tcgen05.mma, S/P and O
//               in TMEM, two Q tiles (A, B) ping-ponged so that the tensor pipe
//               works on one tile while the other is in softmax
//   warp 3      idle (it completes the control warpgroup, which gives its
//               registers to the softmax warpgroups with setmaxnreg)
//   warps 4-7   softmax of tile A, one thread per query row: tcgen05.ld of S in
//               32-column chunks, exp2 against a lazily re-based reference
//               (only the first tile of an item takes a max pass; part of the
//               exponentials runs as a polynomial on the FMA pipe), P (bf16)
//               kept in registers until the tile is known to be in range, then
//               written back over S in TMEM; epilogue
//   warps 8-11  the same for tile B
// A Q tile is 128 rows = (128/G tokens) x (G query heads of one KV head) of one
// slot.  A unit runs two Q tiles side by side: two tiles of one request and KV
// head, which share each K/V tile from shared memory, or the odd tile left
// over, run under two adjacent KV heads at once (two K/V streams, served in
// readiness order).  The mask is per tile: a tile of the frozen prefix is
// fully visible except the ragged last one; the window tile is visible up to
// (s+1)*bl keys for a query in window slot s.  Tiles nobody can see are never
// loaded (the work list only spans visible tiles), and ragged tiles run the
// MMAs on ceil(valid/16)*16 keys only.  With the window resident in the pages
// every key tile is a paged one over absolute positions.
// Work items are sorted longest first by the pack kernel and drawn by the CTAs
// from a global ticket.
// Long key ranges are split across CTAs; partial (max, sum, O) go to the
// workspace and a second kernel merges them in a fixed order.
#include <cudaTypedefs.h>

#include "attn_common.cuh"

namespace fb {

// F8: the KV pages hold FP8 E4M3 bytes (window resident in the pages, D = 128).  Both products
// then run as kind::f8f6f4 MMAs: the softmax warps convert their Q tile to E4M3 once per item
// (per-row power-of-two scale, undone in the row's score factor together with the K scale of
// the KV head) and write P as E4M3; O is scaled by the V scale of the KV head at the end.
template <int D, bool F8>
__global__ void __launch_bounds__(kAttnThreads, 1)
wavefront_attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKwin,
                      const __grid_constant__ CUtensorMap tmVwin, const __grid_constant__ CUtensorMap tmKpool,
                      const __grid_constant__ CUtensorMap tmVpool, const AttnParams p) {
  static_assert(!F8 || D == 128, "8-bit pages: head_dim 128 only (one 128-byte swizzle row per key)");
  constexpr int NH = D / 64;                 // 64-element halves of the head dim (bf16 tiles)
  constexpr int Q_TILE_BYTES = NH * 16384;   // one 128-row bf16 tile
  constexpr int NHKV = F8 ? 1 : NH;          // 16 KB blocks of a K/V tile
  constexpr int TILE_BYTES = NHKV * 16384;   // one 128-key K or V tile
  constexpr int PAGE_BYTES = NHKV * 8192;    // one 64-key page of it
  constexpr int KSTEPS = F8 ? D / 32 : D / 16;   // MMAs per Q K^T
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                        // [2] tiles A, B (bf16, as loaded)
  uint8_t* sQ8 = sQ + 2 * Q_TILE_BYTES;      // [2] the same in E4M3 (F8 only)
  uint8_t* sK = sQ8 + (F8 ? 2 * 16384 : 0);  // [2] stages
  uint8_t* sV = sK + 2 * TILE_BYTES;         // [2] stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + 2 * TILE_BYTES);
  uint64_t* q_full = bars + 0;
  uint64_t* q_empty = bars + 1;
  uint64_t* k_full = bars + 2;    // [2]
  uint64_t* k_empty = bars + 4;   // [2]
  uint64_t* v_full = bars + 6;    // [2]
  uint64_t* v_empty = bars + 8;   // [2]
  uint64_t* s_full = bars + 10;   // [2] A, B
  uint64_t* p_full = bars + 12;   // [2]
  uint64_t* o_full = bars + 14;   // [2]
  uint64_t* item_full = bars + 20;   // [2] next work item published by the producer
  uint64_t* item_empty = bars + 22;  // [2] ... and read by the second producer, the MMA warp and the 8 softmax warps
  volatile int* s_item = reinterpret_cast<volatile int*>(bars + 24);   // [2]
  uint64_t* drain = bars + 25;       // give-up path only: everything the MMA warp has issued is complete
  uint64_t* q8_full = bars + 26;     // [2] F8: tile X converted to E4M3 by its 128 softmax threads
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
  volatile int* abortf = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long LIM = p.wait_cycles;

  if (tid == 0) {
    *abortf = 0;
    mbar_init(q_full, 1); mbar_init(q_empty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
      mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 128); mbar_init(&o_full[i], 1);
      mbar_init(&item_full[i], 1); mbar_init(&item_empty[i], 10);
    }
    mbar_init(drain, 1);
    mbar_init(&q8_full[0], 128); mbar_init(&q8_full[1], 128);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmKwin); tma_prefetch_desc(&tmVwin);
    tma_prefetch_desc(&tmKpool); tma_prefetch_desc(&tmVpool);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();                     // the work list (and everything else) of the previous kernels is complete
  const int n_items = p.hdr->n_items;

  // The control warpgroup (warps 0-3) hands registers to the softmax
  // warpgroups.  All four warps of a warpgroup execute the same setmaxnreg
  // instruction, and each role's code is dominated by its warpgroup's one.
  // Registers only move inside the CTA: what the two softmax warpgroups take
  // (2 x 128 x (208 - 168)) must not exceed what the control warpgroup gives up
  // (128 x (168 - 88)), or setmaxnreg.inc blocks for good.
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
  if (warp == 0 || warp == 2) {
    // ----------------------------------------------------------- producers
    // Warp 0 owns K/V stage 0, warp 2 owns stage 1; warp 0 also draws the work
    // items and loads Q.  A unit whose tiles share K/V takes the stages in turn
    // (rr_k, rr_v), so each warp issues every other tile; a unit with two K/V
    // streams gives stage X to tile X, so each warp feeds one stream.  The MMA
    // warp follows the same rule.  The whole warp runs the loop converged and
    // one elected lane issues the copies: operands of the TMA / MMA
    // instructions then live in uniform registers (issuing from a single
    // diverged lane costs ~200 cycles each).
    const bool leader = elect_one();
    const int mine = warp >> 1;                    // the stage this warp fills
    int q_uses = 0, kfill = 0, vfill = 0, rr_k = 0, rr_v = 0;
    bool ok = true;
    // Page ids of the current request: lane i of pc_cur holds entry 32 * pc_blk + i of its
    // page-table row, pc_next the following 32 (loaded ahead), so a K/V tile costs two
    // shuffles instead of two dependent global loads.
    int pc_blk = 0, pc_cur = 0, pc_next = 0;
    auto load_pages = [&](int req, int blk) -> int {
      const int e = blk * 32 + lane;
      return e < p.max_pages_per_req ? __ldg(&p.page_table[(size_t)req * p.max_pages_per_req + e]) : -1;
    };
    // key tile j of the item, K or V of KV head kvh, into this warp's stage
    auto load_kv = [&](const ItemU& g, int kvh, int j, bool isV) -> bool {
      const int fill = isV ? vfill : kfill;
      uint64_t* full = isV ? &v_full[mine] : &k_full[mine];
      uint64_t* empty = isV ? &v_empty[mine] : &k_empty[mine];
      uint8_t* dst = (isV ? sV : sK) + mine * TILE_BYTES;
      const int gj = g.jb + j;
      const bool paged = gj < g.npt;
      const int npg = (gj * kTileN + kPage < g.prefix_len + (p.resident ? max(g.winA, g.winB) : 0)) ? 2 : 1;
      int page[2] = {0, 0};
      if (paged) {
        // the window of 64 cached entries moves on once V has reached its second half
        if (isV && ((gj * 2) >> 5) >= pc_blk + 1) {
          pc_cur = pc_next; ++pc_blk;
          pc_next = load_pages(g.req, pc_blk + 1);
        }
#pragma unroll
        for (int pg = 0; pg < 2; ++pg) {
          const int pidx = gj * 2 + pg, blk = pidx >> 5;
          int v = __shfl_sync(0xffffffffu, blk == pc_blk ? pc_cur : pc_next, pidx & 31);
          if (blk != pc_blk && blk != pc_blk + 1)                  // outside the window (not expected)
            v = pidx < p.max_pages_per_req ? __ldg(&p.page_table[(size_t)g.req * p.max_pages_per_req + pidx]) : -1;
          page[pg] = pg < npg ? v : 0;
        }
      }
      if (fill > 0 && !warp_wait(empty, (fill - 1) & 1, abortf, LIM)) return false;
      if (paged) {
#pragma unroll
        for (int pg = 0; pg < 2; ++pg) {
          if (page[pg] < 0 || page[pg] >= p.num_pages) { if (leader) atomicOr(p.status, FB_ST_BAD_PAGE); page[pg] = 0; }
        }
        if (leader) {
          mbar_arrive_expect_tx(full, npg * PAGE_BYTES);
          for (int pg = 0; pg < npg; ++pg) {
            const int y = (page[pg] * p.n_kv_heads + kvh) * kPage;
            for (int h = 0; h < NHKV; ++h)
              tma_load_2d(dst + h * 16384 + pg * 8192, isV ? &tmVpool : &tmKpool, full, h * 64, y);
          }
        }
      } else if (leader) {
        mbar_arrive_expect_tx(full, TILE_BYTES);
        const int row0 = g.win_row0 + (gj - g.npt) * kTileN;
        for (int h = 0; h < NH; ++h)
          tma_load_3d(dst + h * 16384, isV ? &tmVwin : &tmKwin, full, h * 64, kvh, row0);
      }
      __syncwarp();
      if (isV) ++vfill; else ++kfill;
      return true;
    };
    // Work items are handed out longest first through a global ticket; warp 0
    // draws the ticket and publishes the item to the other roles.
    for (int k = 0; ok; ++k) {
      int idx = 0;
      if (warp == 0) {
        if (k >= 2 && !warp_wait(&item_empty[k & 1], ((k >> 1) - 1) & 1, abortf, LIM)) { ok = false; break; }
        if (lane == 0) idx = atomicAdd(&p.hdr->ticket, 1);
        idx = uni(idx);
        if (idx >= n_items) idx = -1;
        if (lane == 0) { s_item[k & 1] = idx; mbar_arrive(&item_full[k & 1]); }
        __syncwarp();
        if (idx < 0) break;          // (the combine kernel re-arms the ticket for the next launch)
      } else {
        if (!warp_wait(&item_full[k & 1], (k >> 1) & 1, abortf, LIM)) { ok = false; break; }
        idx = s_item[k & 1];
        __syncwarp();
        if (lane == 0) mbar_arrive(&item_empty[k & 1]);
        if (idx < 0) break;
      }
      ItemU g;
      if (!load_item_uniform(p, idx, g)) continue;
      pc_blk = (g.jb * 2) >> 5;
      pc_cur = load_pages(g.req, pc_blk);
      pc_next = load_pages(g.req, pc_blk + 1);
      if (warp == 0) {
        if (q_uses > 0 && !warp_wait(q_empty, (q_uses - 1) & 1, abortf, LIM)) { ok = false; break; }
        ++q_uses;
        if (leader) {
          mbar_arrive_expect_tx(q_full, ((g.nA > 0) + (g.nB > 0)) * Q_TILE_BYTES);
          if (g.nA > 0)
            for (int h = 0; h < NH; ++h)
              tma_load_3d(sQ + h * 16384, &tmQ, q_full, h * 64, g.kvhA * p.group, g.rowA);
          if (g.nB > 0)
            for (int h = 0; h < NH; ++h)
              tma_load_3d(sQ + Q_TILE_BYTES + h * 16384, &tmQ, q_full, h * 64, g.kvhB * p.group, g.rowB);
        }
        __syncwarp();
      }
      if (!g.dual()) {
        // K runs one tile ahead of V; this warp takes the tiles that fall on its stage
        if ((rr_k++ & 1) == mine && !load_kv(g, g.kvhA, 0, false)) { ok = false; break; }
        for (int j = 0; j < g.n; ++j) {
          if (j + 1 < g.n && (rr_k++ & 1) == mine && !load_kv(g, g.kvhA, j + 1, false)) { ok = false; break; }
          if ((rr_v++ & 1) == mine && !load_kv(g, g.kvhA, j, true)) { ok = false; break; }
        }
      } else {
        const int kvh = mine ? g.kvhB : g.kvhA;
        if (!load_kv(g, kvh, 0, false)) { ok = false; break; }
        for (int j = 0; j < g.n; ++j) {
          if (!load_kv(g, kvh, j, true)) { ok = false; break; }
          if (j + 1 < g.n && !load_kv(g, kvh, j + 1, false)) { ok = false; break; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer
    const bool leader = elect_one();
    int q_cnt = 0, q8A = 0, q8B = 0, cntPA = 0, cntPB = 0;
    bool ok = true;
    // All descriptors are built once; a k-step only adds a constant to the
    // address field (low word, no carry: shared-memory addresses fit the
    // 14-bit field).
    const uint32_t idesc_pv = F8 ? umma_idesc_e4m3(128, D, 0, 1) : umma_idesc_bf16(128, D, 0, 1);
    const uint32_t idesc_qk_full = F8 ? umma_idesc_e4m3(128, kTileN, 0, 0) : umma_idesc_bf16(128, kTileN, 0, 0);
    constexpr int QOP_BYTES = F8 ? 16384 : Q_TILE_BYTES;       // the Q tile the MMAs read
    const uint64_t dQ0 = smem_desc_sw128(smem_u32(F8 ? sQ8 : sQ), 16, 1024);
    const uint64_t dK0 = smem_desc_sw128(smem_u32(sK), 16, 1024);
    const uint64_t dV0 = smem_desc_sw128(smem_u32(sV), 16384, 1024);
    // S_X = Q_X K^T over `ncols` keys of K stage `st`; X is 0 (tile A) or 1 (tile B)
    auto issue_qk = [&](const int X, int st, int ncols) {
      const uint32_t idesc = ncols == kTileN ? idesc_qk_full
                             : (F8 ? umma_idesc_e4m3(128, ncols, 0, 0) : umma_idesc_bf16(128, ncols, 0, 0));
      const uint64_t qa = dQ0 + (uint32_t)((X * QOP_BYTES) >> 4), kb = dK0 + (uint32_t)((st * TILE_BYTES) >> 4);
      const uint32_t d = tmem + X * 128;
      if (leader) {
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {          // 32 bytes of the 128-byte row per step
          const uint32_t off = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;
          if (F8) umma_ss_f8(d, qa + off, kb + off, idesc, ks > 0 ? 1u : 0u);
          else umma_ss(d, qa + off, kb + off, idesc, ks > 0 ? 1u : 0u);
        }
        umma_commit(&s_full[X]);
      }
      __syncwarp();
    };
    // O_X (+)= P_X V over k-steps [ks0, ks1) of V stage `st`; P_X is read from TMEM.  A step
    // is 16 keys (bf16) or 32 keys (E4M3): 8 TMEM columns of P and 2 KB / 4 KB of V rows.
    constexpr int PV_STEPS = F8 ? 4 : 8, PV_STEP_BYTES = F8 ? 4096 : 2048;
    auto issue_pv = [&](const int X, int st, int ks0, int ks1, bool acc) {
      const uint64_t vb = dV0 + (uint32_t)((st * TILE_BYTES) >> 4);
      const uint32_t d = tmem + 256 + X * 128, a = tmem + X * 128;
      if (leader) {
#pragma unroll
        for (int ks = 0; ks < PV_STEPS; ++ks)
          if (ks >= ks0 && ks < ks1) {
            if (F8) umma_ts_f8(d, a + ks * 8, vb + (uint32_t)((ks * PV_STEP_BYTES) >> 4), idesc_pv, (acc || ks > 0) ? 1u : 0u);
            else umma_ts(d, a + ks * 8, vb + (uint32_t)((ks * PV_STEP_BYTES) >> 4), idesc_pv, (acc || ks > 0) ? 1u : 0u);
          }
      }
      __syncwarp();
    };
    // k-steps of P V that cover the first `lim` keys of a tile
    auto pv_steps = [&](int lim) { return F8 ? (lim + 31) >> 5 : round16(lim) >> 4; };
    auto commit = [&](uint64_t* bar) { if (leader) umma_commit(bar); __syncwarp(); };
    // fills consumed from each K / V stage (see the producer)
    int kuse0 = 0, kuse1 = 0, vuse0 = 0, vuse1 = 0, rr_k = 0, rr_v = 0;
    auto wait_k = [&](int st) -> bool {
      const int use = st ? kuse1 : kuse0;
      if (st) ++kuse1; else ++kuse0;
      return warp_wait(&k_full[st], use & 1, abortf, LIM);
    };
    auto wait_v = [&](int st) -> bool {
      const int use = st ? vuse1 : vuse0;
      if (st) ++vuse1; else ++vuse0;
      return warp_wait(&v_full[st], use & 1, abortf, LIM);
    };
    for (int k = 0; ok; ++k) {
      if (!warp_wait(&item_full[k & 1], (k >> 1) & 1, abortf, LIM)) { ok = false; break; }
      const int idx = s_item[k & 1];
      __syncwarp();
      if (lane == 0) mbar_arrive(&item_empty[k & 1]);
      if (idx < 0) break;
      ItemU g;
      if (!load_item_uniform(p, idx, g)) continue;
      const int nA = g.nA, nB = g.nB, n = g.n;
      if (F8) {     // the tiles in E4M3, written by the softmax warps
        if (nA > 0 && !warp_wait(&q8_full[0], q8A & 1, abortf, LIM)) { ok = false; break; }
        if (nB > 0 && !warp_wait(&q8_full[1], q8B & 1, abortf, LIM)) { ok = false; break; }
        q8A += nA > 0; q8B += nB > 0;
        fence_proxy_async_smem();
      } else if (!warp_wait(q_full, q_cnt & 1, abortf, LIM)) { ok = false; break; }
      ++q_cnt;
      if (!g.dual()) {
        // ---- tiles A and B share every K/V tile
        int st = rr_k++ & 1;
        if (!wait_k(st)) { ok = false; break; }
        tc_fence_after();
        if (nA > 0) issue_qk(0, st, round16(g.limit(0, g.winA, p.resident)));
        if (nB > 0) issue_qk(1, st, round16(g.limit(0, g.winB, p.resident)));
        commit(&k_empty[st]);
        if (n == 1) commit(q_empty);               // Q is free once its last QK has run
        for (int j = 0; j < n; ++j) {
          const int sv = rr_v++ & 1;
          const int st1 = rr_k & 1;                // stage of K(j+1), if there is one
          if (!wait_v(sv)) { ok = false; break; }
          // K(j+1) has normally landed by now: taking its barrier here keeps the wait
          // off the P V -> next Q K^T stretch that the softmax warps are waiting for
          if (j + 1 < n) { ++rr_k; if (!wait_k(st1)) { ok = false; break; } }
          // tile A: O_A += P_A(j) V(j), then S_A(j+1) so that softmax A can go on
          if (j < nA) {
            const int nks = pv_steps(g.limit(j, g.winA, p.resident));
            if (!warp_wait(&p_full[0], cntPA & 1, abortf, LIM)) { ok = false; break; }
            ++cntPA;
            tc_fence_after();
            issue_pv(0, sv, 0, nks, j > 0);
          }
          if (j + 1 < nA) {
            tc_fence_after();
            issue_qk(0, st1, round16(g.limit(j + 1, g.winA, p.resident)));
          }
          // tile B
          if (j < nB) {
            const int nks = pv_steps(g.limit(j, g.winB, p.resident));
            if (!warp_wait(&p_full[1], cntPB & 1, abortf, LIM)) { ok = false; break; }
            ++cntPB;
            tc_fence_after();
            issue_pv(1, sv, 0, nks, j > 0);
          }
          commit(&v_empty[sv]);
          if (j + 1 < nB) {
            tc_fence_after();
            issue_qk(1, st1, round16(g.limit(j + 1, g.winB, p.resident)));
          }
          if (j + 1 < n) {
            commit(&k_empty[st1]);
            if (j + 2 == n) commit(q_empty);
          }
        }
      } else {
        // ---- one Q tile under two KV heads: stream X owns K stage X and V stage X
        // (nA == nB == n, and both tiles see the same keys)
        if (!wait_k(0)) { ok = false; break; }
        tc_fence_after();
        issue_qk(0, 0, round16(g.limit(0, g.winA, p.resident)));
        commit(&k_empty[0]);
        if (!wait_k(1)) { ok = false; break; }
        tc_fence_after();
        issue_qk(1, 1, round16(g.limit(0, g.winB, p.resident)));
        commit(&k_empty[1]);
        if (n == 1) commit(q_empty);
        // The streams do not depend on each other: serve whichever tile's P is ready.
        int jA = 0, jB = 0, qk_left = 2 * (n - 1), spins = 0;
        long long t0 = clock64();
        while (jA < n || jB < n) {
          int X = -1;
          if (jA < n && __all_sync(0xffffffffu, mbar_test(&p_full[0], cntPA & 1))) X = 0;
          else if (jB < n && __all_sync(0xffffffffu, mbar_test(&p_full[1], cntPB & 1))) X = 1;
          if (X < 0) {
            if ((++spins & 63) == 0) {
              bool give_up = *abortf != 0;
              if (!give_up && clock64() - t0 > LIM) { *abortf = 1; give_up = true; }
              if (__any_sync(0xffffffffu, give_up)) { ok = false; break; }
            }
            continue;
          }
          const int j = X ? jB : jA;
          if (X) { ++jB; ++cntPB; } else { ++jA; ++cntPA; }
          if (!wait_v(X)) { ok = false; break; }
          tc_fence_after();
          issue_pv(X, X, 0, pv_steps(g.limit(j, g.winA, p.resident)), j > 0);
          commit(&v_empty[X]);
          if (j + 1 < n) {
            // this stream's next K tile could only be requested when its last Q K^T had
            // finished, one softmax ago: give it the time of the P V as well
            if (!wait_k(X)) { ok = false; break; }
            tc_fence_after();
            issue_qk(X, X, round16(g.limit(j + 1, g.winA, p.resident)));
            commit(&k_empty[X]);
            if (--qk_left == 0) commit(q_empty);
          }
          t0 = clock64();
        }
      }
      if (!ok) break;
      if (nA > 0) commit(&o_full[0]);
      if (nB > 0) commit(&o_full[1]);
    }
  }
  } else {
    // ------------------------------------------------- softmax + epilogue
    // Four warps per Q tile, one thread per query row (its TMEM lane).  Every wait is
    // taken by the whole warp with one outcome (warp_wait): tcgen05.ld / st below are
    // warp-wide and must never run with part of a warp gone.
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    const int X = (warp - 4) >> 2;                 // 0: tile A, 1: tile B
    const int quad = warp & 3;                     // TMEM lane quadrant of this warp
    const int row = quad * 32 + lane;              // query row of the tile
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const uint32_t tS = tmem + lane_base + X * 128;
    const uint32_t tO = tmem + lane_base + 256 + X * 128;
    float sl2 = p.scale_log2;          // F8: per item and row (K scale of the KV head, Q scale of the row)
    float out_scale = 1.0f;            // F8: V scale of the KV head
    constexpr float kShift = F8 ? kF8PShift : 0.f;
    int cntS = 0, cntO = 0, qcnt = 0;
    bool ok = true;
    for (int k = 0; ok; ++k) {
      if (!warp_wait(&item_full[k & 1], (k >> 1) & 1, abortf, LIM)) { ok = false; break; }
      const int idx = s_item[k & 1];
      __syncwarp();
      if (lane == 0) mbar_arrive(&item_empty[k & 1]);
      if (idx < 0) break;
      ItemGeom g;
      if (!load_item(p, idx, g)) continue;
      const int q_par = qcnt & 1;        // phase of q_full that carries this item's Q tiles
      ++qcnt;
      const int nMine = X == 0 ? g.nA : g.nB;
      if (nMine == 0) continue;
      const int winX = X == 0 ? g.un.winA : g.un.winB;
      if constexpr (F8) {
        // This thread's Q row, bf16 -> E4M3 with the power of two that brings its largest
        // magnitude into [128, 256) (exact), into the tile the MMAs read.  The 128-byte swizzle
        // puts 16-byte piece c of row r at piece c ^ (r & 7) of its 128-byte line.
        if (!warp_wait(q_full, q_par, abortf, LIM)) { ok = false; break; }
        const uint8_t* src = sQ + X * Q_TILE_BYTES + (row >> 3) * 1024 + (row & 7) * 128;
        uint4 qv[16];
#pragma unroll
        for (int c = 0; c < 16; ++c)
          qv[c] = *reinterpret_cast<const uint4*>(src + (c >> 3) * 16384 + (((c & 7) ^ (row & 7)) << 4));
        uint32_t am = 0;                 // largest |x| as bf16 bits (sign cleared: integer order = magnitude order)
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const uint32_t w[4] = {qv[c].x, qv[c].y, qv[c].z, qv[c].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) am = max(am, max(w[i] & 0x7fffu, (w[i] >> 16) & 0x7fffu));
        }
        int kq = 134 - (int)(am >> 7);   // biased exponent of the bf16 -> 2^kq * amax in [128, 256)
        kq = am < 0x80u ? 0 : min(max(kq, -100), 100);      // zero / subnormal rows: no scaling
        const float f = __int_as_float((kq + 127) << 23);
        uint8_t* dst = sQ8 + X * 16384 + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          const uint4 a = qv[2 * c8], b = qv[2 * c8 + 1];
          const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
          uint32_t o[4];
#pragma unroll
          for (int i = 0; i < 4; ++i)
            o[i] = pack_e4m3x4(__uint_as_float(w[2 * i] << 16) * f, __uint_as_float(w[2 * i] & 0xffff0000u) * f,
                               __uint_as_float(w[2 * i + 1] << 16) * f, __uint_as_float(w[2 * i + 1] & 0xffff0000u) * f);
          *reinterpret_cast<uint4*>(dst + ((c8 ^ (row & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
        }
        fence_proxy_async_smem();
        mbar_arrive(&q8_full[X]);
        const int kvh = X == 0 ? g.kvhA : g.kvhB;
        sl2 = p.scale_log2 * __ldg(&p.k_scale[kvh]) * __int_as_float((127 - kq) << 23);
        out_scale = __ldg(&p.v_scale[kvh]);
      }
      float m_ref = -INFINITY, l = 0.f;
      for (int j = 0; j < nMine; ++j) {
        if (!warp_wait(&s_full[X], cntS & 1, abortf, LIM)) { ok = false; break; }
        ++cntS;
        tc_fence_after();
        const int limit = tile_limit(g, j, winX, p.resident);
        // The running reference m_ref is only re-based when a score exceeds it by
        // more than 2^8 (lazy rescale), so the common tile needs no separate max
        // pass: the exponentials are taken against the old reference while the
        // largest exponent is tracked, P stays in registers, and only if the
        // bound was broken is the tile redone against the new reference.  The
        // first tile of an item has no reference yet and takes a max pass.
        if (j == 0) {
          float m8[8];
#pragma unroll
          for (int t = 0; t < 8; ++t) m8[t] = -INFINITY;
          uint32_t sa[64], sb[64];
          tmem_ld32(tS, sa); tmem_ld32(tS + 32, sa + 32);
          tmem_ld_wait();
          tmem_ld32(tS + 64, sb); tmem_ld32(tS + 96, sb + 32);     // in flight during the first half
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
        uint32_t pk[F8 ? 32 : 64];             // P of this tile: packed bf16 pairs, or E4M3 four to a word
        // 8-bit P saturates at 448, so the largest exponent of the tile is tracked element by
        // element; bf16 P has the range of fp32 and only needs the tile's sum to stay finite
        constexpr bool TRACK = F8;
        float tile_sum = 0.f;
#pragma unroll 1
        for (int attempt = 0; attempt < 2; ++attempt) {
          const float mb = m_ref * sl2 - kShift;
          float2 acc2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
          float xm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          const float2 sl2v = make_float2(sl2, sl2), nmb = make_float2(-mb, -mb);
          uint32_t sc[2][32];
          tmem_ld32(tS, sc[0]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t* sr = sc[c & 1];
            tmem_ld_wait();
            if (c < 3) tmem_ld32(tS + 32 * (c + 1), sc[(c + 1) & 1]);   // next chunk in flight
            if (limit >= 32 * c + 32) {
              float2 prev = make_float2(0.f, 0.f);
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1])), sl2v, nmb);
                if constexpr (TRACK) xm4[(i >> 1) & 3] = max3(xm4[(i >> 1) & 3], x.x, x.y);
                float2 pv;
                if (((i >> 1) & 3) < (F8 ? kPolyOf4F8 : kPolyOf4)) pv = exp2_poly2(x);
                else pv = make_float2(ex2_approx(x.x), ex2_approx(x.y));
                acc2[(i >> 1) & 1] = __fadd2_rn(acc2[(i >> 1) & 1], pv);
                if constexpr (F8) {
                  if (i & 2) pk[8 * c + (i >> 2)] = pack_e4m3x4(prev.x, prev.y, pv.x, pv.y);
                  prev = pv;
                } else {
                  pk[16 * c + (i >> 1)] = pack_bf16x2(pv.x, pv.y);
                }
              }
            } else {
              float2 prev = make_float2(0.f, 0.f);
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const bool v0 = 32 * c + i < limit, v1 = 32 * c + i + 1 < limit;
                const float x0 = fmaf(__uint_as_float(sr[i]), sl2, -mb), x1 = fmaf(__uint_as_float(sr[i + 1]), sl2, -mb);
                if constexpr (TRACK) {
                  if (v0) xm4[0] = fmaxf(xm4[0], x0);
                  if (v1) xm4[1] = fmaxf(xm4[1], x1);
                }
                const float p0 = v0 ? ex2_approx(x0) : 0.f, p1 = v1 ? ex2_approx(x1) : 0.f;
                acc2[0].x += p0 + p1;
                if constexpr (F8) {
                  if (i & 2) pk[8 * c + (i >> 2)] = pack_e4m3x4(prev.x, prev.y, p0, p1);
                  prev = make_float2(p0, p1);
                } else {
                  pk[16 * c + (i >> 1)] = pack_bf16x2(p0, p1);
                }
              }
            }
          }
          tile_sum = (acc2[0].x + acc2[0].y) + (acc2[1].x + acc2[1].y);
          float xmax = fmaxf(fmaxf(xm4[0], xm4[1]), fmaxf(xm4[2], xm4[3]));
          const bool grow = attempt == 0 && (TRACK ? xmax > kRescaleThreshold : !(tile_sum <= kGrowSum));
          if (!__any_sync(0xffffffffu, grow)) break;
          if constexpr (!TRACK) {
            // the largest exponent of the tile was not tracked: one more pass over S (whole warp)
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              uint32_t sr[32];
              tmem_ld32(tS + 32 * c, sr);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (32 * c + i < limit) xmax = fmaxf(xmax, fmaf(__uint_as_float(sr[i]), sl2, -mb));
            }
          }
          // rare: re-base this row's reference, rescale what has been accumulated so far
          // (O is quiescent: the commit behind this S also covered the previous P V)
          const float alpha = grow ? ex2_approx(kShift - xmax) : 1.0f;
          if (grow) { m_ref += (xmax - kShift) / sl2; l *= alpha; }
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
        tmem_st32(tS, pk);
        if constexpr (!F8) tmem_st32(tS + 32, pk + 32);
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&p_full[X]);
      }
      if (!ok) break;
      if (!warp_wait(&o_full[X], cntO & 1, abortf, LIM)) { ok = false; break; }
      ++cntO;
      tc_fence_after();
      if (g.un.n_chunks <= 1) {
        const int slot = X == 0 ? g.un.slotA : g.un.slotB, t0 = X == 0 ? g.un.t0A : g.un.t0B;
        const int grow_ = slot * p.bl + t0 + row / p.group;
        const int head = (X == 0 ? g.kvhA : g.kvhB) * p.group + row % p.group;
        uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)grow_ * p.n_q_heads + head) * D);
        const float inv = out_scale / l;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tO + c * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 2; ++i) {              // two 32-byte stores: whole sectors
            uint32_t v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
              v[k] = pack_bf16x2(__uint_as_float(o[16 * i + 2 * k]) * inv, __uint_as_float(o[16 * i + 2 * k + 1]) * inv);
            st_global_v8(dst + c * 4 + 2 * i, v);
          }
        }
      } else {
        const size_t prow = ((size_t)(g.un.part_base + g.chunk) * 2 + X) * kTileM + row;
        p.part_ml[prow * 2 + 0] = m_ref * sl2 - kShift;     // the reference the exponentials were taken against
        p.part_ml[prow * 2 + 1] = l / out_scale;            // (the merge divides by the sum: the V scale goes in here)
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
      tc_fence_before();
    }
  }
  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abortf) {
    // A bounded wait gave up.  Nothing may still be running on this CTA's shared memory or
    // TMEM when they are handed on: (1) the MMA warp commits everything it has issued to a
    // barrier of its own and waits for it (bounded by a fixed number of polls: an MMA batch
    // takes microseconds); (2) bulk copies the producers have issued land within
    // microseconds as well, the CTA sleeps for 640 us before it leaves.
    if (tid == 0) atomicOr(p.status, FB_ST_DEV_TIMEOUT);
    if (warp == 1) {
      if (elect_one()) umma_commit(drain);
      __syncwarp();
      for (int i = 0; i < 4096 && !mbar_test(drain, 0); ++i) __nanosleep(200);
    }
    for (int i = 0; i < 64; ++i) __nanosleep(10000);
    __syncthreads();
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// Merge of the split-KV partials, chunks in index order.  A unit is cut into
// 32 pieces of 8 of its 256 rows; the CTAs of a fixed-size grid loop over
// the pieces (nothing to do, and an immediate return, when no unit was split).
// A warp takes one row at a time and keeps the loads of four chunks in flight.
constexpr int kCombineSplit = 32;        // pieces of 8 rows: one row per warp, no serial row loop
constexpr int kCombineCtasPerSm = 8;
template <int D>
__global__ void __launch_bounds__(256) attn_combine_kernel(const AttnParams p) {
  pdl_wait();
  // The attention kernel is complete: re-arm its work ticket, so that the same work list can be
  // run again (also after a launch that gave up on a bounded wait half way through its items).
  if (blockIdx.x == 0 && threadIdx.x == 0) p.hdr->ticket = 0;
  if (p.hdr->n_parts == 0) return;
  const int n_pieces = p.hdr->n_units * kCombineSplit;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int PER = D / 32;
  for (int piece = blockIdx.x; piece < n_pieces; piece += gridDim.x) {
  const AttnUnit un = p.units[piece / kCombineSplit];
  if (un.n_chunks <= 1) continue;
  const int row0 = (piece % kCombineSplit) * (2 * kTileM / kCombineSplit);
  for (int rr = row0 + warp; rr < row0 + 2 * kTileM / kCombineSplit; rr += 8) {
    const int X = rr / kTileM, row = rr % kTileM;
    const int slot = X == 0 ? un.slotA : un.slotB;
    if (slot < 0) continue;
    const int nvis = X == 0 ? un.nvisA : un.nvisB, t0 = X == 0 ? un.t0A : un.t0B;
    int nc = 0;                               // chunks that hold keys visible to this tile
    while (nc < un.n_chunks && (int)((long long)nc * un.n_tiles / un.n_chunks) < nvis) ++nc;
    const size_t prow0 = ((size_t)un.part_base * 2 + X) * kTileM + row;   // chunk c: + c * 2 * kTileM
    float M = -INFINITY;
    for (int c = lane; c < nc; c += 32) M = fmaxf(M, p.part_ml[(prow0 + (size_t)c * 2 * kTileM) * 2]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float acc[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) acc[i] = 0.f;
    float L = 0.f;
    for (int c0 = 0; c0 < nc; c0 += 4) {
      float w[4], lv[4], v[4][PER];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = min(c0 + k, nc - 1);
        const size_t prow = prow0 + (size_t)c * 2 * kTileM;
        w[k] = p.part_ml[prow * 2];
        lv[k] = p.part_ml[prow * 2 + 1];
        const float* src = p.part_o + prow * D + lane * PER;
#pragma unroll
        for (int i = 0; i < PER; ++i) v[k][i] = src[i];
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (c0 + k >= nc) break;
        const float wk = ex2_approx(w[k] - M);
        L += wk * lv[k];
#pragma unroll
        for (int i = 0; i < PER; ++i) acc[i] += wk * v[k][i];
      }
    }
    const float inv = 1.0f / L;
    const int grow_ = slot * p.bl + t0 + row / p.group;
    const int head = (X == 0 ? (un.kvh & 0xffff) : (un.kvh >> 16)) * p.group + row % p.group;
    __nv_bfloat16* dst = p.out + ((size_t)grow_ * p.n_q_heads + head) * D + lane * PER;
#pragma unroll
    for (int i = 0; i < PER; i += 2)
      *reinterpret_cast<uint32_t*>(dst + i) = pack_bf16x2(acc[i] * inv, acc[i + 1] * inv);
  }
  }
}

// ------------------------------------------------------------------- host
int ensure_device(fb_ctx* ctx) {
  int dev = 0;
  if (int e = cuda_err(ctx, cudaGetDevice(&dev), "cudaGetDevice")) return e;
  if (ctx->dev_ready && ctx->device == dev) return FB_OK;
  // first use, or the caller moved the context to another device: set up again there and
  // forget the cached tensor maps
  ctx->dev_ready = false;
  for (auto& mp : ctx->map_ptrs) mp = nullptr;
  cudaDeviceProp prop;
  if (int e = cuda_err(ctx, cudaGetDeviceProperties(&prop, dev), "cudaGetDeviceProperties")) return e;
  if (prop.major != 10) return set_err(ctx, FB_ERR_UNSUPPORTED, "the attention kernel needs an sm_100 device");
  ctx->num_sms = prop.multiProcessorCount;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (int e = cuda_err(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q),
                       "cudaGetDriverEntryPoint"))
    return e;
  if (!fn || q != cudaDriverEntryPointSuccess)
    return set_err(ctx, FB_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  ctx->encode_fn = fn;
  const int smem64 = kSmem64, smem128 = kSmem128;
  if (int e = cuda_err(ctx, cudaFuncSetAttribute(wavefront_attn_kernel<64, false>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, smem64), "smem attr"))
    return e;
  if (int e = cuda_err(ctx, cudaFuncSetAttribute(wavefront_attn_kernel<128, false>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, smem128), "smem attr"))
    return e;
  if (int e = cuda_err(ctx, cudaFuncSetAttribute(wavefront_attn_kernel<128, true>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemF8), "smem attr"))
    return e;
  if (int e = lm_head_device_setup(ctx)) return e;
  if (int e = attn_pair_device_setup(ctx)) return e;
  ctx->device = dev;
  ctx->dev_ready = true;
  return FB_OK;
}

static int encode(fb_ctx* ctx, CUtensorMap* m, const void* base, int rank, const cuuint64_t* dims,
                  const cuuint64_t* strides, const cuuint32_t* box,
                  CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16) {
  cuuint32_t es[3] = {1, 1, 1};
  auto fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(ctx->encode_fn);
  CUresult r = fn(m, dtype, rank, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return set_err(ctx, FB_ERR_CUDA, "cuTensorMapEncodeTiled failed: " + std::to_string((int)r));
  return FB_OK;
}

void fill_attn_params(fb_ctx* ctx, AttnParams& p, const int32_t* page_table, void* out, void* ws, int32_t* status,
                      int list) {
  const fb_config& c = ctx->cfg;
  uint8_t* w = static_cast<uint8_t*>(ws);
  p.hdr = reinterpret_cast<SchedHeader*>(w + ctx->ws.l[list].header);
  p.items = reinterpret_cast<const AttnItem*>(w + ctx->ws.l[list].items);
  p.units = reinterpret_cast<const AttnUnit*>(w + ctx->ws.l[list].units);
  p.page_table = page_table;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.part_ml = reinterpret_cast<float*>(w + ctx->ws.l[list].part_ml);
  p.part_o = reinterpret_cast<float*>(w + ctx->ws.l[list].part_o);
  p.status = status;
  p.bl = c.block_len; p.n_q_heads = c.n_q_heads; p.n_kv_heads = c.n_kv_heads; p.group = ctx->group;
  p.max_pages_per_req = c.max_pages_per_req; p.num_pages = c.num_pages;
  p.resident = c.window_in_pages;
  p.k_scale = nullptr; p.v_scale = nullptr;
  p.scale_log2 = ctx->sm_scale * kLog2eF;
  p.wait_cycles = ctx->wait_cycles;
}

int launch_attn_combine(fb_ctx* ctx, const AttnParams& p, int list, cudaStream_t stream) {
  const int grid = min(max(ctx->ws.l[list].max_units, 1) * kCombineSplit, kCombineCtasPerSm * ctx->num_sms);
  if (ctx->cfg.head_dim == 64)
    return cuda_err(ctx, launch_pdl(attn_combine_kernel<64>, grid, 256, 0, stream, p), "attn_combine_kernel launch");
  return cuda_err(ctx, launch_pdl(attn_combine_kernel<128>, grid, 256, 0, stream, p), "attn_combine_kernel launch");
}

static int encode_q(fb_ctx* ctx, const void* q) {
  const fb_config& c = ctx->cfg;
  const cuuint64_t rows = (cuuint64_t)c.max_requests * c.wmax * c.block_len, D = c.head_dim;
  cuuint64_t dims[3] = {D, (cuuint64_t)c.n_q_heads, rows};
  cuuint64_t str[2] = {D * 2, (cuuint64_t)c.n_q_heads * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)ctx->group, (cuuint32_t)ctx->tokens_per_tile};
  return encode(ctx, &ctx->tm_q, q, 3, dims, str, box);
}

int launch_attn(fb_ctx* ctx, const fb_pack* pk, const void* q, const void* k_win, const void* v_win,
                const void* k_pool, const void* v_pool, const int32_t* page_table, void* out, void* ws,
                int32_t* status, cudaStream_t stream) {
  (void)pk;
  if (int e = ensure_device(ctx)) return e;
  const fb_config& c = ctx->cfg;
  const cuuint64_t rows = (cuuint64_t)c.max_requests * c.wmax * c.block_len;
  const cuuint64_t D = c.head_dim;
  const void* ptrs[5] = {q, k_win, v_win, k_pool, v_pool};
  if (ctx->maps_f8 || memcmp(ptrs, ctx->map_ptrs, sizeof(ptrs)) != 0) {
    if (int e = encode_q(ctx, q)) return e;
    {
      cuuint64_t dims[3] = {D, (cuuint64_t)c.n_kv_heads, rows};
      cuuint64_t str[2] = {D * 2, (cuuint64_t)c.n_kv_heads * D * 2};
      cuuint32_t box[3] = {64, 1, 128};
      // window resident in the pages: no window tensors; the two maps are never used then
      if (int e = encode(ctx, &ctx->tm_kwin, k_win ? k_win : k_pool, 3, dims, str, box)) return e;
      if (int e = encode(ctx, &ctx->tm_vwin, v_win ? v_win : v_pool, 3, dims, str, box)) return e;
      cuuint32_t half[3] = {64, 1, 64};       // the CTA-pair kernel: each CTA takes 64 of a tile's 128 window keys
      if (int e = encode(ctx, &ctx->tm_kwin_half, k_win ? k_win : k_pool, 3, dims, str, half)) return e;
    }
    {
      cuuint64_t dims[2] = {D, (cuuint64_t)c.num_pages * c.n_kv_heads * kPage};
      cuuint64_t str[1] = {D * 2};
      cuuint32_t box[2] = {64, 64};
      if (int e = encode(ctx, &ctx->tm_kpool, k_pool, 2, dims, str, box)) return e;
      if (int e = encode(ctx, &ctx->tm_vpool, v_pool, 2, dims, str, box)) return e;
    }
    memcpy(ctx->map_ptrs, ptrs, sizeof(ptrs));
    ctx->maps_f8 = false;
  }
  AttnParams p;
  fill_attn_params(ctx, p, page_table, out, ws, status, 0);
  const int grid = ctx->num_sms;
  if (c.head_dim == 64) {
    if (int e = cuda_err(ctx, launch_pdl(wavefront_attn_kernel<64, false>, grid, kAttnThreads, kSmem64, stream, ctx->tm_q,
                                         ctx->tm_kwin, ctx->tm_vwin, ctx->tm_kpool, ctx->tm_vpool, p),
                         "wavefront_attn_kernel launch"))
      return e;
    return launch_attn_combine(ctx, p, 0, stream);
  }
  // quads first (the CTA-pair kernel), then everything else
  if (ctx->pair_on)
    if (int e = launch_attn_pair(ctx, page_table, out, ws, status, stream)) return e;
  if (int e = cuda_err(ctx, launch_pdl(wavefront_attn_kernel<128, false>, grid, kAttnThreads, kSmem128, stream, ctx->tm_q,
                                       ctx->tm_kwin, ctx->tm_vwin, ctx->tm_kpool, ctx->tm_vpool, p),
                       "wavefront_attn_kernel launch"))
    return e;
  return launch_attn_combine(ctx, p, 0, stream);
}

// Attention over 8-bit pages (window resident in the pages, head_dim 128): the pools are E4M3
// bytes, one (page, KV head) is a 64 x 128-byte tile = one TMA box.
int launch_attn_fp8(fb_ctx* ctx, const fb_pack* pk, const void* q, const void* k_pool8, const void* v_pool8,
                    const float* k_scale, const float* v_scale, const int32_t* page_table, void* out, void* ws,
                    int32_t* status, cudaStream_t stream) {
  (void)pk;
  if (int e = ensure_device(ctx)) return e;
  const fb_config& c = ctx->cfg;
  const void* ptrs[5] = {q, nullptr, nullptr, k_pool8, v_pool8};
  if (!ctx->maps_f8 || memcmp(ptrs, ctx->map_ptrs, sizeof(ptrs)) != 0) {
    if (int e = encode_q(ctx, q)) return e;
    cuuint64_t dims[2] = {128, (cuuint64_t)c.num_pages * c.n_kv_heads * kPage};
    cuuint64_t str[1] = {128};
    cuuint32_t box[2] = {128, 64};
    if (int e = encode(ctx, &ctx->tm_kpool, k_pool8, 2, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_UINT8)) return e;
    if (int e = encode(ctx, &ctx->tm_vpool, v_pool8, 2, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_UINT8)) return e;
    ctx->tm_kwin = ctx->tm_kpool; ctx->tm_vwin = ctx->tm_vpool;        // never used: every key tile is a paged one
    memcpy(ctx->map_ptrs, ptrs, sizeof(ptrs));
    ctx->maps_f8 = true;
  }
  AttnParams p;
  fill_attn_params(ctx, p, page_table, out, ws, status, 0);
  p.k_scale = k_scale; p.v_scale = v_scale;
  if (int e = cuda_err(ctx, launch_pdl(wavefront_attn_kernel<128, true>, ctx->num_sms, kAttnThreads, (size_t)kSmemF8, stream,
                                       ctx->tm_q, ctx->tm_kwin, ctx->tm_vwin, ctx->tm_kpool, ctx->tm_vpool, p),
                       "wavefront_attn_kernel (8-bit pages) launch"))
    return e;
  return launch_attn_combine(ctx, p, 0, stream);
}

}  // namespace fb
