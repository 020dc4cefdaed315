// fb_pack_wavefronts: Heterogeneous Wavefront Packing (Sec. 3.2, Eq. 4).
//
// One launch.  Blocks 0..nb-1 compact the live blocks of all decoding
// requests into slots and gather tokens / position ids; the last two blocks
// build the two attention work lists (units, key-axis chunks, longest first)
// from the same per-request state: list 0 for the one-CTA kernel, list 1 (four
// Q tiles of one request and KV head at a time) for the CTA-pair kernel.
// Everything is integer work on a few KB.
#include "fb_common.cuh"

namespace fb {

constexpr int kPackThreads = 1024;
constexpr int kSlotsPerBlock = 32;
constexpr int kCostBins = 1024;

struct PackParams {
  const int32_t *active, *prefix_len, *L, *R, *tokens;
  int32_t *n_live, *slot_req, *slot_s, *slot_pos0, *slot_kv_len, *slot_flags, *req_slot_begin, *qtok, *pos;
  int32_t* status;
  SchedHeader* hdr[2];
  AttnItem* items[2];
  AttnUnit* units[2];
  int32_t max_items[2], max_units[2], max_parts[2], target_items[2];
  int32_t pair_on;
  int32_t max_requests, wmax, bl, max_slots, max_blocks, mask_id, n_kv_heads;
  int32_t tiles_per_slot, tokens_per_tile, min_chunk_tiles;
  int32_t resident;   // window K/V live in the pages: key tiles follow absolute positions
  int32_t n_gather_blocks;
};

// live-block count of request r, sanitised to [0, wmax]
__device__ __forceinline__ int live_blocks(const PackParams& p, int r, int32_t* status) {
  if (p.active[r] != 1) return 0;
  const int L = p.L[r], R = p.R[r];
  int w = R - L;
  if (L < 0 || R > p.max_blocks || w < 0 || w > p.wmax) {
    if (status) atomicOr(status, FB_ST_BAD_STATE);
    w = w < 0 ? 0 : (w > p.wmax ? p.wmax : w);
    if (L < 0 || L + w > p.max_blocks) w = 0;
  }
  return w;
}

// exclusive block scan of one value per thread; returns the exclusive prefix,
// *total = block sum.  All threads must call.
__device__ __forceinline__ int block_excl_scan(int v, int* total, int* sh /*[kPackThreads/32 + 1]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();
  if (lane == 31) sh[warp] = x;
  __syncthreads();
  if (warp == 0) {
    int w = lane < kPackThreads / 32 ? sh[lane] : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += y;
    }
    if (lane < kPackThreads / 32) sh[lane] = w;   // inclusive warp sums
  }
  __syncthreads();
  const int base = warp == 0 ? 0 : sh[warp - 1];
  *total = sh[kPackThreads / 32 - 1];
  return base + x - v;
}

// Sort key of a work item: its key-tile iterations; an iteration with two Q
// tiles takes about 7/6 of one with a single tile (measured).
__device__ __forceinline__ int item_cost(int nA, int nB) {
  const int n = max(nA, nB), both = min(nA, nB);
  return (6 * n + both + 1) >> 1;
}

__device__ __forceinline__ ReqGeom geom_of(const PackParams& p, int w, int prefix_len, int list) {
  return req_geom_of(w, prefix_len, p.tiles_per_slot, p.bl, p.n_kv_heads, p.resident, list, p.pair_on);
}
__device__ __forceinline__ ReqGeom req_geom(const PackParams& p, int r, int32_t* status, int list) {
  const int w = live_blocks(p, r, status);
  return geom_of(p, w, w ? p.prefix_len[r] : 0, list);
}

// unit record of two Q tiles qa, qb (absolute tile indices of the request; qb < 0: none) under
// KV heads hA, hB
__device__ __forceinline__ AttnUnit make_unit(const PackParams& p, const ReqGeom& q, int req, int first, int qa, int qb,
                                              int hA, int hB) {
  AttnUnit un;
  un.req = req;
  un.kvh = hA | (hB << 16);
  const int sA = qa / p.tiles_per_slot;
  un.slotA = first + sA;
  un.t0A = (qa % p.tiles_per_slot) * p.tokens_per_tile;
  un.winA = (sA + 1) * p.bl;
  un.nvisA = p.resident ? (q.P + un.winA + kTileN - 1) / kTileN : q.npt + (un.winA + kTileN - 1) / kTileN;
  if (qb >= 0) {
    const int sB = qb / p.tiles_per_slot;
    un.slotB = first + sB;
    un.t0B = (qb % p.tiles_per_slot) * p.tokens_per_tile;
    un.winB = (sB + 1) * p.bl;
    un.nvisB = p.resident ? (q.P + un.winB + kTileN - 1) / kTileN : q.npt + (un.winB + kTileN - 1) / kTileN;
  } else {
    un.slotB = -1; un.t0B = 0; un.winB = 0; un.nvisB = 0;
  }
  un.n_tiles = q.nt; un.n_chunks = 0; un.part_base = -1;
  un.prefix_len = q.P; un.npt = q.npt; un.win_row0 = first * p.bl;
  return un;
}

// `list` 0: pairs of tiles and leftover tiles, one record per scheduling unit.  `list` 1: quads,
// two records per scheduling unit (2u for the first CTA of the pair, 2u + 1 for the second), both
// cut into the same chunks; an item names record 2u.
__device__ void build_sched(const PackParams& p, const int list) {
  const int mult = list + 1;            // unit records (and partial-result ranges) per scheduling unit
  SchedHeader* const hdr = p.hdr[list];
  AttnItem* const items = p.items[list];
  AttnUnit* const units = p.units[list];
  const int max_items = p.max_items[list], max_units = p.max_units[list], max_parts = p.max_parts[list];
  __shared__ int sh_scan[kPackThreads / 32 + 1];
  __shared__ int bins[kCostBins];
  __shared__ int sh_total, sh_units;
  __shared__ SplitRule sh_rule;
  const int tid = threadIdx.x;
  // bad states are reported once, by the gather blocks (null status here)
  // phase 1: total key-tile work -> chunk length
  int mine = 0, mine_units = 0;
  for (int r = tid; r < p.max_requests; r += kPackThreads) {
    ReqGeom g = req_geom(p, r, nullptr, list);
    mine += g.nunits * g.nt;
    mine_units += g.nt ? g.nunits : 0;
  }
  if (tid == 0) { sh_total = 0; sh_units = 0; }
  for (int i = tid; i < kCostBins; i += kPackThreads) bins[i] = 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mine += __shfl_xor_sync(0xffffffffu, mine, o);
    mine_units += __shfl_xor_sync(0xffffffffu, mine_units, o);
  }
  __syncthreads();
  if ((tid & 31) == 0) { atomicAdd(&sh_total, mine); atomicAdd(&sh_units, mine_units); }
  __syncthreads();
  if (tid == 0) sh_rule = split_rule(sh_total, sh_units, p.target_items[list], p.min_chunk_tiles);
  __syncthreads();
  const SplitRule rule = sh_rule;
  // phase 2 + 3: per-request bases (chunked scan), then one thread per unit of the chunk's
  // requests: unit record, cost histogram of its items
  __shared__ int s_ub[kPackThreads + 1], s_pb[kPackThreads], s_first[kPackThreads], s_wb[kPackThreads],
      s_w[kPackThreads], s_P[kPackThreads];
  int unit_run = 0, part_run = 0, item_run = 0, slot_run = 0, work_run = 0;
  for (int r0 = 0; r0 < p.max_requests; r0 += kPackThreads) {
    const int r = r0 + tid;
    ReqGeom g{};
    int nunits = 0;
    if (r < p.max_requests) {
      g = req_geom(p, r, nullptr, list);
      nunits = g.nt ? g.nunits : 0;
    }
    int tu, tp, ti, ts, tw;
    const int wbase = work_run + block_excl_scan(nunits * g.nt, &tw, sh_scan);
    work_run += tw;
    const ReqSplit rs = req_split(rule, wbase, nunits, g.nt);
    const int urel = block_excl_scan(nunits, &tu, sh_scan);
    const int pbase = part_run + block_excl_scan(rs.parts(nunits), &tp, sh_scan);
    block_excl_scan(rs.items(nunits), &ti, sh_scan);
    const int first0 = slot_run + block_excl_scan(g.w, &ts, sh_scan);  // first slot of the request
    s_ub[tid] = urel; s_pb[tid] = pbase; s_first[tid] = first0; s_wb[tid] = wbase; s_w[tid] = g.w; s_P[tid] = g.P;
    if (tid == 0) s_ub[kPackThreads] = tu;
    __syncthreads();
    for (int i = tid; i < tu; i += kPackThreads) {
      // the request of unit i: the last k with s_ub[k] <= i (requests without units share
      // their successor's base and are skipped by "last")
      int lo = 0, hi = kPackThreads - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (s_ub[mid] <= i) lo = mid; else hi = mid - 1;
      }
      const int k = lo, ul = i - s_ub[k];
      const int u = unit_run + i;
      if (mult * (u + 1) > max_units) continue;
      const ReqGeom q = geom_of(p, s_w[k], s_P[k], list);
      const ReqSplit qs = req_split(rule, s_wb[k], q.nunits, q.nt);
      const int first = s_first[k], nc = qs.chunks(ul);
      AttnUnit un[2];
      if (list == 0) {
        // Full pairs first, numbered h * nfull + pr: the pairs of one (request, KV head) are
        // adjacent, are handed out back to back and so share their K/V through L2.  Then the
        // leftover tile, one unit per two KV heads.
        const bool full = ul < q.nfull * p.n_kv_heads;
        const int h = full ? ul / q.nfull : 2 * (ul - q.nfull * p.n_kv_heads);
        const int qa = q.tile0 + (full ? 2 * (ul % q.nfull) : q.ntq - 1);
        if (full) un[0] = make_unit(p, q, r0 + k, first, qa, qa + 1, h, h);
        else if (h + 1 < p.n_kv_heads) un[0] = make_unit(p, q, r0 + k, first, qa, qa, h, h + 1);
        else un[0] = make_unit(p, q, r0 + k, first, qa, -1, h, h);
      } else {
        // quad qd of KV head h: tiles 4 qd + r and 4 qd + 2 + r belong to CTA r of the pair
        const int h = ul / q.nquad, qd = ul % q.nquad;
        un[0] = make_unit(p, q, r0 + k, first, 4 * qd, 4 * qd + 2, h, h);
        un[1] = make_unit(p, q, r0 + k, first, 4 * qd + 1, 4 * qd + 3, h, h);
      }
      int nch = nc;
      const int pb = nc > 1 ? mult * (s_pb[k] + qs.part_off(ul)) : -1;
      // the workspace is sized for the bound on the split pieces (split_rule); a unit that
      // would still fall outside it is dropped and FB_ST_BAD_STATE is raised below
      if (nc > 1 && pb + mult * nc > max_parts) nch = 0;
      int nvA = 0, nvB = 0;
      for (int rr = 0; rr < mult; ++rr) {
        un[rr].n_chunks = nch;
        un[rr].part_base = nc > 1 ? pb + rr * nc : -1;
        units[mult * u + rr] = un[rr];
        nvA = max(nvA, un[rr].nvisA); nvB = max(nvB, un[rr].nvisB);
      }
      for (int c = 0; c < nch; ++c) {
        const int jb = c * q.nt / nc, je = (c + 1) * q.nt / nc;
        int cost = item_cost(max(0, min(je, nvA) - jb), max(0, min(je, nvB) - jb));
        atomicAdd(&bins[min(cost, kCostBins - 1)], 1);
      }
    }
    unit_run += tu; part_run += tp; item_run += ti; slot_run += ts;
    __syncthreads();                      // the chunk's tables are overwritten next
  }
  __syncthreads();
  // descending exclusive offsets over the cost bins: thread t owns the bins
  // kCostBins-1-kBinsPer*t and below (largest cost first)
  {
    constexpr int kBinsPer = kCostBins / kPackThreads;
    static_assert(kBinsPer * kPackThreads == kCostBins && kBinsPer >= 1, "whole bins per thread");
    int c[kBinsPer], sum = 0;
#pragma unroll
    for (int j = 0; j < kBinsPer; ++j) { c[j] = bins[kCostBins - 1 - (kBinsPer * tid + j)]; sum += c[j]; }
    int total_items;
    int base = block_excl_scan(sum, &total_items, sh_scan);
#pragma unroll
    for (int j = 0; j < kBinsPer; ++j) { bins[kCostBins - 1 - (kBinsPer * tid + j)] = base; base += c[j]; }
    if (tid == 0) {
      hdr->n_items = min(total_items, max_items);
      hdr->n_units = min(mult * unit_run, max_units);
      hdr->chunk_tiles = rule.ct;
      hdr->n_parts = mult * part_run;
      hdr->total_tiles = sh_total;
      hdr->ticket = 0; hdr->done = 0;
      if (total_items > max_items || mult * unit_run > max_units || mult * part_run > max_parts)
        atomicOr(p.status, FB_ST_BAD_STATE);
    }
  }
  __syncthreads();
  // phase 4: scatter items, longest first
  for (int u = tid; u < min(unit_run, max_units / mult); u += kPackThreads) {
    const AttnUnit un = units[mult * u];
    int nvA = un.nvisA, nvB = un.nvisB;
    if (mult == 2) { const AttnUnit u1 = units[2 * u + 1]; nvA = max(nvA, u1.nvisA); nvB = max(nvB, u1.nvisB); }
    const int nch = un.n_chunks;
    for (int c = 0; c < nch; ++c) {
      const int jb = c * un.n_tiles / nch, je = (c + 1) * un.n_tiles / nch;
      int cost = item_cost(max(0, min(je, nvA) - jb), max(0, min(je, nvB) - jb));
      const int at = atomicAdd(&bins[min(cost, kCostBins - 1)], 1);
      if (at < max_items) {
        AttnItem it; it.unit = mult * u; it.chunk = c; it.jb = jb; it.je = je;
        items[at] = it;
      }
    }
  }
}

__global__ void __launch_bounds__(kPackThreads) pack_kernel(const PackParams p) {
  pdl_wait();
  if ((int)blockIdx.x >= p.n_gather_blocks) { build_sched(p, (int)blockIdx.x - p.n_gather_blocks); return; }
  __shared__ int sh_scan[kPackThreads / 32 + 1];
  __shared__ int s_req[kSlotsPerBlock], s_idx[kSlotsPerBlock], s_w[kSlotsPerBlock];
  const int tid = threadIdx.x;
  const int slot0 = blockIdx.x * kSlotsPerBlock;
  if (tid < kSlotsPerBlock) s_req[tid] = -1;
  __syncthreads();
  int run = 0;
  for (int r0 = 0; r0 < p.max_requests; r0 += kPackThreads) {
    const int r = r0 + tid;
    const int w = r < p.max_requests ? live_blocks(p, r, p.status) : 0;
    int tot;
    const int begin = run + block_excl_scan(w, &tot, sh_scan);
    run += tot;
    if (r < p.max_requests) {
      if (blockIdx.x == 0) p.req_slot_begin[r] = begin;
      for (int s = 0; s < w; ++s) {
        const int slot = begin + s;
        if (slot >= slot0 && slot < slot0 + kSlotsPerBlock) {
          s_req[slot - slot0] = r; s_idx[slot - slot0] = s; s_w[slot - slot0] = w;
        }
      }
    }
  }
  if (blockIdx.x == 0 && tid == 0) { p.req_slot_begin[p.max_requests] = run; *p.n_live = run; }
  __syncthreads();
  // all slots of this block at once: one thread per (slot, token)
  for (int i = tid; i < kSlotsPerBlock * p.bl; i += kPackThreads) {
    const int k = i / p.bl, t = i % p.bl;
    const int slot = slot0 + k;
    if (slot >= p.max_slots) break;
    const int r = s_req[k];
    if (r < 0) {
      if (t == 0) {
        p.slot_req[slot] = -1; p.slot_s[slot] = 0; p.slot_pos0[slot] = 0; p.slot_kv_len[slot] = 0;
        p.slot_flags[slot] = 0;
      }
      p.qtok[slot * p.bl + t] = p.mask_id; p.pos[slot * p.bl + t] = 0;
      continue;
    }
    const int s = s_idx[k], w = s_w[k];
    const int P = p.prefix_len[r], g = p.L[r] + s;
    const int pos0 = P + s * p.bl;
    if (t == 0) {
      p.slot_req[slot] = r; p.slot_s[slot] = s; p.slot_pos0[slot] = pos0;
      p.slot_kv_len[slot] = P + (s + 1) * p.bl;
      p.slot_flags[slot] = (s == 0 ? FB_FLAG_OLDEST : 0) | (s == w - 1 ? FB_FLAG_FRONTIER : 0);
    }
    p.qtok[slot * p.bl + t] = p.tokens[(size_t)r * p.max_blocks * p.bl + (size_t)g * p.bl + t];  // Eq. 4: qtok = x[b, o_b + ...]
    p.pos[slot * p.bl + t] = pos0 + t;                                                           //        pos  = o_b + ...
  }
}

int launch_pack(fb_ctx* ctx, const fb_state* st, const fb_pack* out, void* ws, int32_t* status,
                cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  PackParams p;
  p.active = st->active; p.prefix_len = st->prefix_len; p.L = st->L; p.R = st->R; p.tokens = st->tokens;
  p.n_live = out->n_live; p.slot_req = out->slot_req; p.slot_s = out->slot_s; p.slot_pos0 = out->slot_pos0;
  p.slot_kv_len = out->slot_kv_len; p.slot_flags = out->slot_flags; p.req_slot_begin = out->req_slot_begin;
  p.qtok = out->qtok; p.pos = out->pos; p.status = status;
  uint8_t* w = static_cast<uint8_t*>(ws);
  for (int l = 0; l < 2; ++l) {
    p.hdr[l] = reinterpret_cast<SchedHeader*>(w + ctx->ws.l[l].header);
    p.items[l] = reinterpret_cast<AttnItem*>(w + ctx->ws.l[l].items);
    p.units[l] = reinterpret_cast<AttnUnit*>(w + ctx->ws.l[l].units);
    p.max_items[l] = ctx->ws.l[l].max_items; p.max_units[l] = ctx->ws.l[l].max_units;
    p.max_parts[l] = ctx->ws.l[l].max_parts;
  }
  p.target_items[0] = ctx->target_items;
  p.target_items[1] = ctx->target_items > 1 ? ctx->target_items / 2 : 1;
  p.pair_on = ctx->pair_on;
  p.max_requests = c.max_requests; p.wmax = c.wmax; p.bl = c.block_len;
  p.max_slots = c.max_requests * c.wmax; p.max_blocks = c.max_blocks; p.mask_id = c.mask_id;
  p.n_kv_heads = c.n_kv_heads; p.tiles_per_slot = ctx->tiles_per_slot;
  p.tokens_per_tile = ctx->tokens_per_tile;
  p.min_chunk_tiles = ctx->min_chunk_tiles;
  p.resident = ctx->cfg.window_in_pages;
  p.n_gather_blocks = (p.max_slots + kSlotsPerBlock - 1) / kSlotsPerBlock;
  // one more block per work list in use (the CTA-pair kernel's list only when that kernel is on)
  return cuda_err(ctx, launch_pdl(pack_kernel, p.n_gather_blocks + 1 + (p.pair_on ? 1 : 0), kPackThreads, 0, stream, p),
                  "pack_kernel launch");
}

}  // namespace fb
