// fb_gate_commit: in-order retirement with KV freeze and readiness-gated
// admission (Alg. 1 lines 7-12, Eq. 2-3, Eq. 6 for the committing block).
//
// One CTA per request.  Thread 0 evaluates the block-level predicates from
// the per-slot counts; all threads then copy the retiring blocks' window K/V
// rows into the request's pages with 16-byte accesses; thread 0 publishes the
// new state.  Requests are independent, so no inter-CTA ordering is needed;
// the step counters are integer atomics on a zeroed array.  The batch-synchronous
// variant (fb_config.batch_sync) adds a single-CTA kernel in front that reduces the
// per-request results over the batch into two of the counters, which every CTA here reads.
#include "fb_common.cuh"

namespace fb {

constexpr int kGateThreads = 512;

struct GateParams {
  const int32_t *n_live, *req_slot_begin, *slot_stats;
  int32_t *active, *prefix_len, *L, *R, *tokens;
  uint8_t* pe_done;
  const int32_t* page_table;
  const uint4 *k_win, *v_win;
  uint4 *k_pool, *v_pool;
  int32_t* n_committed;
  uint8_t* spawned;
  int32_t *counters, *status;
  int32_t max_requests, wmax, bl, max_blocks, mask_id, s_pe, n_kv_heads, head_dim, num_pages,
      max_pages_per_req;
  float theta_spawn;
  int32_t batch_sync;
};

// What a request's own block counts say (Alg. 1 l.7-9 before any batch rule): its window,
// the post-edit counters after this forward, the finished prefix c (stopping after a block
// that holds EOS), and whether retiring those c blocks ends the request.
struct ReqEval {
  int first, w, L, R, c;
  bool ok, eos, ends;
  uint8_t pe_new[8];
  int m2t, t2t;
};
__device__ __forceinline__ ReqEval eval_request(const GateParams& p, int r) {
  ReqEval e;
  e.first = p.req_slot_begin[r];
  e.w = p.req_slot_begin[r + 1] - e.first;
  e.L = p.L[r]; e.R = p.R[r];
  e.c = 0; e.eos = false; e.ends = false; e.m2t = 0; e.t2t = 0;
  e.ok = !(e.w != e.R - e.L || e.w < 0 || e.w > p.wmax);
  if (!e.ok) return e;
  bool fin[8];
  for (int s = 0; s < e.w; ++s) {
    const int32_t* st = p.slot_stats + (e.first + s) * FB_SLOT_STATS;
    const int m0 = st[FB_STAT_M0], m1 = st[FB_STAT_M1], nupd = st[FB_STAT_M2T] + st[FB_STAT_T2T];
    int pn = p.pe_done[r * p.wmax + s] + (m0 == 0 ? 1 : 0);
    pn = pn > 255 ? 255 : pn;
    e.pe_new[s] = (uint8_t)pn;
    // locally finished (Sec. 2.1): no masks left, and either a quiet
    // post-edit forward or the S_pe budget is used up
    fin[s] = m1 == 0 && ((m0 == 0 && nupd == 0) || pn >= p.s_pe);
    e.m2t += st[FB_STAT_M2T]; e.t2t += st[FB_STAT_T2T];
  }
  while (e.c < e.w && fin[e.c]) {                    // Alg. 1 l.7-9, in order
    ++e.c;
    if (p.slot_stats[(e.first + e.c - 1) * FB_SLOT_STATS + FB_STAT_EOS]) { e.eos = true; break; }
  }
  e.ends = e.eos || e.L + e.c == p.max_blocks;
  return e;
}
// Eq. 2 on the frontier block as it went into this forward; Eq. 3 with the window bounds
// after c blocks have retired
__device__ __forceinline__ bool clears_gate(const GateParams& p, const ReqEval& e, int c) {
  float rho = 1.0f;
  if (e.w > 0) {
    const int32_t* st = p.slot_stats + (e.first + e.w - 1) * FB_SLOT_STATS;
    if (st[FB_STAT_M0] != 0) rho = __fdiv_rn((float)st[FB_STAT_RDY], (float)st[FB_STAT_M0]);
  }
  return rho >= p.theta_spawn && e.R - (e.L + c) < p.wmax && e.R < p.max_blocks;
}

// batch_sync: the two reductions over the decoding sequences (Sec. 3.2: finished.all(),
// min_b rho_b), one CTA, before any state is touched.  A sequence that ends with its own
// finished prefix never holds the others back beyond it; if every sequence ends, each
// retires its own prefix.
__global__ void __launch_bounds__(kGateThreads) gate_batch_reduce_kernel(const GateParams p) {
  pdl_wait();
  __shared__ int s_min, s_max, s_all;
  if (threadIdx.x == 0) { s_min = 0x7fffffff; s_max = 0; s_all = 1; }
  __syncthreads();
  for (int r = threadIdx.x; r < p.max_requests; r += kGateThreads) {
    if (p.active[r] != 1) continue;
    const ReqEval e = eval_request(p, r);
    if (!e.ok) { atomicMin(&s_min, 0); continue; }   // pack and state disagree: nothing retires
    if (e.ends) atomicMax(&s_max, e.c); else atomicMin(&s_min, e.c);
  }
  __syncthreads();
  const int C = s_min != 0x7fffffff ? s_min : s_max;
  int left = 0;
  for (int r = threadIdx.x; r < p.max_requests; r += kGateThreads) {
    if (p.active[r] != 1) continue;
    const ReqEval e = eval_request(p, r);
    if (!e.ok) { atomicAnd(&s_all, 0); continue; }
    const int c = min(e.c, C);
    if (e.ends && c == e.c) continue;                // done: no longer part of the batch
    left = 1;
    if (!clears_gate(p, e, c)) atomicAnd(&s_all, 0);
  }
  const int any_left = __syncthreads_or(left);
  if (threadIdx.x == 0) {
    p.counters[FB_CT_LOCKSTEP_COMMIT] = C;
    p.counters[FB_CT_LOCKSTEP_ADMIT] = any_left && s_all;
  }
}

__global__ void __launch_bounds__(kGateThreads) gate_commit_kernel(const GateParams p) {
  pdl_wait();
  const int r = blockIdx.x;
  const int tid = threadIdx.x;
  __shared__ int s_c, s_first, s_P, s_done, s_spawn, s_newR;
  if (r == 0 && tid == 0) atomicAdd(&p.counters[FB_CT_LIVE_SLOTS], *p.n_live);
  if (p.active[r] != 1) {
    if (tid == 0) { p.n_committed[r] = 0; p.spawned[r] = 0; }
    return;
  }
  if (tid == 0) {
    const ReqEval e = eval_request(p, r);
    if (!e.ok) {                                   // pack and state disagree: leave the request alone
      atomicOr(p.status, FB_ST_BAD_STATE);
      s_c = 0; s_spawn = 0; s_first = e.first; s_P = 0; s_newR = e.R;
      p.n_committed[r] = 0; p.spawned[r] = 0;
    } else {
      // batch_sync: the batch's retire count caps the sequence's own; a block holding EOS
      // terminates only if it is among the blocks that do retire
      const int c = p.batch_sync ? min(e.c, p.counters[FB_CT_LOCKSTEP_COMMIT]) : e.c;
      const int w = e.w, R = e.R, L = e.L + c;
      const int P = p.prefix_len[r];
      s_c = c; s_first = e.first; s_P = P;
      for (int s = 0; s < p.wmax; ++s) p.pe_done[r * p.wmax + s] = s + c < w ? e.pe_new[s + c] : 0;
      const bool done = (c == e.c && e.eos) || L == p.max_blocks;
      int spawn = 0;
      if (!done) spawn = p.batch_sync ? p.counters[FB_CT_LOCKSTEP_ADMIT] : (int)clears_gate(p, e, c);
      s_done = done; s_spawn = spawn; s_newR = R;
      p.L[r] = L;
      p.prefix_len[r] = P + c * p.bl;
      p.n_committed[r] = c;
      p.spawned[r] = (uint8_t)spawn;
      if (done) p.active[r] = 2;
      if (spawn) {
        p.R[r] = R + 1;
        p.pe_done[r * p.wmax + (R + 1 - L) - 1] = 0;
      }
      if (c) { atomicAdd(&p.counters[FB_CT_BLOCKS], c); atomicAdd(&p.counters[FB_CT_TOKENS], c * p.bl); }
      if (spawn) atomicAdd(&p.counters[FB_CT_SPAWNED], 1);
      if (done) atomicAdd(&p.counters[FB_CT_FINISHED], 1); else atomicAdd(&p.counters[FB_CT_ACTIVE], 1);
      if (e.m2t) atomicAdd(&p.counters[FB_CT_M2T], e.m2t);
      if (e.t2t) atomicAdd(&p.counters[FB_CT_T2T], e.t2t);
    }
  }
  __syncthreads();
  // freeze KV of the retiring blocks: window rows -> absolute positions
  const int c = s_c, first = s_first, P = s_P;
  const int vec_per_head = p.head_dim / 8;                 // uint4 per (token, head)
  const int vec_per_tok = p.n_kv_heads * vec_per_head;
  // (window resident in the pages: nothing to copy, the prefix pointer has moved over it)
  const int total = p.k_win ? c * p.bl * vec_per_tok : 0;
  // four pieces per thread and pass, all loads issued before the first store (source and
  // destination never overlap: window tensors against the page pool)
  constexpr int kBatch = 4;
  for (int i0 = tid; i0 < total; i0 += kBatch * kGateThreads) {
    uint4 kv[kBatch], vv[kBatch];
    size_t dst[kBatch];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      const int i = i0 + j * kGateThreads;
      dst[j] = ~(size_t)0;
      if (i >= total) continue;
      const int tok = i / vec_per_tok, rem = i % vec_per_tok;
      const int h = rem / vec_per_head, v = rem % vec_per_head;
      const int apos = P + tok;
      const int pidx = apos / kPage;
      if (pidx >= p.max_pages_per_req) { atomicOr(p.status, FB_ST_BAD_PAGE); continue; }
      const int page = p.page_table[r * p.max_pages_per_req + pidx];
      if (page < 0 || page >= p.num_pages) { atomicOr(p.status, FB_ST_BAD_PAGE); continue; }
      const size_t src = (size_t)(first * p.bl + tok) * vec_per_tok + rem;
      dst[j] = (((size_t)page * p.n_kv_heads + h) * kPage + apos % kPage) * vec_per_head + v;
      kv[j] = p.k_win[src];
      vv[j] = p.v_win[src];
    }
#pragma unroll
    for (int j = 0; j < kBatch; ++j)
      if (dst[j] != ~(size_t)0) { p.k_pool[dst[j]] = kv[j]; p.v_pool[dst[j]] = vv[j]; }
  }
  // the admitted block starts fully masked
  if (s_spawn) {
    int32_t* nb = p.tokens + (size_t)r * p.max_blocks * p.bl + (size_t)s_newR * p.bl;
    for (int t = tid; t < p.bl; t += kGateThreads) nb[t] = p.mask_id;
  }
}

int launch_gate(fb_ctx* ctx, const fb_pack* pk, const int32_t* slot_stats, const fb_state* st,
                const void* k_win, const void* v_win, void* k_pool, void* v_pool, int32_t* n_committed,
                uint8_t* spawned, int32_t* step_counters, int32_t* status, cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  GateParams p;
  p.n_live = pk->n_live; p.req_slot_begin = pk->req_slot_begin; p.slot_stats = slot_stats;
  p.active = st->active; p.prefix_len = st->prefix_len; p.L = st->L; p.R = st->R; p.tokens = st->tokens;
  p.pe_done = st->pe_done; p.page_table = st->page_table;
  p.k_win = static_cast<const uint4*>(k_win); p.v_win = static_cast<const uint4*>(v_win);
  p.k_pool = static_cast<uint4*>(k_pool); p.v_pool = static_cast<uint4*>(v_pool);
  p.n_committed = n_committed; p.spawned = spawned; p.counters = step_counters; p.status = status;
  p.max_requests = c.max_requests; p.wmax = c.wmax; p.bl = c.block_len; p.max_blocks = c.max_blocks;
  p.mask_id = c.mask_id; p.s_pe = c.s_pe; p.n_kv_heads = c.n_kv_heads; p.head_dim = c.head_dim;
  p.num_pages = c.num_pages; p.max_pages_per_req = c.max_pages_per_req; p.theta_spawn = c.theta_spawn;
  if (int e = cuda_err(ctx, cudaMemsetAsync(step_counters, 0, FB_STEP_COUNTERS * sizeof(int32_t), stream),
                       "clear step counters"))
    return e;
  p.batch_sync = c.batch_sync;
  if (c.batch_sync)
    if (int e = cuda_err(ctx, launch_pdl(gate_batch_reduce_kernel, 1, kGateThreads, 0, stream, p),
                         "gate_batch_reduce_kernel launch"))
      return e;
  if (int e = cuda_err(ctx, launch_pdl(gate_commit_kernel, c.max_requests, kGateThreads, 0, stream, p), "gate_commit_kernel launch")) return e;
  return cuda_err(ctx, cudaGetLastError(), "gate_commit_kernel launch");
}

}  // namespace fb
