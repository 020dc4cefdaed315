// fb_gate_commit: in-order retirement with KV freeze and readiness-gated
// admission (Alg. 1 lines 7-12, Eq. 2-3, Eq. 6 for the committing block).
//
// One CTA per request.  Thread 0 evaluates the block-level predicates from
// the per-slot counts; all threads then copy the retiring blocks' window K/V
// rows into the request's pages with 16-byte accesses; thread 0 publishes the
// new state.  Requests are independent, so no inter-CTA ordering is needed;
// the step counters are integer atomics on a zeroed array.
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
};

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
    const int first = p.req_slot_begin[r];
    int w = p.req_slot_begin[r + 1] - first;
    int L = p.L[r], R = p.R[r];
    if (w != R - L || w < 0 || w > p.wmax) {       // pack and state disagree: leave the request alone
      atomicOr(p.status, FB_ST_BAD_STATE);
      s_c = 0; s_spawn = 0; s_first = first; s_P = 0; s_newR = R;
      p.n_committed[r] = 0; p.spawned[r] = 0;
      w = -1;
    }
    if (w >= 0) {
    uint8_t pe_new[8];
    bool fin[8];
    int m2t = 0, t2t = 0;
    for (int s = 0; s < w; ++s) {
      const int32_t* st = p.slot_stats + (first + s) * FB_SLOT_STATS;
      const int m0 = st[FB_STAT_M0], m1 = st[FB_STAT_M1], nupd = st[FB_STAT_M2T] + st[FB_STAT_T2T];
      int pn = p.pe_done[r * p.wmax + s] + (m0 == 0 ? 1 : 0);
      pn = pn > 255 ? 255 : pn;
      pe_new[s] = (uint8_t)pn;
      // locally finished (Sec. 2.1): no masks left, and either a quiet
      // post-edit forward or the S_pe budget is used up
      fin[s] = m1 == 0 && ((m0 == 0 && nupd == 0) || pn >= p.s_pe);
      m2t += st[FB_STAT_M2T]; t2t += st[FB_STAT_T2T];
    }
    int c = 0;
    bool eos = false;
    while (c < w && fin[c]) {                      // Alg. 1 l.7-9, in order
      ++c;
      if (p.slot_stats[(first + c - 1) * FB_SLOT_STATS + FB_STAT_EOS]) { eos = true; break; }
    }
    const int P = p.prefix_len[r];
    s_c = c; s_first = first; s_P = P;
    L += c;
    for (int s = 0; s < p.wmax; ++s) p.pe_done[r * p.wmax + s] = s + c < w ? pe_new[s + c] : 0;
    const bool done = eos || L == p.max_blocks;
    int spawn = 0;
    if (!done) {
      // Eq. 2 on the frontier block as it went into this forward; Eq. 3
      float rho = 1.0f;
      if (w > 0) {
        const int32_t* st = p.slot_stats + (first + w - 1) * FB_SLOT_STATS;
        if (st[FB_STAT_M0] != 0) rho = __fdiv_rn((float)st[FB_STAT_RDY], (float)st[FB_STAT_M0]);
      }
      if (rho >= p.theta_spawn && R - L < p.wmax && R < p.max_blocks) spawn = 1;
    }
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
    if (m2t) atomicAdd(&p.counters[FB_CT_M2T], m2t);
    if (t2t) atomicAdd(&p.counters[FB_CT_T2T], t2t);
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
  if (int e = cuda_err(ctx, launch_pdl(gate_commit_kernel, c.max_requests, kGateThreads, 0, stream, p), "gate_commit_kernel launch")) return e;
  return cuda_err(ctx, cudaGetLastError(), "gate_commit_kernel launch");
}

}  // namespace fb
