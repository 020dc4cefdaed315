// C ABI entry points: argument validation, workspace layout, dispatch to the
// kernel launchers.  No kernel lives here.
#include <cstdlib>
#include <cstring>
#include <new>

#include "fb_common.cuh"

namespace {

thread_local std::string g_err;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int fail(fb_ctx* ctx, int code, const std::string& msg) {
  g_err = msg;
  if (ctx) ctx->err = msg;
  return code;
}

}  // namespace

namespace fb {

WsLayout make_ws_layout(const fb_config& c, int tiles_per_slot, int target_items, int min_chunk_tiles, int pair_on) {
  WsLayout w{};
  const long long qtiles = (long long)c.max_requests * c.wmax * tiles_per_slot;
  const long long max_tiles = ((long long)c.max_pages_per_req * kPage + kTileN - 1) / kTileN + 2;
  size_t off = 0;
  for (int l = 0; l < 2; ++l) {
    WsList& x = w.l[l];
    // list 0: every two tiles a unit (plus one leftover unit per request and two KV heads);
    // list 1: every four tiles of a request and KV head two unit records
    const long long units = l == 0 ? ((qtiles + c.max_requests + 1) / 2) * c.n_kv_heads
                                   : (pair_on ? (qtiles / 4) * 2 * c.n_kv_heads : 0);
    const int target = l == 0 ? target_items : (target_items > 1 ? target_items / 2 : 1);
    const int mult = l + 1;
    // split pieces: the bound that split_rule derives (per scheduling unit; list 1 has two records
    // per unit), and never more than every unit cut into pieces of the minimum length (a unit spans
    // at most the keys its page-table row can address)
    const long long every = units * ((max_tiles + min_chunk_tiles - 1) / min_chunk_tiles);
    const long long by_target = mult * ((long long)kPartsPerTarget * target + 8);
    x.max_units = (int)units;
    x.max_parts = units ? (int)(by_target < every ? by_target : every) : 0;
    x.max_items = x.max_units + x.max_parts;
    x.header = off;  off = align_up(off + sizeof(SchedHeader), 256);
    x.items = off;   off = align_up(off + (size_t)x.max_items * sizeof(AttnItem), 256);
    x.units = off;   off = align_up(off + (size_t)x.max_units * sizeof(AttnUnit), 256);
    x.part_ml = off; off = align_up(off + (size_t)x.max_parts * 2 * kTileM * 2 * sizeof(float), 256);
    x.part_o = off;  off = align_up(off + (size_t)x.max_parts * 2 * kTileM * c.head_dim * sizeof(float), 256);
  }
  w.total = off;
  return w;
}

int check_state(fb_ctx* ctx, const fb_state* st) {
  if (!st) return fail(ctx, FB_ERR_INVALID_ARG, "state is null");
  const void* ps[] = {st->active, st->prefix_len, st->L, st->R, st->tokens, st->pe_done, st->page_table};
  const char* names[] = {"active", "prefix_len", "L", "R", "tokens", "pe_done", "page_table"};
  for (int i = 0; i < 7; ++i)
    if (!ps[i]) return fail(ctx, FB_ERR_INVALID_ARG, std::string("state.") + names[i] + " is null");
  return FB_OK;
}

int check_pack(fb_ctx* ctx, const fb_pack* pk) {
  if (!pk) return fail(ctx, FB_ERR_INVALID_ARG, "pack is null");
  const void* ps[] = {pk->n_live, pk->slot_req, pk->slot_s, pk->slot_pos0, pk->slot_kv_len,
                      pk->slot_flags, pk->req_slot_begin, pk->qtok, pk->pos};
  const char* names[] = {"n_live", "slot_req", "slot_s", "slot_pos0", "slot_kv_len",
                         "slot_flags", "req_slot_begin", "qtok", "pos"};
  for (int i = 0; i < 9; ++i)
    if (!ps[i]) return fail(ctx, FB_ERR_INVALID_ARG, std::string("pack.") + names[i] + " is null");
  return FB_OK;
}

}  // namespace fb

using fb::check_pack;
using fb::check_state;

extern "C" {

int fb_create(const fb_config* cfg, fb_ctx** out) {
  if (!cfg || !out) return fail(nullptr, FB_ERR_INVALID_ARG, "cfg or out is null");
  *out = nullptr;
  const fb_config& c = *cfg;
  if (c.max_requests < 1 || c.wmax < 1 || c.block_len < 1 || c.n_q_heads < 1 || c.n_kv_heads < 1 ||
      c.head_dim < 1 || c.num_pages < 1 || c.max_pages_per_req < 1 || c.vocab < 1 || c.max_blocks < 1 ||
      c.s_pe < 0)
    return fail(nullptr, FB_ERR_INVALID_ARG, "a size in fb_config is not positive");
  if (c.n_q_heads % c.n_kv_heads != 0)
    return fail(nullptr, FB_ERR_SHAPE, "n_kv_heads must divide n_q_heads");
  if (!(c.tau_mask == c.tau_mask) || !(c.tau_edit == c.tau_edit) || !(c.theta_spawn == c.theta_spawn) ||
      !(c.sm_scale == c.sm_scale) || c.sm_scale < 0.f)
    return fail(nullptr, FB_ERR_INVALID_ARG, "a threshold or the scale is NaN or negative");
  const int G = c.n_q_heads / c.n_kv_heads;
  if (c.head_dim != 64 && c.head_dim != 128)
    return fail(nullptr, FB_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  if (c.page_size != fb::kPage) return fail(nullptr, FB_ERR_UNSUPPORTED, "page_size must be 64");
  if (fb::kTileM % G != 0 || (c.block_len * G) % fb::kTileM != 0)
    return fail(nullptr, FB_ERR_UNSUPPORTED,
                "block_len * (n_q_heads / n_kv_heads) must be a multiple of 128 and the group size must divide 128");
  if (c.wmax > 8) return fail(nullptr, FB_ERR_UNSUPPORTED, "wmax must be at most 8");
  if (c.vocab % 8 != 0) return fail(nullptr, FB_ERR_UNSUPPORTED, "vocab must be a multiple of 8");
  if (c.s_pe > 255) return fail(nullptr, FB_ERR_UNSUPPORTED, "s_pe must be at most 255");
  if ((c.delta_literal != 0 && c.delta_literal != 1) || (c.force_progress != 0 && c.force_progress != 1))
    return fail(nullptr, FB_ERR_INVALID_ARG, "delta_literal and force_progress must be 0 or 1");
  if (c.tau_edit < c.tau_mask && !c.delta_literal)
    return fail(nullptr, FB_ERR_UNSUPPORTED,
                "tau_edit < tau_mask needs delta_literal = 1 (with Delta on revealed positions only the order is fixed)");
  if (c.window_in_pages != 0 && c.window_in_pages != 1)
    return fail(nullptr, FB_ERR_INVALID_ARG, "window_in_pages must be 0 or 1");
  if (c.batch_sync != 0 && c.batch_sync != 1)
    return fail(nullptr, FB_ERR_INVALID_ARG, "batch_sync must be 0 or 1");
  if (c.kv_fp8 != 0 && c.kv_fp8 != 1) return fail(nullptr, FB_ERR_INVALID_ARG, "kv_fp8 must be 0 or 1");
  if (c.kv_fp8 && (!c.window_in_pages || c.head_dim != 128))
    return fail(nullptr, FB_ERR_UNSUPPORTED,
                "kv_fp8 = 1 needs window_in_pages = 1 (the scatter is the quantiser) and head_dim = 128");
  if ((long long)c.max_requests * c.wmax * c.block_len > (1ll << 24))
    return fail(nullptr, FB_ERR_UNSUPPORTED, "max_requests * wmax * block_len is too large");
  fb_ctx* ctx = new (std::nothrow) fb_ctx();
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "out of host memory");
  ctx->cfg = c;
  ctx->group = G;
  ctx->tiles_per_slot = c.block_len * G / fb::kTileM;
  ctx->tokens_per_tile = fb::kTileM / G;
  ctx->target_items = fb::kDefaultTargetItems;
  ctx->min_chunk_tiles = fb::kDefaultMinChunkTiles;
  ctx->wait_cycles = fb::kDefaultWaitCycles;
  ctx->pair_on = 0;                      // the CTA-pair kernel is opt-in (fb_tuning.attn_pair)
  ctx->sm_scale = c.sm_scale > 0.f ? c.sm_scale : 1.0f / sqrtf((float)c.head_dim);
  ctx->ws = fb::make_ws_layout(c, ctx->tiles_per_slot, ctx->target_items, ctx->min_chunk_tiles, ctx->pair_on);
  *out = ctx;
  return FB_OK;
}

int fb_set_tuning(fb_ctx* ctx, const fb_tuning* t) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (!t) return fail(ctx, FB_ERR_INVALID_ARG, "tuning is null");
  if (t->attn_target_items < 0 || t->attn_target_items > (1 << 20) || t->attn_min_chunk_tiles < 0 ||
      t->attn_min_chunk_tiles > 4096 || t->wait_cycles < -1 || (t->attn_pair != 0 && t->attn_pair != 1))
    return fail(ctx, FB_ERR_INVALID_ARG, "a tuning value is out of range");
  ctx->target_items = t->attn_target_items ? t->attn_target_items : fb::kDefaultTargetItems;
  ctx->min_chunk_tiles = t->attn_min_chunk_tiles ? t->attn_min_chunk_tiles : fb::kDefaultMinChunkTiles;
  ctx->wait_cycles = t->wait_cycles ? (long long)t->wait_cycles : fb::kDefaultWaitCycles;
  ctx->pair_on = ctx->cfg.head_dim == 128 && !ctx->cfg.kv_fp8 && t->attn_pair;
  ctx->ws = fb::make_ws_layout(ctx->cfg, ctx->tiles_per_slot, ctx->target_items, ctx->min_chunk_tiles, ctx->pair_on);
  return FB_OK;
}

int fb_destroy(fb_ctx* ctx) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  fb::static_forget(ctx);
  delete ctx;
  return FB_OK;
}

int fb_attn_plan_host(const fb_ctx* ctx, const int32_t* h_prefix_len, const int32_t* h_live_blocks, int32_t n,
                      int32_t* h_out) {
  if (!ctx || !h_prefix_len || !h_live_blocks || !h_out || n < 0 || n > ctx->cfg.max_requests)
    return fail(nullptr, FB_ERR_INVALID_ARG, "fb_attn_plan_host: null argument or n outside [0, max_requests]");
  const fb_config& c = ctx->cfg;
  for (int r = 0; r < n; ++r)
    if (h_live_blocks[r] < 0 || h_live_blocks[r] > c.wmax)
      return fail(nullptr, FB_ERR_INVALID_ARG, "fb_attn_plan_host: live blocks outside [0, wmax]");
  for (int list = 0; list < 2; ++list) {
    const int target = list == 0 ? ctx->target_items : (ctx->target_items > 1 ? ctx->target_items / 2 : 1);
    const int mult = list + 1;
    long long total = 0, units = 0;
    for (int r = 0; r < n; ++r) {
      const fb::ReqGeom g = fb::req_geom_of(h_live_blocks[r], h_prefix_len[r], ctx->tiles_per_slot, c.block_len,
                                            c.n_kv_heads, c.window_in_pages, list, ctx->pair_on);
      total += (long long)g.nunits * g.nt;
      units += g.nt ? g.nunits : 0;
    }
    if (total > 0x7fffffffll) return fail(nullptr, FB_ERR_UNSUPPORTED, "fb_attn_plan_host: work list too long");
    const fb::SplitRule rule = fb::split_rule((int)total, (int)units, target, ctx->min_chunk_tiles);
    long long wbase = 0, items = 0, parts = 0;
    for (int r = 0; r < n; ++r) {
      const fb::ReqGeom g = fb::req_geom_of(h_live_blocks[r], h_prefix_len[r], ctx->tiles_per_slot, c.block_len,
                                            c.n_kv_heads, c.window_in_pages, list, ctx->pair_on);
      const int nunits = g.nt ? g.nunits : 0;
      const fb::ReqSplit rs = fb::req_split(rule, (int)wbase, nunits, g.nt);
      items += rs.items(nunits);
      parts += rs.parts(nunits);
      wbase += (long long)nunits * g.nt;
    }
    int32_t* o = h_out + 6 * list;
    o[0] = (int32_t)(mult * units); o[1] = (int32_t)items; o[2] = (int32_t)(mult * parts);
    o[3] = ctx->ws.l[list].max_units; o[4] = ctx->ws.l[list].max_items; o[5] = ctx->ws.l[list].max_parts;
  }
  return FB_OK;
}

const char* fb_last_error(const fb_ctx* ctx) { return ctx ? ctx->err.c_str() : g_err.c_str(); }

size_t fb_workspace_bytes(const fb_ctx* ctx) { return ctx ? ctx->ws.total : 0; }

int fb_pack_wavefronts(fb_ctx* ctx, const fb_state* st, const fb_pack* out, void* ws, int32_t* status,
                       void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_state(ctx, st)) return e;
  if (int e = check_pack(ctx, out)) return e;
  if (!ws) return fail(ctx, FB_ERR_WORKSPACE, "workspace is null");
  if (!status) return fail(ctx, FB_ERR_INVALID_ARG, "status is null");
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return fail(ctx, FB_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
  return fb::launch_pack(ctx, st, out, ws, status, (cudaStream_t)stream);
}

int fb_wavefront_attn(fb_ctx* ctx, const fb_pack* pk, const void* q, const void* k_win, const void* v_win,
                      const void* k_pool, const void* v_pool, const int32_t* page_table, void* out, void* ws,
                      int32_t* status, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (ctx->cfg.kv_fp8) return fail(ctx, FB_ERR_UNSUPPORTED, "this context holds 8-bit pages: use fb_wavefront_attn_fp8");
  const bool resident = ctx->cfg.window_in_pages != 0;
  if (!q || !k_pool || !v_pool || !page_table || !out)
    return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (resident && (k_win || v_win))
    return fail(ctx, FB_ERR_INVALID_ARG, "window_in_pages = 1: k_win and v_win must be null (the window is read from the pages)");
  if (!resident && (!k_win || !v_win)) return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!ws) return fail(ctx, FB_ERR_WORKSPACE, "workspace is null");
  if (!status) return fail(ctx, FB_ERR_INVALID_ARG, "status is null");
  if (!aligned16(q) || !aligned16(k_win) || !aligned16(v_win) || !aligned16(k_pool) || !aligned16(v_pool) ||
      !aligned16(out))
    return fail(ctx, FB_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return fail(ctx, FB_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
  return fb::launch_attn(ctx, pk, q, k_win, v_win, k_pool, v_pool, page_table, out, ws, status,
                         (cudaStream_t)stream);
}

int fb_scatter_window_kv(fb_ctx* ctx, const fb_pack* pk, const int32_t* page_table, const void* k_new,
                         const void* v_new, void* k_pool, void* v_pool, float rope_base, int32_t* status,
                         void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (ctx->cfg.kv_fp8) return fail(ctx, FB_ERR_UNSUPPORTED, "this context holds 8-bit pages: use fb_scatter_window_kv_fp8");
  if (!page_table || !k_new || !v_new || !k_pool || !v_pool || !status)
    return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pool) || !aligned16(v_pool))
    return fail(ctx, FB_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (!(rope_base == rope_base) || rope_base < 0.f) return fail(ctx, FB_ERR_INVALID_ARG, "rope_base is NaN or negative");
  return fb::launch_scatter(ctx, pk, page_table, k_new, v_new, k_pool, v_pool, rope_base, status,
                            (cudaStream_t)stream);
}

static int check_fp8_ctx(fb_ctx* ctx) {
  if (!ctx->cfg.kv_fp8)
    return fail(ctx, FB_ERR_UNSUPPORTED, "8-bit KV pages need a context created with kv_fp8 = 1 (window_in_pages = 1, head_dim = 128)");
  return FB_OK;
}

int fb_scatter_window_kv_fp8(fb_ctx* ctx, const fb_pack* pk, const int32_t* page_table, const void* k_new,
                             const void* v_new, void* k_pool8, void* v_pool8, const float* k_scale,
                             const float* v_scale, float rope_base, int32_t* status, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (int e = check_fp8_ctx(ctx)) return e;
  if (!page_table || !k_new || !v_new || !k_pool8 || !v_pool8 || !k_scale || !v_scale || !status)
    return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pool8) || !aligned16(v_pool8))
    return fail(ctx, FB_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (!(rope_base == rope_base) || rope_base < 0.f) return fail(ctx, FB_ERR_INVALID_ARG, "rope_base is NaN or negative");
  return fb::launch_scatter_fp8(ctx, pk, page_table, k_new, v_new, k_pool8, v_pool8, k_scale, v_scale, rope_base,
                                status, (cudaStream_t)stream);
}

int fb_wavefront_attn_fp8(fb_ctx* ctx, const fb_pack* pk, const void* q, const void* k_pool8, const void* v_pool8,
                          const float* k_scale, const float* v_scale, const int32_t* page_table, void* out,
                          void* ws, int32_t* status, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (int e = check_fp8_ctx(ctx)) return e;
  if (!q || !k_pool8 || !v_pool8 || !k_scale || !v_scale || !page_table || !out)
    return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!ws) return fail(ctx, FB_ERR_WORKSPACE, "workspace is null");
  if (!status) return fail(ctx, FB_ERR_INVALID_ARG, "status is null");
  if (!aligned16(q) || !aligned16(k_pool8) || !aligned16(v_pool8) || !aligned16(out))
    return fail(ctx, FB_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return fail(ctx, FB_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
  return fb::launch_attn_fp8(ctx, pk, q, k_pool8, v_pool8, k_scale, v_scale, page_table, out, ws, status,
                             (cudaStream_t)stream);
}

int fb_embed_gather(fb_ctx* ctx, const fb_pack* pk, const void* table, int32_t table_rows, int32_t hidden,
                    void* x, int32_t* status, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (!table || !x || !status) return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (table_rows < 1 || hidden < 8 || hidden % 8 != 0)
    return fail(ctx, FB_ERR_SHAPE, "table_rows must be positive and hidden a positive multiple of 8");
  if (!aligned16(table) || !aligned16(x)) return fail(ctx, FB_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  return fb::launch_embed(ctx, pk, table, table_rows, hidden, x, status, (cudaStream_t)stream);
}

int fb_t2t_step(fb_ctx* ctx, const fb_pack* pk, const void* logits, const fb_state* st, int32_t* argmax,
                float* conf, uint8_t* action, int32_t* slot_stats, int32_t* status, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (int e = check_state(ctx, st)) return e;
  if (!logits || !argmax || !conf || !action || !slot_stats || !status)
    return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!aligned16(logits)) return fail(ctx, FB_ERR_ALIGNMENT, "logits must be 16-byte aligned");
  return fb::launch_t2t(ctx, pk, logits, st, argmax, conf, action, slot_stats, status, (cudaStream_t)stream);
}

size_t fb_lm_head_workspace_bytes(const fb_ctx* ctx) { return ctx ? fb::lm_head_workspace_bytes(ctx) : 0; }

int fb_lm_head_t2t(fb_ctx* ctx, const fb_pack* pk, const void* x, const void* w, int32_t hidden,
                   const fb_state* st, int32_t* argmax, float* conf, uint8_t* action, int32_t* slot_stats,
                   void* ws, int32_t* status, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (int e = check_state(ctx, st)) return e;
  if (!x || !w || !argmax || !conf || !action || !slot_stats || !status)
    return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!ws) return fail(ctx, FB_ERR_WORKSPACE, "workspace is null");
  if (hidden < 64 || hidden % 64 != 0) return fail(ctx, FB_ERR_SHAPE, "hidden must be a positive multiple of 64");
  if (!aligned16(x) || !aligned16(w) || !aligned16(ws))
    return fail(ctx, FB_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  return fb::launch_lm_head(ctx, pk, x, w, hidden, st, argmax, conf, action, slot_stats, ws, status,
                            (cudaStream_t)stream);
}

int fb_gate_commit(fb_ctx* ctx, const fb_pack* pk, const int32_t* slot_stats, const fb_state* st,
                   const void* k_win, const void* v_win, void* k_pool, void* v_pool, int32_t* n_committed,
                   uint8_t* spawned, int32_t* step_counters, int32_t* status, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (int e = check_pack(ctx, pk)) return e;
  if (int e = check_state(ctx, st)) return e;
  if (ctx->cfg.window_in_pages) k_win = v_win = nullptr;      // nothing to copy: the window already lives in the pages
  else if (!k_win || !v_win || !k_pool || !v_pool) return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!slot_stats || !n_committed || !spawned || !step_counters || !status)
    return fail(ctx, FB_ERR_INVALID_ARG, "a tensor pointer is null");
  if (!aligned16(k_win) || !aligned16(v_win) || !aligned16(k_pool) || !aligned16(v_pool))
    return fail(ctx, FB_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  return fb::launch_gate(ctx, pk, slot_stats, st, k_win, v_win, k_pool, v_pool, n_committed, spawned,
                         step_counters, status, (cudaStream_t)stream);
}

int fb_step_host(fb_ctx* ctx, const fb_state* st, const fb_pack* pk, const fb_device_bufs* dev,
                 const fb_host_io* io, void* stream) {
  if (!ctx) return fail(nullptr, FB_ERR_INVALID_ARG, "ctx is null");
  if (!dev || !io) return fail(ctx, FB_ERR_INVALID_ARG, "dev or io is null");
  if (!io->h_q || !io->h_k_win || !io->h_v_win || !io->h_logits || !io->h_n_committed || !io->h_spawned ||
      !io->h_step_counters || !io->h_status)
    return fail(ctx, FB_ERR_INVALID_ARG, "a host pointer is null");
  if (!dev->q || !dev->k_win || !dev->v_win || !dev->out || !dev->logits || !dev->status)
    return fail(ctx, FB_ERR_INVALID_ARG, "a device staging pointer is null");
  const fb_config& c = ctx->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  size_t rows = (size_t)c.max_requests * c.wmax * c.block_len;
  if (io->n_rows > 0 && (size_t)io->n_rows < rows) rows = (size_t)io->n_rows;   // only the rows in use travel
  const size_t qb = rows * c.n_q_heads * c.head_dim * 2, kb = rows * c.n_kv_heads * c.head_dim * 2;
  const size_t lb = rows * (size_t)c.vocab * 2;
  int e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(dev->q, io->h_q, qb, cudaMemcpyHostToDevice, s), "copy q"))) return e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(dev->k_win, io->h_k_win, kb, cudaMemcpyHostToDevice, s), "copy k_win"))) return e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(dev->v_win, io->h_v_win, kb, cudaMemcpyHostToDevice, s), "copy v_win"))) return e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(dev->logits, io->h_logits, lb, cudaMemcpyHostToDevice, s), "copy logits"))) return e;
  if ((e = fb_pack_wavefronts(ctx, st, pk, dev->ws, dev->status, stream))) return e;
  const bool resident = c.window_in_pages != 0;
  if (resident && (e = fb_scatter_window_kv(ctx, pk, st->page_table, dev->k_win, dev->v_win, dev->k_pool,
                                            dev->v_pool, 0.f, dev->status, stream))) return e;
  if ((e = fb_wavefront_attn(ctx, pk, dev->q, resident ? nullptr : dev->k_win, resident ? nullptr : dev->v_win,
                             dev->k_pool, dev->v_pool, st->page_table, dev->out, dev->ws, dev->status, stream)))
    return e;
  if ((e = fb_t2t_step(ctx, pk, dev->logits, st, dev->argmax, dev->conf, dev->action, dev->slot_stats,
                       dev->status, stream))) return e;
  if ((e = fb_gate_commit(ctx, pk, dev->slot_stats, st, dev->k_win, dev->v_win, dev->k_pool, dev->v_pool,
                          dev->n_committed, dev->spawned, dev->step_counters, dev->status, stream))) return e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(io->h_n_committed, dev->n_committed, (size_t)c.max_requests * 4,
                                             cudaMemcpyDeviceToHost, s), "copy n_committed"))) return e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(io->h_spawned, dev->spawned, (size_t)c.max_requests,
                                             cudaMemcpyDeviceToHost, s), "copy spawned"))) return e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(io->h_step_counters, dev->step_counters, FB_STEP_COUNTERS * 4,
                                             cudaMemcpyDeviceToHost, s), "copy counters"))) return e;
  if ((e = fb::cuda_err(ctx, cudaMemcpyAsync(io->h_status, dev->status, 4, cudaMemcpyDeviceToHost, s),
                        "copy status"))) return e;
  return FB_OK;
}

}  // extern "C"
