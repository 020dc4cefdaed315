// fb_wavefront_attn_static: the attention call for callers that must not
// allocate device memory.
//
// Who cannot allocate: code that runs inside a region where cudaMalloc is
// forbidden or unavailable -- a serving engine that has handed every byte of
// the device to its own pool allocator, a plugin loaded into a process whose
// memory is pre-partitioned, a real-time loop that may not take the allocator's
// implicit device synchronisation.  fb_wavefront_attn needs a caller-allocated
// workspace for its work list and split-KV partials; this variant keeps that
// scratch in a fixed array inside the library image instead.
//
// The scratch is one file-scope __device__ array of kStaticScratchBytes.  Every
// GPU that loads the library holds it until the process exits.  In host code
// the array's name is only a host-side stand-in, not a device address, so the
// address is fetched once per device with cudaGetSymbolAddress (with that
// device current) and that pointer is what the kernels get.
#include <cstring>
#include <mutex>
#include <unordered_map>

#include "fb_common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;   // 8 MiB per GPU
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};
// One private context per caller context: same configuration, but a work list
// that never splits the key axis, so the scratch holds only the scheduler
// header, the item list and the unit list (no split-KV partials to speak of).
std::unordered_map<const fb_ctx*, fb_ctx*> g_shadow;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

fb::WsLayout unsplit_layout(const fb_ctx* c) {
  fb::WsLayout w{};
  const long long qtiles = (long long)c->cfg.max_requests * c->cfg.wmax * c->tiles_per_slot;
  fb::WsList& x = w.l[0];
  x.max_units = (int)((qtiles + c->cfg.max_requests + 1) / 2) * c->cfg.n_kv_heads;
  x.max_items = x.max_units + 8;
  x.max_parts = 2;        // never used: no unit is split
  size_t off = 0;
  x.header = off;  off = align_up(off + sizeof(fb::SchedHeader), 256);
  x.items = off;   off = align_up(off + (size_t)x.max_items * sizeof(fb::AttnItem), 256);
  x.units = off;   off = align_up(off + (size_t)x.max_units * sizeof(fb::AttnUnit), 256);
  x.part_ml = off; off = align_up(off + (size_t)x.max_parts * 2 * fb::kTileM * 2 * sizeof(float), 256);
  x.part_o = off;  off = align_up(off + (size_t)x.max_parts * 2 * fb::kTileM * c->cfg.head_dim * sizeof(float), 256);
  // the second work list (CTA-pair kernel) stays empty here: a header and nothing else
  fb::WsList& y = w.l[1];
  y.max_units = y.max_items = y.max_parts = 0;
  y.header = off;  off = align_up(off + sizeof(fb::SchedHeader), 256);
  y.items = y.units = y.part_ml = y.part_o = off;
  w.total = off;
  return w;
}

}  // namespace

// fb_destroy calls this: the private context of a destroyed context goes with it, so a new
// context that happens to be allocated at the same address starts from nothing.
void fb::static_forget(const fb_ctx* ctx) {
  std::lock_guard<std::mutex> lock(g_mu);
  auto it = g_shadow.find(ctx);
  if (it == g_shadow.end()) return;
  delete it->second;
  g_shadow.erase(it);
}

extern "C" int fb_wavefront_attn_static(fb_ctx* ctx, const fb_state* st, const fb_pack* pk, const void* q,
                                        const void* k_win, const void* v_win, const void* k_pool,
                                        const void* v_pool, void* out, int32_t* status, void* stream) {
  if (!ctx) return FB_ERR_INVALID_ARG;
  // every array of the state and of the pack is read or written by the pack kernel
  if (int e = fb::check_state(ctx, st)) return e;
  if (int e = fb::check_pack(ctx, pk)) return e;
  if (!q || !k_win || !v_win || !k_pool || !v_pool || !out || !status)
    return fb::set_err(ctx, FB_ERR_INVALID_ARG, "fb_wavefront_attn_static: a pointer is null");
  if (ctx->cfg.window_in_pages)
    return fb::set_err(ctx, FB_ERR_UNSUPPORTED, "fb_wavefront_attn_static: contexts with window_in_pages = 1 are not supported");
  const void* ps[] = {q, k_win, v_win, k_pool, v_pool, out};
  for (const void* p : ps)
    if (reinterpret_cast<uintptr_t>(p) & 15u)
      return fb::set_err(ctx, FB_ERR_ALIGNMENT, "fb_wavefront_attn_static: tensor pointers must be 16-byte aligned");
  const fb::WsLayout lay = unsplit_layout(ctx);
  if (lay.total > kStaticScratchBytes)
    return fb::set_err(ctx, FB_ERR_WORKSPACE,
                       "fb_wavefront_attn_static: this configuration needs " + std::to_string(lay.total) +
                           " bytes of scratch, the built-in array holds " + std::to_string(kStaticScratchBytes) +
                           " (8 MiB); use fb_wavefront_attn with a caller-provided workspace");
  std::lock_guard<std::mutex> lock(g_mu);
  int dev = 0;
  if (int e = fb::cuda_err(ctx, cudaGetDevice(&dev), "cudaGetDevice")) return e;
  if (dev < 0 || dev >= kMaxDevices) return fb::set_err(ctx, FB_ERR_UNSUPPORTED, "device index out of range");
  if (!g_scratch_ptr[dev]) {
    // once per device, with that device current: the device address of the array
    void* p = nullptr;
    if (int e = fb::cuda_err(ctx, cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress")) return e;
    if (!p) return fb::set_err(ctx, FB_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
    g_scratch_ptr[dev] = p;
  }
  fb_ctx*& sh = g_shadow[ctx];
  if (!sh) {
    sh = new fb_ctx();
    sh->cfg = ctx->cfg;
    sh->group = ctx->group;
    sh->tiles_per_slot = ctx->tiles_per_slot;
    sh->tokens_per_tile = ctx->tokens_per_tile;
    sh->sm_scale = ctx->sm_scale;
    sh->target_items = 1;                 // chunk length = all tiles: nothing is split
    sh->min_chunk_tiles = 1 << 20;
    sh->pair_on = 0;                      // one work list, one kernel
    sh->ws = lay;
  }
  sh->wait_cycles = ctx->wait_cycles;
  void* ws = g_scratch_ptr[dev];
  cudaStream_t s = (cudaStream_t)stream;
  // The work list is rebuilt from the current state by the pack kernel (it
  // overwrites header, items and units completely, so nothing in the array has
  // to start at zero), then the attention kernel consumes it.
  int e = fb::launch_pack(sh, st, pk, ws, status, s);
  if (!e) e = fb::launch_attn(sh, pk, q, k_win, v_win, k_pool, v_pool, st->page_table, out, ws, status, s);
  if (e) ctx->err = sh->err;
  return e;
}
