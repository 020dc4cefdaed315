// Shared declarations of the CUDA path: context, workspace layout, the
// attention work list.  Nothing here is used by the CPU oracle.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string>

#include "../../include/flowblock.h"

namespace fb {

constexpr int kTileM = 128;      // query rows per Q tile (tokens x group heads)
constexpr int kTileN = 128;      // keys per K/V tile (two 64-token pages)
constexpr int kPage = 64;
constexpr int kDefaultMinChunkTiles = 4;
constexpr int kDefaultTargetItems = 2 * 148;   // about two work items per SM before key ranges are split

// One unit = two Q tiles of one request that run side by side in a CTA: either
// two different tiles under one KV head (they share every K/V tile), or one
// tile under two adjacent KV heads (two K/V streams).  Split along the key
// axis into n_chunks items.  16 ints each, read as four int4.
struct __align__(16) AttnUnit {
  int32_t req, kvh, slotA, slotB;      // kvh: KV head of tile A | KV head of tile B << 16
                                       // slotB = -1: single tile
  int32_t t0A, t0B, n_tiles, n_chunks; // n_tiles: key tiles of the request
  int32_t nvisA, nvisB, part_base, prefix_len;
  int32_t npt, win_row0, winA, winB;   // npt prefix tiles; winX = window keys
                                       // visible to tile X = (s+1)*bl
};
struct __align__(16) AttnItem {
  int32_t unit, chunk, jb, je;         // key tiles [jb, je) of the unit
};

struct SchedHeader {
  int32_t n_items, n_units, chunk_tiles, n_parts;
  int32_t total_tiles;
  int32_t ticket, done;                // dynamic item hand-out of the attention kernel
  int32_t pad[9];
};

// The workspace holds two work lists: list 0 for the one-CTA kernel, list 1 ("quads": four Q
// tiles of one request and KV head) for the CTA-pair kernel.  List 1 is empty when pairing is off.
struct WsList {
  size_t header, items, units, part_ml, part_o;
  int32_t max_items, max_units, max_parts;
};
struct WsLayout {
  WsList l[2];
  size_t total;
};

// ---------------------------------------------------------------------------
// Arithmetic of the attention work list, shared by the pack kernel (which
// builds the list on the device) and by the host code that sizes the workspace.
// ---------------------------------------------------------------------------

// A request's Q tiles are paired two by two (a pair shares every K/V tile).
// An odd tile left over is paired with itself across two adjacent KV heads
// instead: the two halves stream different K/V but keep both tile slots of a
// CTA busy, which a lone tile cannot.  nunits counts both kinds.
// With pairing on, the first 4 * nquad tiles of a request go to list 1 as quads (one scheduling
// unit per quad and KV head, run by a pair of CTAs: tiles 4q + r and 4q + 2 + r in CTA r); list 0
// takes the remaining ntq tiles, starting at tile0.
struct ReqGeom {
  int w, ntq, tile0, nquad, P, npt, nt;
  int nfull, odd, nunits;   // full pairs per KV head; leftover tile; scheduling units of the request in this list
};
__host__ __device__ inline ReqGeom req_geom_of(int w, int prefix_len, int tiles_per_slot, int bl, int n_kv_heads,
                                               int resident, int list, int pair_on) {
  ReqGeom g;
  g.w = w;
  const int ntq_all = g.w * tiles_per_slot;
  g.nquad = pair_on ? ntq_all >> 2 : 0;
  if (list == 1) {
    g.ntq = 4 * g.nquad; g.tile0 = 0; g.nfull = 0; g.odd = 0;
    g.nunits = g.nquad * n_kv_heads;
  } else {
    g.ntq = ntq_all - 4 * g.nquad; g.tile0 = 4 * g.nquad;
    g.nfull = g.ntq >> 1;
    g.odd = g.ntq & 1;
    g.nunits = g.nfull * n_kv_heads + g.odd * ((n_kv_heads + 1) >> 1);
  }
  g.P = g.w ? (prefix_len > 0 ? prefix_len : 0) : 0;
  g.npt = (g.P + kTileN - 1) / kTileN;
  g.nt = g.w ? g.npt + (g.w * bl + kTileN - 1) / kTileN : 0;
  if (resident) {         // one run of keys [0, P + w*bl), all of it paged
    g.nt = g.w ? (g.P + g.w * bl + kTileN - 1) / kTileN : 0;
    g.npt = g.nt;
  }
  if (g.nunits == 0) g.nt = 0;
  return g;
}

// Key-axis split.  `total` = key-tile iterations of all units, `units` = units with work.
//   ct        chunk length of the coarse split: ceil(total / target), at least min_chunk.
//   fine_ct   chunk length of the filler pieces.  Items are handed out longest first, so the
//             CTAs run dry within one shortest item of each other; when even the short items
//             are long (few, long requests), the units whose work lies wholly inside the last
//             15 % of the work are cut into pieces of 1/8 of a CTA's share (target = two items
//             per CTA), which level that tail.
//   fine_from work offset from which on a unit is a filler unit (INT_MAX: no filler).
// Bound on the split pieces ("parts": chunks of units cut into more than one): a unit is only
// cut when it is longer than its chunk length, so at most total / ct <= target coarse units are
// cut, into at most 2 target pieces; the filler units hold at most 0.15 total + 1 tiles and
// fine_ct >= total / (4 target), so at most 0.6 target + 1 of them are cut, into at most
// 1.2 target + 2 pieces: parts <= 3.2 target + 2 <= kPartsPerTarget * target + 8.
constexpr int kFillerPercent = 15;
constexpr int kFillerDiv = 8;
constexpr int kPartsPerTarget = 4;
struct SplitRule { int ct, fine_ct, fine_from; };
__host__ __device__ inline SplitRule split_rule(int total, int units, int target, int min_chunk) {
  SplitRule s;
  const int ct = (int)(((long long)total + target - 1) / target);
  s.ct = ct < min_chunk ? min_chunk : ct;
  const long long den = (long long)target * kFillerDiv;
  const int fine = (int)((2ll * total + den - 1) / den);
  s.fine_ct = fine < min_chunk ? min_chunk : fine;
  const bool on = units > 0 && total / units > 2 * s.fine_ct && s.fine_ct < s.ct;
  s.fine_from = on ? total - (int)((long long)kFillerPercent * total / 100) : 0x7fffffff;
  return s;
}
// One request under the rule: its first `ufine` units take chunks of ct, the others (work
// offset >= fine_from) chunks of fine_ct.  wbase = work offset of the request's first unit.
struct ReqSplit {
  int ufine, nch_c, nch_f;
  __host__ __device__ int chunks(int ul) const { return ul < ufine ? nch_c : nch_f; }
  __host__ __device__ int items(int nunits) const { return ufine * nch_c + (nunits - ufine) * nch_f; }
  __host__ __device__ int parts(int nunits) const {
    return (nch_c > 1 ? ufine * nch_c : 0) + (nch_f > 1 ? (nunits - ufine) * nch_f : 0);
  }
  // offset of unit ul's partial results inside the request's range (only used when chunks(ul) > 1)
  __host__ __device__ int part_off(int ul) const {
    return ul < ufine ? ul * nch_c : (nch_c > 1 ? ufine * nch_c : 0) + (ul - ufine) * nch_f;
  }
};
__host__ __device__ inline ReqSplit req_split(const SplitRule& s, int wbase, int nunits, int nt) {
  ReqSplit r;
  r.ufine = nunits; r.nch_c = 0; r.nch_f = 0;
  if (nt <= 0 || nunits <= 0) { r.ufine = 0; return r; }
  r.nch_c = (nt + s.ct - 1) / s.ct;
  r.nch_f = (nt + s.fine_ct - 1) / s.fine_ct;
  if (s.fine_from != 0x7fffffff) {
    const long long first = ((long long)s.fine_from - wbase + nt - 1) / nt;   // first unit with wbase + ul*nt >= fine_from
    r.ufine = first < 0 ? 0 : (first > nunits ? nunits : (int)first);
  }
  return r;
}

}  // namespace fb

struct fb_ctx {
  fb_config cfg;
  int group;            // G = n_q_heads / n_kv_heads
  int tiles_per_slot;   // bl * G / 128
  int tokens_per_tile;  // 128 / G
  int target_items;       // list 0; list 1 aims for target_items / 2 (half as many executors)
  int min_chunk_tiles;
  int pair_on;            // quads go to the CTA-pair kernel (bf16 pages, head_dim 128)
  long long wait_cycles;  // limit of every bounded device-side wait, in SM clock cycles
  float sm_scale;
  fb::WsLayout ws;
  std::string err;
  // lazily initialised at the first attention launch
  bool dev_ready = false;
  int device = -1;        // the device the lazily initialised members belong to
  int num_sms = 0;
  void* encode_fn = nullptr;
  // cached tensor maps (re-encoded when a base pointer changes)
  CUtensorMap tm_kwin_half;   // 64-row boxes of the window keys (CTA-pair kernel)
  const void* map_ptrs[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  bool maps_f8 = false;   // the cached pool maps describe 8-bit pages
  CUtensorMap tm_q, tm_kwin, tm_vwin, tm_kpool, tm_vpool;
};

namespace fb {

// Launch with programmatic stream serialisation: the kernel may be scheduled while its
// predecessor in the stream is still running and runs up to its pdl_wait() (barrier set-up, TMEM
// allocation, descriptor prefetch); everything after pdl_wait() sees the predecessor complete.
// cluster_x > 1 groups that many consecutive CTAs (along x) into a thread-block cluster.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                      cudaStream_t stream, int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  if (cluster_x > 1) {
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = cluster_x; at[1].val.clusterDim.y = 1; at[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  return launch_pdl_cluster(kernel, grid, block, smem, stream, 1, static_cast<Args&&>(args)...);
}
#ifdef __CUDACC__
// Lets the next kernel of the stream be scheduled, then waits for the previous one to be complete
// (a no-op pair when the kernel was launched the ordinary way).
__device__ __forceinline__ void pdl_wait() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

int launch_pack(fb_ctx*, const fb_state*, const fb_pack*, void* ws, int32_t* status, cudaStream_t);
int launch_attn(fb_ctx*, const fb_pack*, const void* q, const void* k_win, const void* v_win,
                const void* k_pool, const void* v_pool, const int32_t* page_table, void* out,
                void* ws, int32_t* status, cudaStream_t);
int launch_attn_fp8(fb_ctx*, const fb_pack*, const void* q, const void* k_pool8, const void* v_pool8,
                    const float* k_scale, const float* v_scale, const int32_t* page_table, void* out, void* ws,
                    int32_t* status, cudaStream_t);
int launch_scatter_fp8(fb_ctx*, const fb_pack*, const int32_t* page_table, const void* k_new, const void* v_new,
                       void* k_pool8, void* v_pool8, const float* k_scale, const float* v_scale, float rope_base,
                       int32_t* status, cudaStream_t);
int launch_scatter(fb_ctx*, const fb_pack*, const int32_t* page_table, const void* k_new, const void* v_new,
                   void* k_pool, void* v_pool, float rope_base, int32_t* status, cudaStream_t);
int ensure_device(fb_ctx*);   // device properties, driver entry point for tensor maps, kernel attributes
int launch_t2t_update(fb_ctx*, const fb_pack*, const fb_state*, const int32_t* argmax, const float* conf,
                      uint8_t* action, int32_t* slot_stats, cudaStream_t);
int launch_lm_head(fb_ctx*, const fb_pack*, const void* x, const void* w, int hidden, const fb_state*,
                   int32_t* argmax, float* conf, uint8_t* action, int32_t* slot_stats, void* ws, int32_t* status,
                   cudaStream_t);
size_t lm_head_workspace_bytes(const fb_ctx*);
int lm_head_device_setup(fb_ctx*);
int launch_embed(fb_ctx*, const fb_pack*, const void* table, int table_rows, int hidden, void* x,
                 int32_t* status, cudaStream_t);
int launch_t2t(fb_ctx*, const fb_pack*, const void* logits, const fb_state*, int32_t* argmax,
               float* conf, uint8_t* action, int32_t* slot_stats, int32_t* status, cudaStream_t);
int launch_gate(fb_ctx*, const fb_pack*, const int32_t* slot_stats, const fb_state*,
                const void* k_win, const void* v_win, void* k_pool, void* v_pool,
                int32_t* n_committed, uint8_t* spawned, int32_t* step_counters, int32_t* status,
                cudaStream_t);

constexpr long long kDefaultWaitCycles = 2000000000LL;   // about a second at the SM clock

fb::WsLayout make_ws_layout(const fb_config& c, int tiles_per_slot, int target_items, int min_chunk_tiles, int pair_on);
int launch_attn_pair(fb_ctx*, const int32_t* page_table, void* out, void* ws, int32_t* status, cudaStream_t);
int attn_pair_device_setup(fb_ctx*);
int check_state(fb_ctx* ctx, const fb_state* st);   // every member non-null, else FB_ERR_INVALID_ARG
int check_pack(fb_ctx* ctx, const fb_pack* pk);
void static_forget(const fb_ctx* ctx);              // drops what fb_wavefront_attn_static keeps per context

inline int set_err(fb_ctx* ctx, int code, const std::string& msg) {
  if (ctx) ctx->err = msg;
  return code;
}
inline int cuda_err(fb_ctx* ctx, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return FB_OK;
  return set_err(ctx, FB_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

}  // namespace fb
