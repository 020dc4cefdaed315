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

struct WsLayout {
  size_t header, items, units, part_ml, part_o, total;
  int32_t max_items, max_units, max_parts;
};

}  // namespace fb

struct fb_ctx {
  fb_config cfg;
  int group;            // G = n_q_heads / n_kv_heads
  int tiles_per_slot;   // bl * G / 128
  int tokens_per_tile;  // 128 / G
  int target_items;
  int min_chunk_tiles;
  float sm_scale;
  fb::WsLayout ws;
  std::string err;
  // lazily initialised at the first attention launch
  bool dev_ready = false;
  int num_sms = 0;
  void* encode_fn = nullptr;
  // cached tensor maps (re-encoded when a base pointer changes)
  const void* map_ptrs[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
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
int launch_scatter(fb_ctx*, const fb_pack*, const int32_t* page_table, const void* k_new, const void* v_new,
                   void* k_pool, void* v_pool, float rope_base, int32_t* status, cudaStream_t);
int ensure_device(fb_ctx*);   // device properties, driver entry point for tensor maps, kernel attributes
int launch_t2t_update(fb_ctx*, const fb_pack*, const fb_state*, const int32_t* argmax, const float* conf,
                      uint8_t* action, int32_t* slot_stats, cudaStream_t);
int launch_lm_head(fb_ctx*, const fb_pack*, const void* x, const void* w, int hidden, const fb_state*,
                   int32_t* argmax, float* conf, uint8_t* action, int32_t* slot_stats, void* ws, int32_t* status,
                   cudaStream_t);
size_t lm_head_workspace_bytes(const fb_ctx*);
int launch_embed(fb_ctx*, const fb_pack*, const void* table, int table_rows, int hidden, void* x,
                 int32_t* status, cudaStream_t);
int launch_t2t(fb_ctx*, const fb_pack*, const void* logits, const fb_state*, int32_t* argmax,
               float* conf, uint8_t* action, int32_t* slot_stats, int32_t* status, cudaStream_t);
int launch_gate(fb_ctx*, const fb_pack*, const int32_t* slot_stats, const fb_state*,
                const void* k_win, const void* v_win, void* k_pool, void* v_pool,
                int32_t* n_committed, uint8_t* spawned, int32_t* step_counters, int32_t* status,
                cudaStream_t);

inline int set_err(fb_ctx* ctx, int code, const std::string& msg) {
  if (ctx) ctx->err = msg;
  return code;
}
inline int cuda_err(fb_ctx* ctx, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return FB_OK;
  return set_err(ctx, FB_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

}  // namespace fb
