// Pieces shared by the attention kernels (one CTA per work item; a pair of CTAs per work item):
// launch parameters, the geometry of a work item, the exponential on the FMA pipe.
#pragma once
#include "fb_common.cuh"
#include "ptx_sm100.cuh"

namespace fb {

constexpr int kAttnThreads = 384;   // 3 warpgroups: control, softmax A, softmax B
constexpr float kLog2eF = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;   // log2 units (8-bit P: bound on every element)
// bf16 P: the reference is re-based when the exponentials of one key tile sum to more than 2^8
// (a bound on every element that costs no per-element work; inf and NaN fail the test too).
// Kept this low on purpose: after a re-base the largest weight is exactly 1, so a row that one key
// dominates carries no rounding error of P on that key.
constexpr float kGrowSum = 256.0f;
// Dynamic shared memory per CTA.  Both sizes exceed half of the 227 KB an SM
// offers, so two CTAs never share an SM: each CTA allocates all 512 TMEM columns.
constexpr int kSmem64 = 120 * 1024;
constexpr int kSmem128 = 6 * 32768 + 8192;
constexpr int kSmemF8 = 2 * 32768 + 6 * 16384 + 8192;   // Q staging (bf16), Q / K / V tiles in 8 bits
// 8-bit pages: the exponentials are taken 2^4 above the reference, so that E4M3 (normal down to
// 2^-6, largest value 448) holds P from 2^-10 of the reference up to the 2^8 bound of the lazy re-base
constexpr float kF8PShift = 4.0f;

struct AttnParams {
  SchedHeader* hdr;
  const AttnItem* items;
  const AttnUnit* units;
  const int32_t* page_table;
  __nv_bfloat16* out;
  float* part_ml;
  float* part_o;
  int32_t* status;
  int32_t bl, n_q_heads, n_kv_heads, group, max_pages_per_req, num_pages;
  int32_t resident;     // 1: the window is read from the pages (every key tile is a paged one)
  const float* k_scale; // 8-bit pages only: value = code * scale of the KV head, [n_kv_heads]
  const float* v_scale;
  float scale_log2;
  long long wait_cycles;
};

// Geometry of one work item, computed identically by every role.
struct ItemGeom {
  AttnUnit un;
  int jb, n, nA, nB, chunk, kvhA, kvhB;
};

__device__ __forceinline__ bool load_item(const AttnParams& p, int idx, ItemGeom& g) {
  const int4 it = *reinterpret_cast<const int4*>(&p.items[idx]);
  const int4* up = reinterpret_cast<const int4*>(&p.units[it.x]);
  const int4 u0 = up[0], u1 = up[1], u2 = up[2], u3 = up[3];
  g.un.req = u0.x; g.un.kvh = u0.y; g.un.slotA = u0.z; g.un.slotB = u0.w;
  g.kvhA = u0.y & 0xffff; g.kvhB = u0.y >> 16;
  g.un.t0A = u1.x; g.un.t0B = u1.y; g.un.n_tiles = u1.z; g.un.n_chunks = u1.w;
  g.un.nvisA = u2.x; g.un.nvisB = u2.y; g.un.part_base = u2.z; g.un.prefix_len = u2.w;
  g.un.npt = u3.x; g.un.win_row0 = u3.y; g.un.winA = u3.z; g.un.winB = u3.w;
  g.chunk = it.y; g.jb = it.z;
  const int je = it.w;
  g.nA = max(0, min(je, g.un.nvisA) - g.jb);
  g.nB = g.un.slotB >= 0 ? max(0, min(je, g.un.nvisB) - g.jb) : 0;
  g.n = max(g.nA, g.nB);
  return g.n > 0;
}

// 2^x for a pair of values on the FMA pipe (the MUFU pipe is as busy as the
// tensor pipe in this kernel, so a share of the exponentials is moved off it):
// round-to-nearest split x = n + f, f in [-0.5, 0.5], cubic minimax fit of 2^f
// (max relative error 7.5e-5, far below bf16 resolution), then n is added to
// the exponent field.  Valid for -120 <= x <= 120.
constexpr int kPolyOf4 = 1;   // pairs out of every 4 that take this path (bf16 pages)
constexpr int kPolyOf4F8 = 1;   // the same share with 8-bit pages (0, 2 and 3 of 4 measured slower)
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
  x.x = fminf(fmaxf(x.x, -120.f), 120.f);     // beyond +120 the result stays huge: the caller's overflow check fires
  x.y = fminf(fmaxf(x.y, -120.f), 120.f);
  const float kMagic = 12582912.f;   // 1.5 * 2^23: x + kMagic has round(x) in its low mantissa bits
  const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
  const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
  float2 q = __ffma2_rn(make_float2(0.05517137795686722f, 0.05517137795686722f), f,
                        make_float2(0.24261121451854706f, 0.24261121451854706f));
  q = __ffma2_rn(q, f, make_float2(0.6932610273361206f, 0.6932610273361206f));
  q = __ffma2_rn(q, f, make_float2(0.9999280571937561f, 0.9999280571937561f));
  q.x = __int_as_float(__float_as_int(q.x) + (__float_as_int(t.x) << 23));
  q.y = __int_as_float(__float_as_int(q.y) + (__float_as_int(t.y) << 23));
  return q;
}

__device__ __forceinline__ int uni(int x) { return __shfl_sync(0xffffffffu, x, 0); }

// The subset of an item the control warps need, made warp-uniform (every lane
// holds lane 0's copy) so that the compiler keeps it in uniform registers.
struct ItemU {
  int req, kvhA, kvhB, rowA, rowB, jb, n, nA, nB, npt, prefix_len, win_row0, winA, winB;
  __device__ __forceinline__ bool dual() const { return kvhA != kvhB; }   // two K/V streams
  // keys of local tile j that a tile with window reach winX may see; `resident`: the
  // window follows the prefix in the pages, one run of keys [0, prefix_len + winX)
  __device__ __forceinline__ int limit(int j, int winX, int resident) const {
    const int gj = jb + j;
    const int lim = gj < npt ? prefix_len + (resident ? winX : 0) - gj * kTileN : winX - (gj - npt) * kTileN;
    return min(lim, kTileN);
  }
};

__device__ __forceinline__ bool load_item_uniform(const AttnParams& p, int idx, ItemU& u) {
  ItemGeom g;
  load_item(p, idx, g);
  u.req = uni(g.un.req); u.kvhA = uni(g.kvhA); u.kvhB = uni(g.kvhB);
  u.rowA = uni(g.un.slotA * p.bl + g.un.t0A); u.rowB = uni(g.un.slotB * p.bl + g.un.t0B);
  u.jb = uni(g.jb); u.n = uni(g.n); u.nA = uni(g.nA); u.nB = uni(g.nB);
  u.npt = uni(g.un.npt); u.prefix_len = uni(g.un.prefix_len); u.win_row0 = uni(g.un.win_row0);
  u.winA = uni(g.un.winA); u.winB = uni(g.un.winB);
  return u.n > 0;
}

// All lanes of a converged warp wait on the barrier; the result is uniform.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort, long long limit) {
  const bool ok = mbar_wait(bar, parity, abort, limit);
  return __all_sync(0xffffffffu, ok);
}

// number of keys of local tile j that tile X (window reach winX) may see
__device__ __forceinline__ int tile_limit(const ItemGeom& g, int j, int winX, int resident) {
  const int gj = g.jb + j;
  const int lim = gj < g.un.npt ? g.un.prefix_len + (resident ? winX : 0) - gj * kTileN
                                : winX - (gj - g.un.npt) * kTileN;
  return min(lim, kTileN);
}
__device__ __forceinline__ int round16(int x) { return (x + 15) & ~15; }

void fill_attn_params(fb_ctx* ctx, AttnParams& p, const int32_t* page_table, void* out, void* ws, int32_t* status,
                      int list);
// merge of the split-KV partial results of work list `list` (and the re-arming of its ticket)
int launch_attn_combine(fb_ctx* ctx, const AttnParams& p, int list, cudaStream_t stream);

}  // namespace fb
