// fb_scatter_window_kv: Eq. 6 as data movement.  The fresh K/V rows of every
// live window position go to the request's pages at their absolute positions
// (all KV heads), optionally with the rotary embedding applied to the keys.
// HBM-bound: 2 x rows x Hkv x d x 2 bytes read and as many written.
//
// One CTA per slot.  For a (token, head) the head_dim elements are contiguous
// in the source (slot-order rows) and in the destination (pool row of that
// position), so a thread moves 16-byte pieces: with the rotary embedding a
// thread owns the two pieces that hold elements i and i + d/2 of eight pairs.
#include "fb_common.cuh"

namespace fb {

constexpr int kScatterThreads = 256;

struct ScatterParams {
  const int32_t* n_live; const int32_t* slot_req; const int32_t* slot_pos0;
  const int32_t* page_table;
  const uint4 *k_new, *v_new;
  uint4 *k_pool, *v_pool;
  int32_t* status;
  int32_t bl, n_kv_heads, head_dim, max_pages_per_req, num_pages;
  float rope_base;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t to_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// cos / sin of pos * base^(-2i/d) for the eight pairs a thread owns; the angle is
// formed and reduced in fp64 (positions reach tens of thousands of radians)
__device__ __forceinline__ void rope_angles(int pos, int i0, int d, float base, float (&c)[8], float (&s)[8]) {
  const double l2b = log2((double)base);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const double ang = (double)pos * exp2(-2.0 * (double)(i0 + k) / (double)d * l2b);
    double sd, cd;
    sincos(ang, &sd, &cd);
    c[k] = (float)cd; s[k] = (float)sd;
  }
}

__global__ void __launch_bounds__(kScatterThreads) scatter_window_kv_kernel(const ScatterParams p) {
  const int slot = blockIdx.x;
  if (slot >= *p.n_live) return;
  const int r = p.slot_req[slot], pos0 = p.slot_pos0[slot];
  const int vph = p.head_dim / 8;                    // 16-byte pieces per (token, head)
  const int vpt = p.n_kv_heads * vph;                // ... per token
  const bool rope = p.rope_base > 0.f;
  // work item = (token, head, piece); with the rotary embedding only the lower half of the
  // pieces is enumerated and each item also handles its partner piece + d/16
  const int per_head = rope ? vph / 2 : vph;
  const int total = p.bl * p.n_kv_heads * per_head;
  for (int i = threadIdx.x; i < total; i += kScatterThreads) {
    const int t = i / (p.n_kv_heads * per_head), rem = i % (p.n_kv_heads * per_head);
    const int h = rem / per_head, v = rem % per_head;
    const int pos = pos0 + t, pidx = pos / kPage;
    if (pidx >= p.max_pages_per_req) { atomicOr(p.status, FB_ST_BAD_PAGE); continue; }
    const int page = p.page_table[(size_t)r * p.max_pages_per_req + pidx];
    if (page < 0 || page >= p.num_pages) { atomicOr(p.status, FB_ST_BAD_PAGE); continue; }
    const size_t src = (size_t)(slot * p.bl + t) * vpt + h * vph + v;
    const size_t dst = (((size_t)page * p.n_kv_heads + h) * kPage + pos % kPage) * vph + v;
    if (!rope) {
      p.k_pool[dst] = p.k_new[src];
      p.v_pool[dst] = p.v_new[src];
      continue;
    }
    const uint4 a = p.k_new[src], b = p.k_new[src + vph / 2];      // elements i0.. and i0 + d/2..
    float c[8], s[8];
    rope_angles(pos, v * 8, p.head_dim, p.rope_base, c, s);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    uint32_t lo[4], hi[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float x0 = bf16_lo(aw[k]), x1 = bf16_hi(aw[k]), y0 = bf16_lo(bw[k]), y1 = bf16_hi(bw[k]);
      lo[k] = to_bf16x2(x0 * c[2 * k] - y0 * s[2 * k], x1 * c[2 * k + 1] - y1 * s[2 * k + 1]);
      hi[k] = to_bf16x2(y0 * c[2 * k] + x0 * s[2 * k], y1 * c[2 * k + 1] + x1 * s[2 * k + 1]);
    }
    p.k_pool[dst] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    p.k_pool[dst + vph / 2] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    p.v_pool[dst] = p.v_new[src];
    p.v_pool[dst + vph / 2] = p.v_new[src + vph / 2];
  }
}

int launch_scatter(fb_ctx* ctx, const fb_pack* pk, const int32_t* page_table, const void* k_new,
                   const void* v_new, void* k_pool, void* v_pool, float rope_base, int32_t* status,
                   cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  ScatterParams p;
  p.n_live = pk->n_live; p.slot_req = pk->slot_req; p.slot_pos0 = pk->slot_pos0;
  p.page_table = page_table;
  p.k_new = static_cast<const uint4*>(k_new); p.v_new = static_cast<const uint4*>(v_new);
  p.k_pool = static_cast<uint4*>(k_pool); p.v_pool = static_cast<uint4*>(v_pool);
  p.status = status;
  p.bl = c.block_len; p.n_kv_heads = c.n_kv_heads; p.head_dim = c.head_dim;
  p.max_pages_per_req = c.max_pages_per_req; p.num_pages = c.num_pages;
  p.rope_base = rope_base;
  scatter_window_kv_kernel<<<c.max_requests * c.wmax, kScatterThreads, 0, stream>>>(p);
  return cuda_err(ctx, cudaGetLastError(), "scatter_window_kv_kernel launch");
}

}  // namespace fb
