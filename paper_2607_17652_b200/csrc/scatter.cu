// Data movement either side of the packed forward: fb_embed_gather (at the end of this
// file) and
// fb_scatter_window_kv: Eq. 6 as data movement.  The fresh K/V rows of every
// live window position go to the request's pages at their absolute positions
// (all KV heads), optionally with the rotary embedding applied to the keys.
// HBM-bound: 2 x rows x Hkv x d x 2 bytes read and as many written.
//
// One to four CTAs per slot (the slot's tokens are dealt among them).  For a (token, head) the head_dim elements are contiguous
// in the source (slot-order rows) and in the destination (pool row of that
// position), so a thread moves 16-byte pieces: with the rotary embedding a
// thread owns the two pieces that hold elements i and i + d/2 of eight pairs,
// and the rotation angles come from a per-slot table in shared memory.
#include <cuda_fp8.h>

#include <cmath>

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
  const float *k_scale, *v_scale;   // 8-bit pages: [n_kv_heads]
  double inv_freq[64];              // rope_base^(-2k/d), k < d/2 (formed on the host in fp64)
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t to_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// stored byte of x under `scale`: the binary32 quotient, rounded to nearest even onto the E4M3
// grid, saturating at +-448
__device__ __forceinline__ uint32_t e4m3x4(float a, float b, float c, float d, float scale) {
  const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(a, scale), __fdiv_rn(b, scale)), __NV_SATFINITE, __NV_E4M3);
  const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(c, scale), __fdiv_rn(d, scale)), __NV_SATFINITE, __NV_E4M3);
  return lo | (hi << 16);
}
// eight bf16 (one 16-byte piece) -> eight E4M3 bytes
__device__ __forceinline__ uint2 quant8(const uint4 v, float scale) {
  return make_uint2(e4m3x4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y), scale),
                    e4m3x4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w), scale));
}

// F8: the pools hold E4M3 bytes (8-byte pieces instead of 16-byte ones), each value divided by
// the scale of its KV head before it is rounded.
template <bool F8>
__global__ void __launch_bounds__(kScatterThreads) scatter_window_kv_kernel(const ScatterParams p) {
  pdl_wait();
  const int slot = blockIdx.x;
  if (slot >= *p.n_live) return;
  const int r = p.slot_req[slot], pos0 = p.slot_pos0[slot];
  const int vph = p.head_dim / 8;                    // 16-byte pieces per (token, head)
  const int vpt = p.n_kv_heads * vph;                // ... per token
  const bool rope = p.rope_base > 0.f;
  // cos / sin of pos * base^(-2i/d), once per (token, pair) and shared by all KV heads, for
  // 32 tokens of the slot at a time; the angle is formed and reduced in fp64 (positions
  // reach tens of thousands of radians)
  constexpr int kTokBatch = 32;
  __shared__ float2 cs[kTokBatch * 64];              // [token of the batch][pair] (cos, sin), d/2 <= 64
  const int half = p.head_dim / 2;
  // work item = (token, head, piece); with the rotary embedding only the lower half of the
  // pieces is enumerated and each item also handles its partner piece + d/16
  const int per_head = rope ? vph / 2 : vph;
  // the slot's tokens are dealt to the gridDim.y CTAs of the slot (each builds the table of its
  // own tokens only)
  const int tpc = (p.bl + (int)gridDim.y - 1) / (int)gridDim.y;
  const int tbeg = (int)blockIdx.y * tpc, tend = min(p.bl, tbeg + tpc);
  for (int t0 = tbeg; t0 < tend; t0 += kTokBatch) {
  const int nt = min(kTokBatch, tend - t0);
  if (rope) {
    __syncthreads();                                 // the previous batch has been read
    for (int i = threadIdx.x; i < nt * half; i += kScatterThreads) {
      const int t = i / half, k = i % half;
      // angle in fp64, reduced to [-pi, pi] there; sine and cosine of the remainder in fp32
      const double ang = (double)(pos0 + t0 + t) * p.inv_freq[k];
      const double red = fma(-rint(ang * 0.15915494309189535), 6.283185307179586, ang);
      float sf, cf;
      sincosf((float)red, &sf, &cf);
      cs[i] = make_float2(cf, sf);
    }
    __syncthreads();
  }
  const int nh = p.n_kv_heads;
  const int total = nt * nh * per_head;
  for (int i = threadIdx.x; i < total; i += kScatterThreads) {
    const int tb = i / (nh * per_head), rem = i % (nh * per_head);
    const int t = t0 + tb;
    const int h = rem / per_head, v = rem % per_head;
    const int pos = pos0 + t, pidx = pos / kPage;
    if (pidx >= p.max_pages_per_req) { atomicOr(p.status, FB_ST_BAD_PAGE); continue; }
    const int page = p.page_table[(size_t)r * p.max_pages_per_req + pidx];
    if (page < 0 || page >= p.num_pages) { atomicOr(p.status, FB_ST_BAD_PAGE); continue; }
    const size_t src = (size_t)(slot * p.bl + t) * vpt + h * vph + v;
    const size_t dst = (((size_t)page * p.n_kv_heads + h) * kPage + pos % kPage) * vph + v;
    [[maybe_unused]] uint2* k8 = reinterpret_cast<uint2*>(p.k_pool);
    [[maybe_unused]] uint2* v8 = reinterpret_cast<uint2*>(p.v_pool);
    [[maybe_unused]] float ksc = 1.f, vsc = 1.f;
    if constexpr (F8) { ksc = p.k_scale[h]; vsc = p.v_scale[h]; }
    if (!rope) {
      if constexpr (F8) {
        k8[dst] = quant8(p.k_new[src], ksc);
        v8[dst] = quant8(p.v_new[src], vsc);
      } else {
        p.k_pool[dst] = p.k_new[src];
        p.v_pool[dst] = p.v_new[src];
      }
      continue;
    }
    const uint4 a = p.k_new[src], b = p.k_new[src + vph / 2];      // elements i0.. and i0 + d/2..
    float c[8], s[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float2 a2 = cs[tb * half + v * 8 + k];
      c[k] = a2.x; s[k] = a2.y;
    }
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    if constexpr (F8) {
      float lo[8], hi[8];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float x0 = bf16_lo(aw[k]), x1 = bf16_hi(aw[k]), y0 = bf16_lo(bw[k]), y1 = bf16_hi(bw[k]);
        lo[2 * k] = x0 * c[2 * k] - y0 * s[2 * k]; lo[2 * k + 1] = x1 * c[2 * k + 1] - y1 * s[2 * k + 1];
        hi[2 * k] = y0 * c[2 * k] + x0 * s[2 * k]; hi[2 * k + 1] = y1 * c[2 * k + 1] + x1 * s[2 * k + 1];
      }
      k8[dst] = make_uint2(e4m3x4(lo[0], lo[1], lo[2], lo[3], ksc), e4m3x4(lo[4], lo[5], lo[6], lo[7], ksc));
      k8[dst + vph / 2] = make_uint2(e4m3x4(hi[0], hi[1], hi[2], hi[3], ksc), e4m3x4(hi[4], hi[5], hi[6], hi[7], ksc));
      v8[dst] = quant8(p.v_new[src], vsc);
      v8[dst + vph / 2] = quant8(p.v_new[src + vph / 2], vsc);
    } else {
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
  }
}

static void fill_inv_freq(ScatterParams& p, int head_dim, float rope_base) {
  for (int k = 0; k < 64; ++k)
    p.inv_freq[k] = (rope_base > 0.f && k < head_dim / 2)
                        ? exp2(-2.0 * (double)k / (double)head_dim * log2((double)rope_base)) : 0.0;
}
// enough (token, head, piece) items per CTA to keep 256 threads busy: four CTAs per slot once a
// slot holds 32 tokens of at least four KV heads
static int scatter_ctas_per_slot(const fb_config& c) { return c.block_len >= 32 && c.n_kv_heads >= 4 ? 4 : 1; }

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
  p.k_scale = p.v_scale = nullptr;
  fill_inv_freq(p, c.head_dim, rope_base);
  const dim3 grid(c.max_requests * c.wmax, scatter_ctas_per_slot(c));
  return cuda_err(ctx, launch_pdl(scatter_window_kv_kernel<false>, grid, kScatterThreads, 0, stream, p),
                  "scatter_window_kv_kernel launch");
}

int launch_scatter_fp8(fb_ctx* ctx, const fb_pack* pk, const int32_t* page_table, const void* k_new,
                       const void* v_new, void* k_pool8, void* v_pool8, const float* k_scale, const float* v_scale,
                       float rope_base, int32_t* status, cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  ScatterParams p;
  p.n_live = pk->n_live; p.slot_req = pk->slot_req; p.slot_pos0 = pk->slot_pos0;
  p.page_table = page_table;
  p.k_new = static_cast<const uint4*>(k_new); p.v_new = static_cast<const uint4*>(v_new);
  p.k_pool = static_cast<uint4*>(k_pool8); p.v_pool = static_cast<uint4*>(v_pool8);
  p.status = status;
  p.bl = c.block_len; p.n_kv_heads = c.n_kv_heads; p.head_dim = c.head_dim;
  p.max_pages_per_req = c.max_pages_per_req; p.num_pages = c.num_pages;
  p.rope_base = rope_base;
  p.k_scale = k_scale; p.v_scale = v_scale;
  fill_inv_freq(p, c.head_dim, rope_base);
  const dim3 grid(c.max_requests * c.wmax, scatter_ctas_per_slot(c));
  return cuda_err(ctx, launch_pdl(scatter_window_kv_kernel<true>, grid, kScatterThreads, 0, stream, p),
                  "scatter_window_kv_kernel (8-bit pages) launch");
}

// fb_embed_gather: x[i, :] = table[qtok[i], :] for live rows; one warp per row, 16-byte pieces.
__global__ void __launch_bounds__(256) embed_gather_kernel(const int32_t* n_live, const int32_t* qtok,
                                                           const uint4* table, int table_rows, int vec_per_row,
                                                           uint4* x, int bl, int32_t* status) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= *n_live * bl) return;
  const int tok = qtok[row];
  if (tok < 0 || tok >= table_rows) { if (lane == 0) atomicOr(status, FB_ST_BAD_TOKEN); return; }
  const uint4* src = table + (size_t)tok * vec_per_row;
  uint4* dst = x + (size_t)row * vec_per_row;
  for (int v = lane; v < vec_per_row; v += 32) dst[v] = src[v];
}

int launch_embed(fb_ctx* ctx, const fb_pack* pk, const void* table, int table_rows, int hidden, void* x,
                 int32_t* status, cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  const int rows = c.max_requests * c.wmax * c.block_len;
  embed_gather_kernel<<<(rows + 7) / 8, 256, 0, stream>>>(pk->n_live, pk->qtok, static_cast<const uint4*>(table),
                                                        table_rows, hidden / 8, static_cast<uint4*>(x),
                                                        c.block_len, status);
  return cuda_err(ctx, cudaGetLastError(), "embed_gather_kernel launch");
}

}  // namespace fb
