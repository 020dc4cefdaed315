// fb_t2t_step: the token-to-token step over the logits (Sec. 2.1, Eq. 1; the
// counts of Eq. 2).
//
// Kernel 1 (bandwidth-bound): one CTA (128 threads, eight 16-byte loads in
// flight each: the best of the shapes tried) per live row, or a cluster of two
// CTAs per row when the batch has few rows, streams the row's bf16
// logits once with 16-byte loads and keeps, per thread, a running
// (max, first index of the max, sum of exp relative to that max); a
// warp-shuffle + shared-memory reduction merges them with the lowest-index
// rule.  Output: top-1 token and its softmax probability 1 / sum exp(z - max).
// Kernel 2 (tiny): one warp per slot applies Eq. 1 to the slot's bl positions,
// updates the tokens in place and produces the per-block counts.
#include <cfloat>

#include <cooperative_groups.h>

#include "fb_common.cuh"

namespace fb {

constexpr int kRowThreads = 128;
constexpr int kRowUnroll = 8;   // 16-byte loads in flight per thread
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct RowAcc {
  float m;    // running max
  float s;    // sum of exp(z - m)
  int idx;    // first index where z == m
};

__device__ __forceinline__ void merge(RowAcc& a, const RowAcc& b) {
  // lowest index wins ties; sums are rescaled to the larger max
  if (b.m > a.m || (b.m == a.m && b.idx < a.idx)) {
    const float sc = a.m == -INFINITY ? 0.f : fast_ex2((a.m - b.m) * kLog2e);
    a.s = a.s * sc + b.s; a.m = b.m; a.idx = b.idx;
  } else {
    const float sc = b.m == -INFINITY ? 0.f : fast_ex2((b.m - a.m) * kLog2e);
    a.s += b.s * sc;
  }
}

__device__ __forceinline__ void absorb8(RowAcc& a, const uint4 v, int base) {
  float z[8] = {bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y),
                bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w)};
  float cm = fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), fmaxf(fmaxf(z[4], z[5]), fmaxf(z[6], z[7])));
  if (cm > a.m) {                       // rare after the first few chunks
    a.s *= a.m == -INFINITY ? 0.f : fast_ex2((a.m - cm) * kLog2e);
    a.m = cm;
    int k = 7;
#pragma unroll
    for (int i = 6; i >= 0; --i) k = z[i] == cm ? i : k;
    a.idx = base + k;
  }
  if (a.m == -INFINITY) return;          // nothing but -inf so far: contributes 0
  const float mb = a.m * kLog2e;
  float acc = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) acc += fast_ex2(fmaf(z[i], kLog2e, -mb));
  a.s += acc;
}

__global__ void __launch_bounds__(kRowThreads)
t2t_rows_kernel(const uint4* __restrict__ logits, const int32_t* __restrict__ n_live, int bl, int nvec,
                int32_t* __restrict__ argmax, float* __restrict__ conf, int32_t* __restrict__ status) {
  pdl_wait();
  // a cluster of cl CTAs shares one row: CTA `rank` streams the rank-th piece of it and rank 0
  // merges the pieces through distributed shared memory (cl == 1: the whole row, no exchange)
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int cl = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int row = blockIdx.x / cl;
  const int tid = threadIdx.x;
  if (row >= *n_live * bl) {            // padding slot: no bytes read (the whole cluster leaves)
    if (tid == 0 && rank == 0) { argmax[row] = -1; conf[row] = 0.f; }
    return;
  }
  const int seg = (nvec + cl - 1) / cl;
  const int vend = min(nvec, (rank + 1) * seg);
  const uint4* p = logits + (size_t)row * nvec;
  RowAcc a{-INFINITY, 0.f, 0x7fffffff};
  int i = rank * seg + tid;
  for (; i + (kRowUnroll - 1) * kRowThreads < vend; i += kRowUnroll * kRowThreads) {
    uint4 v[kRowUnroll];
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) v[u] = ld_stream16(p + i + u * kRowThreads);
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) absorb8(a, v[u], (i + u * kRowThreads) * 8);
  }
  for (; i < vend; i += kRowThreads) absorb8(a, ld_stream16(p + i), i * 8);
  // warp reduce
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    RowAcc b;
    b.m = __shfl_xor_sync(0xffffffffu, a.m, o);
    b.s = __shfl_xor_sync(0xffffffffu, a.s, o);
    b.idx = __shfl_xor_sync(0xffffffffu, a.idx, o);
    merge(a, b);
  }
  __shared__ RowAcc sh[kRowThreads / 32];
  if ((tid & 31) == 0) sh[tid >> 5] = a;
  __syncthreads();
  RowAcc b{-INFINITY, 0.f, 0x7fffffff};
  auto warp_merge = [&](int from) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      if (o > from) continue;
      RowAcc c;
      c.m = __shfl_xor_sync(0xffffffffu, b.m, o);
      c.s = __shfl_xor_sync(0xffffffffu, b.s, o);
      c.idx = __shfl_xor_sync(0xffffffffu, b.idx, o);
      merge(b, c);
    }
  };
  if (tid < 32) {
    if (tid < kRowThreads / 32) b = sh[tid];
    warp_merge(16);
  }
  if (cl > 1) {                          // uniform over the cluster
    __shared__ RowAcc part;
    if (tid == 0) part = b;
    cluster.sync();
    if (rank == 0 && tid < 32) {
      b = tid < cl ? *cluster.map_shared_rank(&part, tid) : RowAcc{-INFINITY, 0.f, 0x7fffffff};
      warp_merge(4);                     // cl <= 8
    }
    cluster.sync();                      // the pieces stay put until rank 0 has read them
    if (rank != 0) return;
  }
  if (tid == 0) {
    const float pr = 1.0f / b.s;         // the max itself contributes exp(0) = 1
    if (!(b.s >= 1.0f) || !(pr == pr) || b.s > FLT_MAX) {
      atomicOr(status, FB_ST_NAN_LOGIT);
      argmax[row] = b.idx == 0x7fffffff ? 0 : b.idx;
      conf[row] = 0.f;
    } else {
      argmax[row] = b.idx;
      conf[row] = pr;
    }
  }
}

struct UpdParams {
  const int32_t *n_live, *slot_req, *slot_s, *L;
  int32_t* tokens;
  const int32_t* argmax;
  const float* conf;
  uint8_t* action;
  int32_t* slot_stats;
  int32_t max_slots, bl, max_blocks, mask_id, eos_id;
  float tau_mask, tau_edit;
  int32_t delta_literal, force_progress;
};

__global__ void __launch_bounds__(128) t2t_update_kernel(const UpdParams p) {
  pdl_wait();
  const int slot = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (slot >= p.max_slots) return;
  if (slot >= *p.n_live) {
    for (int t = lane; t < p.bl; t += 32) p.action[slot * p.bl + t] = 0;
    if (lane < FB_SLOT_STATS) p.slot_stats[slot * FB_SLOT_STATS + lane] = 0;
    return;
  }
  const int r = p.slot_req[slot];
  const int g = p.L[r] + p.slot_s[slot];
  int32_t* tok = p.tokens + (size_t)r * p.max_blocks * p.bl + (size_t)g * p.bl;
  int m0 = 0, rdy = 0, m2t = 0, t2t = 0, m1 = 0, eos = 0;
  float bestp = -1.f;                               // most confident mask this lane left in place
  int bestt = 0x7fffffff;
  for (int t = lane; t < p.bl; t += 32) {
    const int i = slot * p.bl + t;
    int x = tok[t];
    const int xh = p.argmax[i];
    const float pr = p.conf[i];
    uint8_t act = FB_ACT_NONE;
    if (x == p.mask_id) {                         // Gamma of Eq. 1: strict >
      m0++;
      rdy += pr >= p.tau_mask;                    // Eq. 2 numerator: >=
      // Delta as printed has no "revealed" condition: with delta_literal a mask whose
      // prediction is not [M] itself is updated once p > tau_edit as well
      if (pr > p.tau_mask || (p.delta_literal && x != xh && pr > p.tau_edit)) { x = xh; act = FB_ACT_M2T; m2t++; }
      else if (pr > bestp) { bestp = pr; bestt = t; }
    } else if (x != xh && pr > p.tau_edit) {      // Delta of Eq. 1, revealed only
      x = xh; act = FB_ACT_T2T; t2t++;
    }
    if (act) tok[t] = x;
    p.action[i] = act;
    m1 += x == p.mask_id;
    eos |= x == p.eos_id;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    m0 += __shfl_xor_sync(0xffffffffu, m0, o);
    rdy += __shfl_xor_sync(0xffffffffu, rdy, o);
    m2t += __shfl_xor_sync(0xffffffffu, m2t, o);
    t2t += __shfl_xor_sync(0xffffffffu, t2t, o);
    m1 += __shfl_xor_sync(0xffffffffu, m1, o);
    eos |= __shfl_xor_sync(0xffffffffu, eos, o);
  }
  // forced progress: the oldest block went in with masks and Eq. 1 revealed none -> its most
  // confident masked position (lowest position on ties) is revealed
  if (p.force_progress && p.slot_s[slot] == 0 && m0 > 0 && m2t == 0) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float op = __shfl_xor_sync(0xffffffffu, bestp, o);
      const int ot = __shfl_xor_sync(0xffffffffu, bestt, o);
      if (op > bestp || (op == bestp && ot < bestt)) { bestp = op; bestt = ot; }
    }
    const int xh = p.argmax[slot * p.bl + bestt];
    if (lane == 0) { tok[bestt] = xh; p.action[slot * p.bl + bestt] = FB_ACT_FORCED; }
    m2t = 1; m1 -= xh != p.mask_id; eos |= xh == p.eos_id;
  }
  if (lane == 0) {
    int32_t* s = p.slot_stats + slot * FB_SLOT_STATS;
    s[FB_STAT_M0] = m0; s[FB_STAT_RDY] = rdy; s[FB_STAT_M2T] = m2t; s[FB_STAT_T2T] = t2t; s[FB_STAT_M1] = m1;
    s[FB_STAT_EOS] = eos;
  }
}

int launch_t2t(fb_ctx* ctx, const fb_pack* pk, const void* logits, const fb_state* st, int32_t* argmax,
               float* conf, uint8_t* action, int32_t* slot_stats, int32_t* status, cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  const int max_slots = c.max_requests * c.wmax;
  const int rows = max_slots * c.block_len;
  // few rows: a pair of CTAs per row (measured on 1024 rows of 151,936 logits: 42 us against
  // 50 us for one CTA per row, 45 us for four, 50 us for eight; on 8192 rows a pair loses 6 %)
  const int cl = rows >= 2048 ? 1 : 2;
  if (int e = cuda_err(ctx, launch_pdl_cluster(t2t_rows_kernel, rows * cl, kRowThreads, 0, stream, cl,
                                               static_cast<const uint4*>(logits), pk->n_live, c.block_len,
                                               c.vocab / 8, argmax, conf, status),
                       "t2t_rows_kernel launch"))
    return e;
  return launch_t2t_update(ctx, pk, st, argmax, conf, action, slot_stats, stream);
}

// Eq. 1 and the block counts from (argmax, conf), whoever produced them.
int launch_t2t_update(fb_ctx* ctx, const fb_pack* pk, const fb_state* st, const int32_t* argmax, const float* conf,
                      uint8_t* action, int32_t* slot_stats, cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  const int max_slots = c.max_requests * c.wmax;
  UpdParams u;
  u.n_live = pk->n_live; u.slot_req = pk->slot_req; u.slot_s = pk->slot_s; u.L = st->L; u.tokens = st->tokens;
  u.argmax = argmax; u.conf = conf; u.action = action; u.slot_stats = slot_stats;
  u.max_slots = max_slots; u.bl = c.block_len; u.max_blocks = c.max_blocks; u.mask_id = c.mask_id;
  u.eos_id = c.eos_id; u.tau_mask = c.tau_mask; u.tau_edit = c.tau_edit;
  u.delta_literal = c.delta_literal; u.force_progress = c.force_progress;
  return cuda_err(ctx, launch_pdl(t2t_update_kernel, (max_slots + 3) / 4, 128, 0, stream, u), "t2t_update_kernel launch");
}

}  // namespace fb
