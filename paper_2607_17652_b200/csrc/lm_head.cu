// fb_lm_head_t2t: the T2T row pass taken straight from the LM head.  z = x W^T
// (hidden states x [rows, hidden], head weights W [V, hidden], bf16, fp32
// accumulation on the tensor cores) is never written: the epilogue of every
// 128 x 256 output tile reduces its rows to (max, sum of exponentials, first
// index of the max), a second kernel merges the tiles of a row, and the Eq. 1
// update runs on the result as in fb_t2t_step.  What the fused form saves is
// the 2 V bytes per row that the stand-alone row pass has to read.
//
// Persistent, warp-specialised tcgen05 GEMM, one CTA per SM, 256 threads:
//   warp 0      TMA producer: A tile (128 rows of x) and B tile (256 rows of W)
//               per 64-element slice of the hidden dimension, 4 stages
//   warp 1      MMA issuer: 4 x tcgen05.mma (M 128, N 256, K 16) per stage into
//               one of two 256-column accumulators in TMEM
//   warps 4-7   epilogue: one thread per output row, 32 columns at a time
// Tiles are taken vocabulary-major (all row tiles of one 256-token slice of W
// next to each other), so W streams from HBM once and x stays in L2.
#include <cudaTypedefs.h>

#include <cfloat>

#include "fb_common.cuh"
#include "ptx_sm100.cuh"

namespace fb {

constexpr int kLmThreads = 256;
constexpr int kLmBM = 128, kLmBN = 256, kLmBK = 64, kLmStages = 4;
constexpr int kLmABytes = kLmBM * kLmBK * 2, kLmBBytes = kLmBN * kLmBK * 2;
constexpr int kLmStageBytes = kLmABytes + kLmBBytes;                 // 48 KB
constexpr int kLmSmem = kLmStages * kLmStageBytes + 2048;            // + barriers + 1 KB alignment slack
constexpr float kLmLog2e = 1.4426950408889634f;

struct LmParams {
  const int32_t* n_live;
  float4* part;          // [n_tiles_n][rows_pad] (max, sum exp, first index of the max as bits, -)
  int32_t* status;
  int32_t bl, vocab, hidden, n_tiles_n, rows_pad;
  long long wait_cycles;
};

__device__ __forceinline__ bool lm_warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort, long long limit) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort, limit));
}

__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_stats_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                     const LmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kLmStages * kLmStageBytes);
  uint64_t* full = bars;                    // [4] stage filled (TMA bytes)
  uint64_t* empty = bars + 4;               // [4] stage consumed (MMA commit)
  uint64_t* acc_full = bars + 8;            // [2] accumulator complete (MMA commit)
  uint64_t* acc_empty = bars + 10;          // [2] accumulator read out (4 epilogue warps)
  uint64_t* drain = bars + 13;              // give-up path only
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 12);
  volatile int* abortf = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long LIM = p.wait_cycles;
  if (tid == 0) {
    *abortf = 0;
    for (int i = 0; i < kLmStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
    mbar_init(drain, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmW);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int live_rows = *p.n_live * p.bl;
  const int m_tiles = (live_rows + kLmBM - 1) / kLmBM;          // row tiles that hold live rows
  const int n_tiles = m_tiles * p.n_tiles_n;
  const int k_blocks = p.hidden / kLmBK;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    const bool leader = elect_one();
    int fill = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
      const int n = t / m_tiles, m = t % m_tiles;
      for (int kb = 0; kb < k_blocks; ++kb, ++fill) {
        const int st = fill % kLmStages, round = fill / kLmStages;
        if (round > 0 && !lm_warp_wait(&empty[st], (round - 1) & 1, abortf, LIM)) { ok = false; break; }
        if (leader) {
          uint8_t* a = smem + st * kLmStageBytes;
          mbar_arrive_expect_tx(&full[st], kLmStageBytes);
          tma_load_2d(a, &tmX, &full[st], kb * kLmBK, m * kLmBM);
          tma_load_2d(a + kLmABytes, &tmW, &full[st], kb * kLmBK, n * kLmBN);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer
    const bool leader = elect_one();
    const uint32_t idesc = umma_idesc_bf16(kLmBM, kLmBN, 0, 0);
    const uint64_t dA0 = smem_desc_sw128(smem_u32(smem), 16, 1024);
    const uint64_t dB0 = smem_desc_sw128(smem_u32(smem + kLmABytes), 16, 1024);
    int fill = 0, i = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
      const int b = i & 1;
      if (i >= 2 && !lm_warp_wait(&acc_empty[b], ((i >> 1) - 1) & 1, abortf, LIM)) { ok = false; break; }
      tc_fence_after();
      for (int kb = 0; kb < k_blocks; ++kb, ++fill) {
        const int st = fill % kLmStages, round = fill / kLmStages;
        if (!lm_warp_wait(&full[st], round & 1, abortf, LIM)) { ok = false; break; }
        tc_fence_after();
        if (leader) {
          const uint32_t so = (uint32_t)((st * kLmStageBytes) >> 4);
#pragma unroll
          for (int ks = 0; ks < kLmBK / 16; ++ks)
            umma_ss(tmem + b * kLmBN, dA0 + so + (uint32_t)((ks * 32) >> 4), dB0 + so + (uint32_t)((ks * 32) >> 4),
                    idesc, (kb > 0 || ks > 0) ? 1u : 0u);
          umma_commit(&empty[st]);
          if (kb == k_blocks - 1) umma_commit(&acc_full[b]);
        }
        __syncwarp();
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------ epilogue
    const int quad = warp & 3;
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    int i = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
      const int n = t / m_tiles, m = t % m_tiles, b = i & 1;
      if (!lm_warp_wait(&acc_full[b], (i >> 1) & 1, abortf, LIM)) { ok = false; break; }   // one outcome per warp
      tc_fence_after();
      const uint32_t tacc = tmem + lane_base + b * kLmBN;
      const int col0 = n * kLmBN;
      float mx = -INFINITY, sum = 0.f;
      int arg = 0x7fffffff;
      uint32_t buf[2][32];
      tmem_ld32(tacc, buf[0]);
#pragma unroll
      for (int c = 0; c < kLmBN / 32; ++c) {
        const uint32_t* v = buf[c & 1];
        tmem_ld_wait();
        if (c + 1 < kLmBN / 32) tmem_ld32(tacc + (c + 1) * 32, buf[(c + 1) & 1]);
        const int valid = min(32, p.vocab - (col0 + c * 32));        // columns of this chunk inside the vocabulary
        float cm = -INFINITY;
#pragma unroll
        for (int j = 0; j < 32; ++j) cm = fmaxf(cm, j < valid ? __uint_as_float(v[j]) : -INFINITY);
        if (cm > mx) {                                              // strict: an equal later maximum keeps the first index
          int first = 31;
#pragma unroll
          for (int j = 31; j >= 0; --j) if (j < valid && __uint_as_float(v[j]) == cm) first = j;
          sum *= ex2_approx((mx - cm) * kLmLog2e);                    // 0 * 2^-inf = 0 on the first chunk
          mx = cm; arg = col0 + c * 32 + first;
        }
        const float mb = mx * kLmLog2e;
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 32; ++j)
          s4[j & 3] += j < valid ? ex2_approx(fmaf(__uint_as_float(v[j]), kLmLog2e, -mb)) : 0.f;
        sum += (s4[0] + s4[1]) + (s4[2] + s4[3]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[b]);
      const int row = m * kLmBM + quad * 32 + lane;
      if (row < live_rows)
        p.part[(size_t)n * p.rows_pad + row] = make_float4(mx, sum, __int_as_float(arg), 0.f);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abortf) {
    // give-up path: the MMA warp waits for everything it has issued (own barrier, bounded
    // polls), copies in flight land while the CTA sleeps, then TMEM and shared memory go back
    if (tid == 0) atomicOr(p.status, FB_ST_DEV_TIMEOUT);
    if (warp == 1) {
      if (elect_one()) umma_commit(drain);
      __syncwarp();
      for (int i = 0; i < 4096 && !mbar_test(drain, 0); ++i) __nanosleep(200);
    }
    for (int i = 0; i < 64; ++i) __nanosleep(10000);
    __syncthreads();
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// Tiles of a row -> top-1 token (lowest index on ties) and its confidence 1 / sum exp(z - max).
__global__ void __launch_bounds__(256) lm_head_merge_kernel(const LmParams p, int32_t* argmax, float* conf,
                                                            int max_rows) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= max_rows) return;
  if (row >= *p.n_live * p.bl) {
    if (lane == 0) { argmax[row] = -1; conf[row] = 0.f; }
    return;
  }
  float M = -INFINITY;
  for (int n = lane; n < p.n_tiles_n; n += 32) M = fmaxf(M, p.part[(size_t)n * p.rows_pad + row].x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float S = 0.f;
  int arg = 0x7fffffff;
  for (int n = lane; n < p.n_tiles_n; n += 32) {
    const float4 q = p.part[(size_t)n * p.rows_pad + row];
    S += q.y * ex2_approx((q.x - M) * kLmLog2e);
    if (q.x == M) arg = min(arg, __float_as_int(q.z));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    S += __shfl_xor_sync(0xffffffffu, S, o);
    arg = min(arg, __shfl_xor_sync(0xffffffffu, arg, o));
  }
  if (lane == 0) {
    if (!(S >= 1.0f) || S > FLT_MAX || arg == 0x7fffffff) {
      atomicOr(p.status, FB_ST_NAN_LOGIT);
      argmax[row] = arg == 0x7fffffff ? 0 : arg;
      conf[row] = 0.f;
    } else {
      argmax[row] = arg;
      conf[row] = 1.0f / S;
    }
  }
}

static int lm_rows_pad(const fb_config& c) {
  const int rows = c.max_requests * c.wmax * c.block_len;
  return (rows + kLmBM - 1) / kLmBM * kLmBM;
}

size_t lm_head_workspace_bytes(const fb_ctx* ctx) {
  const fb_config& c = ctx->cfg;
  const size_t n_tiles_n = (c.vocab + kLmBN - 1) / kLmBN;
  return n_tiles_n * (size_t)lm_rows_pad(c) * sizeof(float4);
}

// per-device kernel attribute (called from ensure_device with that device current)
int lm_head_device_setup(fb_ctx* ctx) {
  return cuda_err(ctx, cudaFuncSetAttribute(lm_head_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kLmSmem), "smem attr");
}

int launch_lm_head(fb_ctx* ctx, const fb_pack* pk, const void* x, const void* w, int hidden, const fb_state* st,
                   int32_t* argmax, float* conf, uint8_t* action, int32_t* slot_stats, void* ws, int32_t* status,
                   cudaStream_t stream) {
  if (int e = ensure_device(ctx)) return e;
  const fb_config& c = ctx->cfg;
  const int rows = c.max_requests * c.wmax * c.block_len;
  auto fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(ctx->encode_fn);
  CUtensorMap tmX, tmW;
  const cuuint32_t es[2] = {1, 1};
  {
    const cuuint64_t dims[2] = {(cuuint64_t)hidden, (cuuint64_t)rows};
    const cuuint64_t str[1] = {(cuuint64_t)hidden * 2};
    const cuuint32_t box[2] = {kLmBK, kLmBM};
    if (fn(&tmX, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, str, box, es,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return set_err(ctx, FB_ERR_CUDA, "cuTensorMapEncodeTiled failed for x");
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)hidden, (cuuint64_t)c.vocab};
    const cuuint64_t str[1] = {(cuuint64_t)hidden * 2};
    const cuuint32_t box[2] = {kLmBK, kLmBN};
    if (fn(&tmW, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w), dims, str, box, es,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return set_err(ctx, FB_ERR_CUDA, "cuTensorMapEncodeTiled failed for w");
  }
  LmParams p;
  p.n_live = pk->n_live;
  p.part = static_cast<float4*>(ws);
  p.status = status;
  p.bl = c.block_len; p.vocab = c.vocab; p.hidden = hidden;
  p.n_tiles_n = (c.vocab + kLmBN - 1) / kLmBN;
  p.rows_pad = lm_rows_pad(c);
  p.wait_cycles = ctx->wait_cycles;
  lm_head_stats_kernel<<<ctx->num_sms, kLmThreads, kLmSmem, stream>>>(tmX, tmW, p);
  if (int e = cuda_err(ctx, cudaGetLastError(), "lm_head_stats_kernel launch")) return e;
  lm_head_merge_kernel<<<(rows + 7) / 8, 256, 0, stream>>>(p, argmax, conf, rows);
  if (int e = cuda_err(ctx, cudaGetLastError(), "lm_head_merge_kernel launch")) return e;
  return launch_t2t_update(ctx, pk, st, argmax, conf, action, slot_stats, stream);
}

}  // namespace fb
