/* flowblock.h -- C ABI of the packed-wavefront decode step (sm_100a).
 *
 * One decode step of Gated Wavefront Decoding under Heterogeneous Wavefront
 * Packing is four stream-ordered calls:
 *
 *   fb_pack_wavefronts   per-request windows (L_b, R_b) -> dense slot batch
 *   fb_wavefront_attn    W-shaped block-causal GQA attention over the slots
 *   fb_t2t_step          top-1 / confidence per row, joint M2T u T2T update
 *   fb_gate_commit       in-order retirement, KV freeze, readiness-gated
 *                        admission
 *
 * Conventions
 *   - Every function returns FB_OK (0) or a negative fb_error.  After an
 *     error fb_last_error(ctx) returns a human-readable host string.
 *   - Unless stated otherwise every pointer inside fb_state / fb_pack and
 *     every tensor argument is a DEVICE pointer owned by the caller, at
 *     least 16-byte aligned.  The library never frees or reallocates them.
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*)
 *     and never synchronise.  Nothing is allocated after fb_create; scratch
 *     comes from the caller's workspace of fb_workspace_bytes(ctx) bytes.
 *   - Data-dependent problems (a page id out of range, a window wider than
 *     W, a wait that ran out of time) never trap: the kernel skips the
 *     offending access and ORs an fb_status bit into the caller's device
 *     int32 `status` word.
 *   - A "slot" is one live block of one request.  Slots are numbered in
 *     (request, block) order; there are max_slots = max_requests * wmax of
 *     them and the first *n_live are in use.  Row i of a [max_slots*bl, ...]
 *     tensor is token i % bl of slot i / bl.
 *   - K/V memory that a request's page table or the window tensors cover must
 *     hold finite values even where it is masked out (masked entries get
 *     weight exactly 0, and 0 * inf is not 0).
 *   - A context belongs to one host thread at a time and to one device at a
 *     time: the calls cache per-device set-up and tensor-map descriptors
 *     inside it.  Use one context per thread / device; contexts are cheap.
 *   - No environment variable is read anywhere.
 */
#ifndef FLOWBLOCK_H
#define FLOWBLOCK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FB_OK = 0,
  FB_ERR_INVALID_ARG = -1, /* null pointer, non-positive size            */
  FB_ERR_SHAPE = -2,       /* sizes inconsistent with each other         */
  FB_ERR_ALIGNMENT = -3,   /* a pointer is not 16-byte aligned           */
  FB_ERR_UNSUPPORTED = -4, /* shape outside what the kernels implement   */
  FB_ERR_WORKSPACE = -5,   /* workspace missing                          */
  FB_ERR_CUDA = -6         /* a CUDA runtime / driver call failed        */
} fb_error;

typedef enum {
  FB_ST_BAD_PAGE = 1,     /* page id outside [0, num_pages): tile skipped */
  FB_ST_BAD_TOKEN = 2,    /* fb_embed_gather: token id outside the table  */
  FB_ST_BAD_STATE = 4,    /* R-L outside [0, wmax] or L,R outside [0, n]  */
  FB_ST_NAN_LOGIT = 8,    /* a row's softmax sum was not finite           */
  FB_ST_DEV_TIMEOUT = 16  /* a bounded device-side wait gave up           */
} fb_status;

enum { FB_FLAG_OLDEST = 1, FB_FLAG_FRONTIER = 2 };          /* slot_flags  */
enum { FB_ACT_NONE = 0, FB_ACT_M2T = 1, FB_ACT_T2T = 2,
       FB_ACT_FORCED = 3 /* force_progress reveal */ };     /* action code */
/* slot_stats columns */
enum { FB_STAT_M0 = 0, FB_STAT_RDY, FB_STAT_M2T, FB_STAT_T2T, FB_STAT_M1, FB_STAT_EOS,
       FB_SLOT_STATS = 6 };
/* step_counters entries */
enum { FB_CT_BLOCKS = 0, FB_CT_TOKENS, FB_CT_SPAWNED, FB_CT_FINISHED,
       FB_CT_M2T, FB_CT_T2T, FB_CT_LIVE_SLOTS, FB_CT_ACTIVE,
       FB_CT_LOCKSTEP_COMMIT, /* batch_sync: window positions the batch retired */
       FB_CT_LOCKSTEP_ADMIT,  /* batch_sync: 1 if the batch admitted a block    */
       FB_STEP_COUNTERS = 10 };

typedef struct fb_ctx fb_ctx;

/* Immutable per context.  Notation follows the paper: W (wmax), bl
 * (block_len), n (max_blocks), tau_mask / tau_edit (Eq. 1), theta_spawn
 * (Eq. 3), S_pe (Sec. 2.1). */
typedef struct {
  int32_t max_requests;      /* R_max >= 1                                  */
  int32_t wmax;              /* W, window bound, 1..8                       */
  int32_t block_len;         /* bl; bl * (n_q_heads/n_kv_heads) % 128 == 0  */
  int32_t n_q_heads;
  int32_t n_kv_heads;        /* divides n_q_heads; group size divides 128   */
  int32_t head_dim;          /* 64 or 128                                   */
  int32_t page_size;         /* 64                                          */
  int32_t num_pages;         /* pages in the shared K and V pools           */
  int32_t max_pages_per_req; /* columns of the page table                   */
  int32_t vocab;             /* V, multiple of 8                            */
  int32_t mask_id;           /* token id of [M] (may be >= vocab)           */
  int32_t eos_id;            /* -1: none                                    */
  int32_t max_blocks;        /* n, generation blocks per request            */
  int32_t s_pe;              /* S_pe, post-edit forwards, 0..255            */
  float tau_mask;
  float tau_edit;            /* >= tau_mask unless delta_literal = 1        */
  float theta_spawn;
  float sm_scale;            /* 0 -> 1/sqrt(head_dim)                       */
  int32_t window_in_pages;   /* 0: this step's window K/V are passed to the
                                attention and copied to the pages when a block
                                retires.  1: they are scattered to the pages
                                every step (fb_scatter_window_kv, Eq. 6), the
                                attention reads every key through the page
                                table and retirement copies nothing          */
  int32_t batch_sync;        /* 0: per-sequence wavefronts (Sec. 3.2).  1: the
                                batch-synchronous wavefront that Sec. 3.2 and
                                the packing ablation set against them: window
                                position c retires only when it is finished in
                                every decoding sequence, and one block per
                                sequence is admitted only when every sequence
                                clears the gate (min over the batch of rho)
                                and has room                                 */
  int32_t delta_literal;     /* 0: Delta of Eq. 1 on revealed positions only
                                (the prose's reading; needs tau_edit >=
                                tau_mask).  1: Delta as printed: a masked
                                position whose prediction is not [M] is also
                                updated once p > tau_edit; tau_edit may then
                                be below tau_mask                            */
  int32_t force_progress;    /* 1: when the oldest live block of a request
                                went into the forward with masks and Eq. 1
                                revealed none, its most confident masked
                                position (lowest position on ties, binary32
                                compare) is revealed (action FB_ACT_FORCED,
                                counted as M2T).  Not in the paper: Eq. 1 is
                                threshold-only; off by default               */
  int32_t kv_fp8;            /* 1: the pools are FP8 E4M3 bytes with per-KV-head
                                scales (fb_scatter_window_kv_fp8,
                                fb_wavefront_attn_fp8); needs window_in_pages =
                                1 and head_dim = 128.  0: bf16 pools          */
} fb_config;

/* Per-request wavefront state (Sec. 3.2: (L_b, R_b), in-order commit
 * pointer).  The caller admits / removes requests by writing rows between
 * steps. */
typedef struct {
  int32_t* active;      /* [R_max] 0 free, 1 decoding, 2 done               */
  int32_t* prefix_len;  /* [R_max] o_b: tokens in the frozen prefix
                           (prompt + committed blocks)                      */
  int32_t* L;           /* [R_max] oldest live block                        */
  int32_t* R;           /* [R_max] one past the frontier block; 0<=L<=R<=n  */
  int32_t* tokens;      /* [R_max, n*bl] generation region; mask_id = [M]   */
  uint8_t* pe_done;     /* [R_max, wmax] post-edit forwards seen, by slot   */
  int32_t* page_table;  /* [R_max, max_pages_per_req] page of absolute
                           positions [64 j, 64 j + 64); must cover
                           prefix_len + wmax*bl positions                    */
} fb_state;

/* Output of fb_pack_wavefronts, input of the other three calls. */
typedef struct {
  int32_t* n_live;          /* [1]                                          */
  int32_t* slot_req;        /* [max_slots] request index, -1 = padding      */
  int32_t* slot_s;          /* [max_slots] window slot index s = g - L      */
  int32_t* slot_pos0;       /* [max_slots] absolute position of token 0     */
  int32_t* slot_kv_len;     /* [max_slots] keys visible: o_b + (s+1) bl     */
  int32_t* slot_flags;      /* [max_slots] FB_FLAG_*                        */
  int32_t* req_slot_begin;  /* [R_max+1] CSR over requests                  */
  int32_t* qtok;            /* [max_slots*bl] gathered tokens (Eq. 4)       */
  int32_t* pos;             /* [max_slots*bl] absolute position ids (Eq. 4) */
} fb_pack;

/* Validates the configuration and creates a context (host memory only; no
 * CUDA call is made).  FB_ERR_UNSUPPORTED for shapes the kernels do not
 * implement, including tau_edit < tau_mask without delta_literal. */
int fb_create(const fb_config* cfg, fb_ctx** out);
int fb_destroy(fb_ctx* ctx);
const char* fb_last_error(const fb_ctx* ctx); /* ctx may be NULL */

/* Execution knobs; no result depends on them beyond the rounding order of the
 * split-KV merge.  The paper has no counterpart (it states no kernel design).
 * 0 in a field selects the default. */
typedef struct {
  int32_t attn_target_items;     /* work items the key-axis split aims for
                                    (default 2 x 148: two per SM); 1 = never
                                    split, large = split down to the minimum  */
  int32_t attn_min_chunk_tiles;  /* shortest key range of a split piece, in
                                    128-key tiles (default 4)                 */
  int32_t attn_pair;             /* 1: four Q tiles of one request and KV head
                                    at a time run on a pair of CTAs that share
                                    every K/V tile (tcgen05 cta_group::2; bf16
                                    pages and head_dim 128 only), the remaining
                                    tiles on single CTAs.  Off by default: on
                                    the measured workloads the single-CTA
                                    kernel alone is faster                     */
  int32_t reserved;              /* 0                                         */
  int64_t wait_cycles;           /* limit of every bounded device-side wait
                                    (mbarrier, hand-off flags) in SM clock
                                    cycles (default 2e9, about a second); when
                                    it runs out the kernel stops issuing work,
                                    sets FB_ST_DEV_TIMEOUT and returns.  -1 is
                                    the self-test of that path: every wait
                                    gives up at once, so fb_wavefront_attn and
                                    fb_lm_head_t2t do no useful work, set the
                                    status bit and return (outputs undefined);
                                    the next call with a positive limit runs
                                    normally                                   */
} fb_tuning;

/* Applies `t` to the context.  Changes fb_workspace_bytes(ctx): query it
 * again and call before the first step.  FB_ERR_INVALID_ARG for negative or
 * out-of-range values (attn_target_items <= 2^20, attn_min_chunk_tiles <=
 * 4096). */
int fb_set_tuning(fb_ctx* ctx, const fb_tuning* t);

/* Bytes of device scratch the caller must pass as `ws` (256-byte aligned) to
 * fb_pack_wavefronts and fb_wavefront_attn of the same step: the attention
 * work list and the split-KV partial results. */
size_t fb_workspace_bytes(const fb_ctx* ctx);

/* Host-side mirror of the attention work-list arithmetic that
 * fb_pack_wavefronts runs on the device (the paper has no counterpart: the
 * work list is this library's execution plan).  For n <= max_requests decoding
 * requests with HOST arrays h_prefix_len[n] and h_live_blocks[n] (R - L of
 * each) it writes twelve int32 to h_out, six per work list (first the list of
 * the one-CTA kernel, then the list of the CTA-pair kernel): unit records,
 * work items and split pieces the batch produces, then the capacities
 * max_units, max_items, max_parts that the workspace of this context is sized
 * for.  No CUDA call is made. */
int fb_attn_plan_host(const fb_ctx* ctx, const int32_t* h_prefix_len,
                      const int32_t* h_live_blocks, int32_t n, int32_t* h_out);

/* Sec. 3.2, Eq. 4 (gather): compacts the live blocks of all decoding
 * requests into slots, writes every array of `out`, pads the rest
 * (slot_req = -1, qtok = mask_id, pos = 0) and builds the attention work
 * list inside `ws`.  Reads st->{active, prefix_len, L, R, tokens}. */
int fb_pack_wavefronts(fb_ctx* ctx, const fb_state* st, const fb_pack* out,
                       void* ws, int32_t* status, void* stream);

/* Sec. 3.1 "W-shaped block-causal attention", Sec. 3.2 Eq. 5: for every live
 * slot (r, s), token and query head: softmax(sm_scale * q k^T) v over the
 * keys {frozen prefix [0, o_r) of request r, read through its page table}
 * u {window blocks 0..s of request r, all bl tokens each}.
 *   q, out        [max_slots*bl, n_q_heads, head_dim]  bf16
 *   k_win, v_win  [max_slots*bl, n_kv_heads, head_dim] bf16  (this step's
 *                 fresh K/V of the window, slot order)
 *   k_pool,v_pool [num_pages, n_kv_heads, 64, head_dim] bf16
 *   page_table    [R_max, max_pages_per_req] int32
 * bf16 inputs, fp32 accumulation, bf16 output.  Rows of padding slots are
 * not written.  `pk` and `ws` must come from fb_pack_wavefronts of this
 * step.  In a context with window_in_pages = 1 the window blocks are read
 * from the pages too (positions [o_r, o_r + (s+1) bl), written there by
 * fb_scatter_window_kv); k_win and v_win must then be NULL. */
int fb_wavefront_attn(fb_ctx* ctx, const fb_pack* pk, const void* q,
                      const void* k_win, const void* v_win,
                      const void* k_pool, const void* v_pool,
                      const int32_t* page_table, void* out, void* ws,
                      int32_t* status, void* stream);

/* Sec. 3.2 Eq. 6 as data movement (contexts with window_in_pages = 1): the
 * fresh K/V of every live window position go to the request's pages at their
 * absolute positions, cache[r, o_r + s*bl + t] = k_new[slot, t], for all KV
 * heads; the frozen prefix [0, o_r) and positions right of the window are
 * not touched.  Retirement then freezes what is already in place.
 *   k_new, v_new  [max_slots*bl, n_kv_heads, head_dim] bf16, slot order
 *   rope_base     0: keys are stored as given.  > 0: each key is first
 *                 rotated by its absolute position (pairs (x_i, x_{i+d/2})
 *                 turned by pos * rope_base^(-2i/d); the paper only says the
 *                 window carries absolute position ids for RoPE, the pairing
 *                 and the base are the model's), fp32 arithmetic with the
 *                 angle formed in fp64, result rounded to bf16
 * `pk` must come from fb_pack_wavefronts of this step; rows of padding slots
 * are not read.  A page id outside the pool sets FB_ST_BAD_PAGE and that row
 * is skipped. */
int fb_scatter_window_kv(fb_ctx* ctx, const fb_pack* pk,
                         const int32_t* page_table, const void* k_new,
                         const void* v_new, void* k_pool, void* v_pool,
                         float rope_base, int32_t* status, void* stream);

/* The cache of Sec. 3.2 "KV Retrieval and Write-back" (Eq. 6) held in 8 bits.
 * The paper states no numeric precision (Sec. 4.1); this is the reading taken:
 * a page stores K and V as OCP FP8 E4M3 bytes (largest finite value 448, no
 * infinities) and the caller supplies one fp32 scale per KV head for K and one
 * for V (calibration is the model's business): stored byte = e4m3(x / scale),
 * value read back = byte * scale.  x / scale is the correctly rounded fp32
 * quotient, rounded to nearest even onto the E4M3 grid, saturating at +-448.
 * One scale per head rather than per page: a page is filled by several commits
 * and frozen positions are never rewritten.  Contexts need window_in_pages = 1
 * (the scatter is the quantiser, so every key the attention reads is a paged
 * 8-bit one), head_dim = 128 and kv_fp8 = 1 in the configuration;
 * FB_ERR_UNSUPPORTED otherwise (and fb_wavefront_attn / fb_scatter_window_kv
 * refuse a kv_fp8 context).
 *   k_pool8, v_pool8  [num_pages, n_kv_heads, 64, head_dim] uint8 (E4M3)
 *   k_scale, v_scale  [n_kv_heads] fp32, positive, DEVICE pointers
 *
 * fb_scatter_window_kv_fp8: fb_scatter_window_kv into such pages (the rotary
 * embedding, if asked for, is applied in fp32 before the division).
 *
 * fb_wavefront_attn_fp8: fb_wavefront_attn over such pages.  Both products run
 * on the tensor cores in 8 bits: the queries are rounded to E4M3 after an exact
 * per-row power-of-two scaling, and the softmax weights are rounded to E4M3
 * (three mantissa bits) before they multiply V; accumulation is fp32, the
 * row sums are taken from the unrounded weights.  Against exact arithmetic on
 * the values the pages hold this costs a few percent of relative error per
 * output row (the parity tests state and derive the bound); it is the price of
 * the 8-bit tensor-core rate.  fb_gate_commit works unchanged (with the window
 * in the pages it copies nothing); fb_step_host does not drive these calls. */
int fb_scatter_window_kv_fp8(fb_ctx* ctx, const fb_pack* pk,
                             const int32_t* page_table, const void* k_new,
                             const void* v_new, void* k_pool8, void* v_pool8,
                             const float* k_scale, const float* v_scale,
                             float rope_base, int32_t* status, void* stream);
int fb_wavefront_attn_fp8(fb_ctx* ctx, const fb_pack* pk, const void* q,
                          const void* k_pool8, const void* v_pool8,
                          const float* k_scale, const float* v_scale,
                          const int32_t* page_table, void* out, void* ws,
                          int32_t* status, void* stream);

/* Sec. 3.2 Eq. 4 feeding the model: input embeddings of the packed window,
 * x[i, :] = table[qtok[i], :] for the rows of live slots (rows of padding
 * slots are not written).
 *   table  [table_rows, hidden] bf16 (hidden a multiple of 8; table_rows must
 *          exceed every token id in use, mask_id included)
 *   x      [max_slots*bl, hidden] bf16
 * A token id outside [0, table_rows) sets FB_ST_BAD_TOKEN and leaves its row
 * unwritten. */
int fb_embed_gather(fb_ctx* ctx, const fb_pack* pk, const void* table,
                    int32_t table_rows, int32_t hidden, void* x,
                    int32_t* status, void* stream);

/* The paper has no counterpart to this call: it exists for callers that
 * cannot allocate device memory (an engine that has given the whole device
 * to its own pool, a plugin in a pre-partitioned process, a loop that must
 * not take cudaMalloc's implicit synchronisation) and therefore cannot
 * provide the workspace fb_wavefront_attn needs.  Same computation and same
 * tensors as fb_pack_wavefronts followed by fb_wavefront_attn, but the
 * scratch (the attention work list) lives in an 8 MiB __device__ array inside
 * the library image; no cudaMalloc / cudaFree / allocating library routine is
 * called.  The work list is rebuilt from `st` (the arrays of `pk` are
 * rewritten with the same values fb_pack_wavefronts gives) and never splits
 * the key axis, so results may differ from fb_wavefront_attn in the last
 * rounding only.
 *   - FB_ERR_UNSUPPORTED for contexts with window_in_pages = 1.
 *   - FB_ERR_WORKSPACE when the configuration's work list does not fit in
 *     8 MiB (about 100,000 (request, KV head, Q-tile pair) units).
 *   - FB_ERR_INVALID_ARG when a member of `st` or `pk` or a tensor is NULL.
 *   - The first call on each device looks up the array's device address and
 *     sets kernel attributes; make that call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous
 *     call's contents (every call overwrites all it reads, nothing needs
 *     clearing): two calls that overlap on the GPU, e.g. on two streams, race.
 *   - Every GPU that loads the library holds the 8 MiB until the process
 *     exits. */
int fb_wavefront_attn_static(fb_ctx* ctx, const fb_state* st,
                             const fb_pack* pk, const void* q,
                             const void* k_win, const void* v_win,
                             const void* k_pool, const void* v_pool, void* out,
                             int32_t* status, void* stream);

/* Sec. 2.1 Eq. 1 and the numerator / denominator of Eq. 2.
 *   logits     [max_slots*bl, vocab] bf16, slot order
 *   argmax     [max_slots*bl] int32  top-1 token (lowest index on ties)
 *   conf       [max_slots*bl] fp32   its softmax probability
 *   action     [max_slots*bl] uint8  FB_ACT_*
 *   slot_stats [max_slots, 6] int32  m0, rdy, n_m2t, n_t2t, m1, has_eos
 * st->tokens is updated in place (x <- x_hat on Gamma u Delta).  Rows of
 * padding slots get argmax -1, conf 0, action 0, stats 0. */
int fb_t2t_step(fb_ctx* ctx, const fb_pack* pk, const void* logits,
                const fb_state* st, int32_t* argmax, float* conf,
                uint8_t* action, int32_t* slot_stats, int32_t* status,
                void* stream);

/* fb_t2t_step with the LM head in front of it (Sec. 3.1: the readiness
 * statistics come "from the current-step logits"): the logits z = x W^T are
 * formed on the tensor cores (bf16 inputs, fp32 accumulation, no rounding to
 * a storage type) and reduced to top-1 token and confidence tile by tile, so
 * the [rows, vocab] logits are never written or read back; then Eq. 1 and the
 * block counts exactly as in fb_t2t_step.
 *   x       [max_slots*bl, hidden] bf16 hidden states, slot order
 *   w       [vocab, hidden] bf16 head weights
 *   hidden  multiple of 64
 *   ws      fb_lm_head_workspace_bytes(ctx) bytes of device scratch, 16-byte
 *           aligned (per row and 256-token slice of the vocabulary: max, sum
 *           of exponentials, first index of the max)
 * Outputs and state update as in fb_t2t_step. */
size_t fb_lm_head_workspace_bytes(const fb_ctx* ctx);
int fb_lm_head_t2t(fb_ctx* ctx, const fb_pack* pk, const void* x,
                   const void* w, int32_t hidden, const fb_state* st,
                   int32_t* argmax, float* conf, uint8_t* action,
                   int32_t* slot_stats, void* ws, int32_t* status,
                   void* stream);

/* Alg. 1 lines 7-12, Eq. 2-3, Eq. 6 for the committing block: per decoding
 * request retire the maximal locally-finished prefix of its window in order
 * (stopping after a block that holds EOS), copy those blocks' window K/V to
 * absolute positions [o_r, o_r + c*bl) of the request's pages, advance L and
 * prefix_len, mark the request done on a committed EOS or L == n, then admit
 * at most one new all-[M] block when rho(frontier) >= theta_spawn and
 * R - L < W and R < n.
 *   n_committed   [R_max] int32 blocks retired this step
 *   spawned       [R_max] uint8
 *   step_counters [FB_STEP_COUNTERS] int32 (FB_CT_*), overwritten
 * Mutates st->{active, prefix_len, L, R, tokens (new block), pe_done} and the
 * pool pages of committed blocks; frozen positions are never rewritten.
 * With window_in_pages = 1 nothing is copied (k_win, v_win, k_pool, v_pool
 * may be NULL): advancing prefix_len freezes what the scatter put in place.
 * With batch_sync = 1 the same per-block predicates feed two reductions over
 * the decoding sequences first: a sequence retires min(its own finished
 * prefix, the batch's), where a sequence that terminates (committed EOS, or
 * L == n) stops counting once its last block is out; then all remaining
 * sequences admit one block, or none does.  One extra single-CTA launch. */
int fb_gate_commit(fb_ctx* ctx, const fb_pack* pk, const int32_t* slot_stats,
                   const fb_state* st, const void* k_win, const void* v_win,
                   void* k_pool, void* v_pool, int32_t* n_committed,
                   uint8_t* spawned, int32_t* step_counters, int32_t* status,
                   void* stream);

/* One whole step (the four calls above in order) on HOST inputs: copies this
 * step's q / k_win / v_win / logits from host (pinned) memory into the
 * caller's device staging buffers, runs the step, and copies n_committed,
 * spawned and step_counters back to host memory.  All asynchronous on
 * `stream`.  h_* are host pointers; everything else is as above.  A harness
 * convenience with no counterpart in the paper (its engine keeps Q/K/V and
 * logits on the device); it is what an end-to-end timing with host buffers
 * calls. */
typedef struct {
  const void* h_q;
  const void* h_k_win;
  const void* h_v_win;
  const void* h_logits;
  int32_t* h_n_committed;    /* [R_max]  */
  uint8_t* h_spawned;        /* [R_max]  */
  int32_t* h_step_counters;  /* [FB_STEP_COUNTERS] */
  int32_t* h_status;         /* [1]      */
  int64_t n_rows;            /* leading rows of q / k_win / v_win / logits
                                the caller has filled (live slots * bl);
                                0 or out of range: all max_slots*bl rows    */
} fb_host_io;

typedef struct {
  void* q; void* k_win; void* v_win; void* out; void* logits;
  void* k_pool; void* v_pool;
  int32_t* argmax; float* conf; uint8_t* action; int32_t* slot_stats;
  int32_t* n_committed; uint8_t* spawned; int32_t* step_counters;
  int32_t* status; void* ws;
} fb_device_bufs;

int fb_step_host(fb_ctx* ctx, const fb_state* st, const fb_pack* pk,
                 const fb_device_bufs* dev, const fb_host_io* io,
                 void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FLOWBLOCK_H */
