/*
 * dsa.h -- C ABI of the diagonal-aware sparse decode-attention library for NVIDIA B200 (sm_100a).
 *
 * One call = one decode step of one transformer layer: every request of a batch has ONE query
 * token per head and attends over its KV cache.  The sparse call keeps the whole prompt and,
 * inside a recent window of the decode (image) tokens, drops the keys that lie on the skipped
 * diagonals -- keys at fixed distances behind the query -- so that dropped keys are never read
 * from memory.  (Paper: "Understanding and Exploiting Diagonal Attention Sparsity in
 * Autoregressive Image Generation", Section 4 and Algorithm 1.)
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; it must stay valid until the
 *     work queued on `stream` has finished.  The dsa_problem / dsa_diag_params structs themselves
 *     are HOST memory, read during the call only.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default stream);
 *     the library never synchronises and allocates no device memory.  It reads no environment
 *     variable and carries no result from one call to the next (the one piece of device state that
 *     outlives a call is a diagnostic counter, see dsa_wait_timeouts()); what it does remember per
 *     device are idempotent set-up caches (which kernel variants have been configured, the SM
 *     count, the addresses of the built-in scratch array and of that counter, the driver entry
 *     point that encodes tensor maps), written with atomics, so calls may come from several host
 *     threads.  Scratch comes from the caller's `workspace` (device, 256-byte aligned), sized
 *     by dsa_workspace_size(); it may be reused by the next call on the same stream.  The one
 *     exception is dsa_decode_attention_static_scratch(), whose scratch is a fixed array inside
 *     the library image.
 *   - Arguments are checked on the host before anything is launched.  Values that live in
 *     device memory (seq_len, prompt_len, block ids, skip offsets) cannot be checked there;
 *     kernels clamp them into range instead, so bad values give wrong numbers, not faults.
 *   - Return value: DSA_OK or a negative dsa_status.  After DSA_ERR_CUDA the CUDA error code is
 *     available from dsa_last_cuda_error().
 *   - The first launch of each kernel variant on a device also configures it (one-time
 *     attribute and address queries that must not happen inside a stream capture): call
 *     dsa_prepare() once per device, or make the first call of a given shape, before capturing.
 *   - There is no CPU path: without a CUDA device every compute call fails with DSA_ERR_CUDA.
 *
 * Positions.  For request b, prompt_len[b] = L_p tokens of prompt come first in the cache and
 * are always attended.  p = seq_len[b] - prompt_len[b] decode tokens follow, the last of which
 * is the token being decoded (its K/V are already in the cache); Algorithm 1's 0-based step is
 * t = p - 1.  A key at cache position s >= L_p lies o = seq_len - 1 - s tokens behind the query.
 */
#ifndef DSA_H
#define DSA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DSA_VERSION 101  /* 101: dsa_problem.plan_flags promise bit, dsa_diag_params.skip_bitmap, dsa_plan_info grew */

/* exported symbols (the library is built with hidden visibility for everything else) */
#if defined(__GNUC__)
#define DSA_API __attribute__((visibility("default")))
#else
#define DSA_API
#endif

typedef enum dsa_status {
    DSA_OK = 0,
    DSA_ERR_INVALID_ARG = -1,         /* null pointer, bad size, bad stride, N_att > window ...   */
    DSA_ERR_UNSUPPORTED = -2,         /* head_dim not 64/128, group size not 1/2/4/8, window too   */
                                      /* large for a LIST mask, ...                                */
    DSA_ERR_WORKSPACE_TOO_SMALL = -3,
    DSA_ERR_CUDA = -4                 /* a CUDA runtime call failed; see dsa_last_cuda_error()     */
} dsa_status;

typedef enum dsa_dtype { DSA_BF16 = 0, DSA_F32 = 1 } dsa_dtype;

typedef enum dsa_mask_mode {
    DSA_MASK_WINDOW = 0,  /* prompt + the `window` most recent decode tokens, nothing skipped      */
    DSA_MASK_GRID = 1,    /* skipped diagonals derived from the raster grid (see dsa_diag_params)  */
    DSA_MASK_LIST = 2     /* skipped diagonals given per head as a list of distances               */
} dsa_mask_mode;

/*
 * The attention problem (inputs of Algorithm 1: the prompt KV cache K_p,V_p and the decode KV
 * cache K,V, stored back to back per request, plus the query of the current step).
 */
typedef struct dsa_problem {
    int32_t batch;             /* B, number of requests (>= 0)                                     */
    int32_t num_q_heads;       /* H_q                                                              */
    int32_t num_kv_heads;      /* H_kv; H_q / H_kv must be 1, 2, 4 or 8.  Query head h reads kv    */
                               /* head h / (H_q / H_kv)                                            */
    int32_t head_dim;          /* D: 64 or 128                                                     */
    int32_t dtype;             /* dsa_dtype of q, k_cache, v_cache and out                         */
    float sm_scale;            /* logit scale; 0 means 1/sqrt(D)                                   */
    const void *q;             /* [B, H_q, D] contiguous                                           */
    const void *k_cache;       /* keys;   rows of D contiguous elements, 16-byte aligned           */
    const void *v_cache;       /* values; same layout and strides as k_cache                       */
    /* Element strides.  Contiguous cache (block_table == NULL): token s of request b, kv head g
     * starts at b*stride_batch + s*stride_token + g*stride_head (stride_batch may be 0 to let all
     * requests read one cache).  Paged cache: token s lives in block
     * id = block_table[b*max_blocks + s/block_size] at
     * id*stride_batch + (s % block_size)*stride_token + g*stride_head.
     * All strides must be multiples of 16 bytes. */
    int64_t stride_batch;
    int64_t stride_token;
    int64_t stride_head;
    const int32_t *seq_len;    /* [B] tokens in the cache, prompt included                         */
    const int32_t *prompt_len; /* [B] L_p; values above seq_len[b] are read as seq_len[b]          */
    const int32_t *block_table;/* [B, max_blocks] or NULL                                          */
    int32_t max_blocks;        /* row length of block_table                                        */
    int32_t block_size;        /* tokens per block (> 0 when paged)                                */
    int32_t num_blocks;        /* blocks in the pool; block ids are clamped to [0, num_blocks)     */
    int32_t max_seq_len;       /* HOST upper bound of seq_len[b]; sizes the launch.  Longer        */
                               /* sequences are read as if they ended there                        */
    int32_t max_prompt_len;    /* HOST upper bound of prompt_len[b], or 0 if unknown (the sparse   */
                               /* call then plans for max_seq_len kept tokens)                     */
    int32_t split_tokens;      /* kept tokens handled by one thread block; 0 = library chooses.    */
                               /* Rounded up to the tile size, at most 1024                        */
    /* Bounded cache (the eviction step of Algorithm 1, phase 3; footprint N_r + L_p of Section 4's
     * cost analysis).  ring_size == 0: every token is stored at its logical position.
     * ring_size > 0: the prompt and the first ring_sinks decode tokens are stored at their logical
     * positions; decode token j >= ring_sinks is stored at position
     * L_p + ring_sinks + (j - ring_sinks) mod ring_size, overwriting the token that left the
     * window ring_size steps earlier.  seq_len stays the LOGICAL length.  Needs
     * max_prompt_len > 0; sparse calls need window <= ring_size and n_sink <= ring_sinks; the
     * dense call is refused.  The cache then needs max_prompt_len + ring_sinks + ring_size
     * tokens per request instead of max_seq_len; a device prompt_len[b] above max_prompt_len is
     * read as max_prompt_len, so that no row is addressed outside that region. */
    int32_t ring_size;
    int32_t ring_sinks;
    /* 0 in production: the library chooses the launch plan.  Comparison runs and tests may force
     * single planner decisions with the DSA_PLAN_* bits below; results never depend on them
     * beyond summation order. */
    uint32_t plan_flags;
} dsa_problem;

#define DSA_PLAN_CUDA_CORES    0x01u  /* bf16 through the CUDA-core kernel instead of the tensor-core one */
#define DSA_PLAN_NO_ITEM_WARPS 0x02u  /* small launches: split + combine, never four warps on one item   */
#define DSA_PLAN_RING_DEEP     0x04u  /* two-heads-per-block kernel: keep the 3-stage ring               */
#define DSA_PLAN_RING_SHALLOW  0x08u  /* two-heads-per-block kernel: take the 2-stage ring               */
#define DSA_PLAN_GROUP         0x10u  /* take the head-group / per-head-list kernels wherever they can run */
#define DSA_PLAN_NO_GROUP      0x20u  /* never take them                                                 */
#define DSA_PLAN_GROUP_W4      0x40u  /* forced head-group kernel: 4 warps per block instead of 2        */
#define DSA_PLAN_NO_CLUSTER    0x80u  /* small launches: never let a thread-block cluster share a work item */
#define DSA_PLAN_CLUSTER2      0x10000u /* small launches (several warps per item): clusters of 2 blocks  */
#define DSA_PLAN_CLUSTER4      0x20000u /*                                           clusters of 4 blocks  */
#define DSA_PLAN_GATHER        0x40000u /* head-group kernel, 4 warps: stage tiles by tensor-map gather copies */
                                        /* (TMA, four scattered rows per copy) where the cache has a 2-D view */
#define DSA_PLAN_NO_GATHER     0x80000u /* never do                                                        */
#define DSA_PLAN_PRODUCERS     0x100000u /* head-group kernel, 4 warps: a producer warp beside every consumer warp */
#define DSA_PLAN_NO_PRODUCERS  0x200000u /* never                                                       */
/* Not a planner switch but a promise about the stream: no launch that can still be running when this
 * call's kernel starts writes seq_len, prompt_len, block_table or the skip lists (skip_offsets and
 * skip_bitmap; a call with `select` writes both, for its own layer).  The attention kernels
 * chain with programmatic dependent launch and let their successor start before they have waited for
 * their own predecessor, so "still running" means: the launch just before this call and, if that is an
 * attention call of this library, the launches before it in turn, back to the first launch that does
 * not let its successor in early (a projection, dsa_advance_seq_len: those complete before anything
 * behind them starts).  dsa_append_kv does let its successor in early and, when it advances, writes
 * seq_len: the call behind it cannot make the promise.  In a decode loop of fused steps every layer's
 * call but the one that follows dsa_advance_seq_len can.
 * The head-group, per-head-list, several-warps-per-item and cluster kernels then work out which rows to
 * read BEFORE they wait for the launch in front, and touch q, the new rows and the caches only after;
 * the other kernels (producer-warp and tensor-map forms, one warp per item, CUDA cores) ignore it. */
#define DSA_PLAN_METADATA_STABLE 0x800000u
#define DSA_PLAN_HEADS_PER_WARP_SHIFT 8  /* forced head-group kernel: kv heads per warp in bits 8..15    */
#define DSA_PLAN_HEADS_PER_WARP_MASK  0xff00u

/*
 * Which decode keys are kept (Algorithm 1 with its data-dependent selection made an input).
 *
 * With t = p - 1, the window holds the distances o = 0 .. min(t, window - 1) (the `window` = N_r
 * most recent decode tokens, the current one included).  m = window - n_att diagonals are
 * skipped in steady state.  Algorithm 1 selects them one per step from step n_att - 1 on, and an
 * entry selected at step s is skipped from step s + 1 on; so at step t the first
 * n_act = clamp(t - (n_att - 1), 0, m) selected distances are skipped.  A key chosen at step s
 * with cache index j keeps the distance s - j at every later step (the "+1" shift of skip_idx).
 *
 *   LIST  skip_offsets[b][mask_head][k] is the distance of the k-th selection, in selection
 *         order; it must be a valid trace: 0 <= o_k <= n_att - 1 + k (0-based k), no repeats.
 *         mask_heads is 1 (all heads share), H_kv (per kv head) or H_q (per query head, the
 *         paper's setting; with grouped queries a KV row is read if any head of its group keeps
 *         it, the other heads ignore it).
 *   GRID  the trace is generated from the grid instead of being passed: with
 *         stride = grid_w + row_extra tokens per image row, the column distance of o is
 *         d(o) = min(o mod stride, stride - o mod stride) and every selection step skips the
 *         attended key with the largest (d(o), o).  Same mask for all heads.  (Not in the
 *         paper: a data-free stand-in for its argmin that keeps the diagonals next to the
 *         multiples of the row stride.)
 *   WINDOW nothing skipped (n_att is ignored).  This is the paper's SlidingWindow baseline.
 *
 * Selection (the choice of the next skipped key in Algorithm 1, phase 2, fused into the attention
 * pass as in Section 5.1).  With `select` set, a request whose step t lies in N_att-1 .. N_r-2 also gets
 * the next trace entry: among the decode keys it attends (sinks excluded) the one with the lowest
 * softmax weight -- the lowest logit; equal logits go to the lowest cache index -- is found per
 * query head and its distance is written to skip_offsets[b][h][t - (N_att-1)], which takes effect
 * from the next step on.  Calling the sparse call once per decode step with the same buffer thus
 * grows the trace exactly as Algorithm 1 grows skip_idx.  Entries are decided on float32 logits;
 * -1 is written if there is no candidate.  Requests outside those steps are left untouched.
 *
 * Sinks (Section 5.1, the "Diagonal + sink4" variant and the StreamingLLM baseline): the first
 * n_sink decode tokens are kept at every step in addition to what the mode keeps, and are never
 * counted against n_att: in steady state n_att + n_sink decode keys are attended.  WINDOW with
 * n_sink = 4 is StreamingLLM (4 sinks + recent window); GRID or LIST with n_sink = 4 is
 * Diagonal + sink4 with n_att = budget - 4.
 */
typedef struct dsa_diag_params {
    int32_t mode;                 /* dsa_mask_mode                                                 */
    int32_t window;               /* N_r >= 1                                                      */
    int32_t n_att;                /* N_att, 1 <= n_att <= window                                   */
    int32_t grid_w;               /* GRID: image tokens per row                                    */
    int32_t row_extra;            /* GRID: row-end / separator tokens per row (>= 0)               */
    int32_t *skip_offsets;        /* LIST: device [B, mask_heads, trace_len] int32 (written when   */
                                  /* `select` is set, otherwise only read)                         */
    int32_t mask_heads;           /* LIST: 1, H_kv or H_q                                          */
    int32_t trace_len;            /* LIST: entries per trace, >= window - n_att                    */
    int32_t n_sink;               /* first decode tokens always kept (>= 0; 0 = none)              */
    int32_t select;               /* LIST, mask_heads == H_q: also run the phase-2 selection       */
    uint32_t *skip_bitmap;        /* LIST, optional (NULL: none): device [B, mask_heads, ceil(window / 32)]  */
                                  /* words; bit o of a head's row is set iff distance o is one of its        */
                                  /* ACTIVE skip_offsets entries (the first n_act).  The same information    */
                                  /* as the list, in the form the per-head-list kernel wants: it then reads  */
                                  /* window / 8 bytes per head instead of scattering the list into a bitmap  */
                                  /* itself.  dsa_build_skip_bitmap() fills it from skip_offsets; calls with */
                                  /* `select` keep it up to date (they set the bit of every entry they       */
                                  /* write).  The caller clears it together with the list when a request     */
                                  /* starts over.  Kernels other than the per-head-list one read the list.   */
} dsa_diag_params;

/* What a call will launch (filled by dsa_query_plan; for reporting and for tests). */
typedef struct dsa_plan_info {
    int32_t split_tokens;   /* kept tokens per work item                                           */
    int32_t n_split;        /* splits per (request, kv head); 1 = results written directly         */
    int32_t launches;       /* kernels launched by the call (1, or 2 with the combine)             */
    int32_t grid_blocks;    /* thread blocks of the attention kernel                               */
    int32_t smem_bytes;     /* dynamic shared memory per block                                     */
    int32_t tile_tokens;    /* tokens per staged K/V tile                                          */
    int32_t stages;         /* tiles in flight per block (per warp for the tensor-core kernel)     */
    int32_t tensor_cores;   /* 1: tensor-core kernel (bf16), one warp per work item;               */
                            /* 0: CUDA-core kernel (fp32), one 128-thread block per work item      */
    int32_t work_items;     /* (request, kv head, split) items                                     */
    int32_t item_warps;     /* warps that share one work item (4 in small tensor-core launches,    */
                            /* merged in shared memory; else 1)                                    */
    int32_t heads_per_block;/* head-group tensor-core kernel: kv heads that share the one row list */
                            /* a block builds (its warps stream heads_per_block / block_warps      */
                            /* heads each, back to back); 0: another kernel                        */
    int32_t block_warps;    /* warps per thread block that compute (producer_warps come on top)     */
    int32_t per_head_lists; /* 1: the per-head-list tensor-core kernel (list masks per head, fused  */
                            /* selection): shared tables per block, one candidate list per head    */
    int32_t cluster_blocks; /* blocks of a thread-block cluster that share one work item and merge */
                            /* through distributed shared memory (small launches); 1: no cluster   */
    int32_t tensor_map_copies; /* 1: the head-group kernel stages its tiles with tensor-map gather  */
                            /* copies (TMA) completing on mbarriers; 0: 16-byte cp.async copies    */
    int32_t producer_warps; /* warps per block that only issue copies (one per consumer warp, handing */
                            /* tiles over through mbarriers); 0: every warp copies and computes       */
} dsa_plan_info;

DSA_API int32_t dsa_version(void);
DSA_API const char *dsa_status_string(int32_t status);
/* CUDA error code recorded by the last failing call of this thread (0 if none). */
DSA_API int32_t dsa_last_cuda_error(void);
/* Number of bounded waits that gave up on the current device since the library was loaded.  The
 * tensor-map kernel waits for each tile on an mbarrier for about a second at most; a copy that
 * never lands makes it count here, stop waiting and run to its end, so that the context stays
 * usable (the numbers of that call are then wrong).  0 in a healthy run.  count_out: host pointer.
 * Synchronises with the device (a copy from a device symbol): not for use inside a capture. */
DSA_API int32_t dsa_wait_timeouts(int32_t *count_out);
/* Measuring hook: the sparse / dense call (diag NULL: dense) with the arithmetic taken out.  The launch
 * has the plan's grid, builds the same row lists and stages the same K / V tiles through the same
 * shared-memory rings, but a landed tile is only read once; what it leaves in out / lse (and the
 * workspace) is meaningless.  Its time is what the staging alone costs for this very problem -- the
 * attention call's own speed of light.  DSA_ERR_UNSUPPORTED unless the plan is the four-warp head-group
 * kernel (dsa_plan_info.block_warps == 4, per_head_lists == 0).  Arguments as dsa_decode_attention_sparse. */
DSA_API int32_t dsa_debug_copy_only(const dsa_problem *problem, const dsa_diag_params *diag, void *out, float *lse,
                                    void *workspace, size_t workspace_bytes, void *stream);
/* Fills diag->skip_bitmap from diag->skip_offsets for the requests' current seq_len: row (b, mask head)
 * gets the bits of that head's first n_act entries that lie in [0, window), all other bits are cleared.
 * LIST mode only; both pointers required.  Asynchronous on `stream`. */
DSA_API int32_t dsa_build_skip_bitmap(const dsa_problem *problem, const dsa_diag_params *diag, void *stream);
/* Test hook for that mechanism: launches one warp on `stream` that waits, with the same bound, on an
 * mbarrier nothing ever arrives on.  The wait runs out after about a second, the counter above goes
 * up by one, the kernel ends and the context stays usable.  Asynchronous like every launch. */
DSA_API int32_t dsa_debug_wait_giveup(void *stream);

/*
 * Configure every kernel variant of the library for the CURRENT device (a few hundred one-time
 * attribute calls, the SM count and the address of the built-in scratch array of
 * dsa_decode_attention_static_scratch; no launch, no allocation).  Optional: calls do it lazily
 * for what they need; required only before a stream capture whose calls would otherwise be the
 * first of their shape on this device.
 */
DSA_API int32_t dsa_prepare(void);

/* Bytes of workspace the attention calls need for `problem` (diag == NULL: dense call). */
DSA_API int32_t dsa_workspace_size(const dsa_problem *problem, const dsa_diag_params *diag, size_t *bytes);

/* The launch plan the attention calls will use for `problem` (diag == NULL: dense call). */
DSA_API int32_t dsa_query_plan(const dsa_problem *problem, const dsa_diag_params *diag, dsa_plan_info *info);

/*
 * Dense decode attention (the paper's baseline; Algorithm 1's Attn over every cached token):
 *   s_j = sm_scale * q_h . k_j  for j in [0, seq_len),  lse = ln sum_j e^{s_j},
 *   out = sum_j e^{s_j - lse} v_j.
 * out [B, H_q, D] in problem->dtype; lse [B, H_q] float32, natural log.  A request with
 * seq_len <= 0 gets out = 0, lse = -inf.
 */
DSA_API int32_t dsa_decode_attention_dense(const dsa_problem *problem, void *out, float *lse,
                                   void *workspace, size_t workspace_bytes, void *stream);

/*
 * Diagonal-aware sparse decode attention (Algorithm 1, one step t for every request):
 *   Attn(Q_t, K_p + K[idx], V_p + V[idx]) with idx = window - skip_idx,
 * softmax taken jointly over the prompt keys and the kept decode keys.  Only kept rows are read.
 * Outputs as for the dense call.
 */
DSA_API int32_t dsa_decode_attention_sparse(const dsa_problem *problem, const dsa_diag_params *diag,
                                    void *out, float *lse,
                                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * One decode step's attention with the step's inputs and results in HOST memory (the call a
 * serving loop makes when the scheduler lives on the CPU; the KV cache, which is decode state,
 * stays on the device).  Not in the paper; it is the dense (diag == NULL) or sparse call above
 * wrapped in the copies a step needs, all queued on `stream`:
 *   host_q -> problem->q, host_seq_len -> problem->seq_len, host_prompt_len -> problem->prompt_len,
 *   host_block_table -> problem->block_table (paged caches only; NULL otherwise),
 *   attention into dev_out / dev_lse, then dev_out -> host_out, dev_lse -> host_lse.
 * The device pointers inside `problem` are therefore WRITTEN by this call.  Host buffers should
 * be pinned for the copies to be asynchronous; they must stay valid, and host_out / host_lse
 * must not be read, until the stream has been synchronised by the caller.
 */
DSA_API int32_t dsa_decode_attention_host_io(const dsa_problem *problem, const dsa_diag_params *diag,
                                             const void *host_q, const int32_t *host_seq_len,
                                             const int32_t *host_prompt_len, const int32_t *host_block_table,
                                             void *dev_out, float *dev_lse, void *host_out, float *host_lse,
                                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same step as dsa_decode_attention_host_io, with the large transfers folded into the
 * kernels (not in the paper): the attention kernels read q from, and write out / lse to, the
 * caller's PINNED host buffers directly over the bus (mapped, zero-copy), so no separate q upload
 * precedes the attention and no download follows it.  What every head of a request re-reads
 * (host_seq_len, host_prompt_len, host_block_table) is still copied into the device arrays named
 * in `problem`, which are therefore WRITTEN.  problem->q is scratch: when the plan splits the
 * keys of one (request, kv head) over several work items, q is first copied there so that it
 * crosses the bus once; otherwise it is left untouched.
 * host_q, host_out and host_lse must be page-locked host memory that the device can address
 * (cudaHostAlloc / cudaHostRegister; checked with cudaPointerGetAttributes before anything is
 * queued: DSA_ERR_INVALID_ARG otherwise), host_q and host_out 16-byte aligned.  They must stay valid, and
 * host_out / host_lse must not be read, until the caller has synchronised the stream.
 */
DSA_API int32_t dsa_decode_attention_host_mapped(const dsa_problem *problem, const dsa_diag_params *diag,
                                                 const void *host_q, const int32_t *host_seq_len,
                                                 const int32_t *host_prompt_len, const int32_t *host_block_table,
                                                 void *host_out, float *host_lse,
                                                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * Merge split-KV partial results (not in the paper; the exact identity that a softmax over a
 * union of key sets is the lse-weighted mix of the softmaxes over the parts):
 *   lse = ln sum_i e^{lse_i},  out = sum_i e^{lse_i - lse} out_i.
 * out_part [B, H_q, n_split, D] float32, lse_part [B, H_q, n_split] float32 (natural log; a
 * part with lse_i = -inf is empty and its out_i is not read).  out [B, H_q, D] in out_dtype,
 * lse [B, H_q] float32 (may be NULL).
 */
DSA_API int32_t dsa_combine_splits(const float *out_part, const float *lse_part,
                           int32_t batch, int32_t num_q_heads, int32_t head_dim, int32_t n_split,
                           void *out, float *lse, int32_t out_dtype, void *stream);

/*
 * Append the K/V rows of the token being decoded (the cache write that precedes attention in a
 * decode step; with a bounded cache this is also Algorithm 1's eviction, since the new token
 * takes the slot of the one that left the window).  k_new, v_new: device [B, H_kv, D] in
 * problem->dtype.  The rows of request b go to logical position seq_len[b] (the value BEFORE
 * the call); a request whose seq_len is already max_seq_len is left alone.  With advance != 0
 * seq_len[b] is then incremented on the device by the same kernel, so that a captured sequence
 * "append, attend" can be replayed step after step without the host touching seq_len.
 */
DSA_API int32_t dsa_append_kv(const dsa_problem *problem, const void *k_new, const void *v_new,
                              int32_t advance, void *stream);

/*
 * One decode step of one layer in a single launch (plus the combine when the plan splits):
 * dsa_append_kv followed by the dense (diag == NULL) or sparse attention call, fused.  Not a
 * method of its own: Algorithm 1's "K.append(K_t)" and "Attn(Q_t, K_p + K[idx], ...)" of one
 * step, issued together.
 *   seq_len[b] counts the tokens ALREADY cached, without the token being decoded, and is not
 *   modified: a model's layers share one seq_len array, which the caller advances once per token
 *   after its last layer (dsa_advance_seq_len).
 *   k_new, v_new: device [B, H_kv, D] in problem->dtype, 16-byte aligned.  The rows of request b
 *   are written to logical position seq_len[b] of the cache and the request attends over
 *   seq_len[b] + 1 tokens, the mask taking p = seq_len[b] + 1 - prompt_len[b].  A request whose
 *   seq_len is already max_seq_len has no room: its token is dropped and it attends over what
 *   is cached, exactly as dsa_append_kv followed by attention would do.
 * For bf16 the attention kernel itself reads the current token's rows from k_new / v_new and
 * stores them to the cache; for float32 the rows are stored by a launch of their own first.
 * Everything else (outputs, workspace, plan, fused selection, bounded caches) as for the
 * attention calls.
 */
DSA_API int32_t dsa_decode_step(const dsa_problem *problem, const dsa_diag_params *diag,
                                const void *k_new, const void *v_new, void *out, float *lse,
                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * seq_len[b] += 1 for every request below `max_seq_len` (device array of `batch` int32), queued on
 * `stream`: the once-per-token counterpart of dsa_decode_step, so that a captured token step
 * (every layer's dsa_decode_step, then this) can be replayed without the host touching seq_len.
 */
DSA_API int32_t dsa_advance_seq_len(int32_t *seq_len, int32_t batch, int32_t max_seq_len, void *stream);

/*
 * The kept cache positions, produced by the same device code that the sparse attention kernel
 * uses to decide which rows to read (Algorithm 1: K_p, then window - skip_idx as positions).
 * Positions are LOGICAL (before any ring mapping).
 * idx_out [B, mask_heads, max_kept] int32, ascending, entries beyond the count untouched;
 * count_out [B, mask_heads] int32 holds the full count even when it exceeds max_kept.
 * mask_heads is diag->mask_heads for LIST and 1 otherwise; diag == NULL reports the dense set.
 */
DSA_API int32_t dsa_debug_kept_indices(const dsa_problem *problem, const dsa_diag_params *diag,
                               int32_t *idx_out, int32_t *count_out, int32_t max_kept,
                               void *stream);

/*
 * The attention calls above for callers that cannot hand over a workspace.  (The paper has no
 * counterpart: this is a packaging variant of the two calls, not another method.)
 *
 * Who needs it: code that must not allocate device memory at the point of the call -- an
 * extension running inside a host application's allocation-free section, a latency-critical
 * serving loop that forbids allocator calls, a process whose device memory was carved up
 * completely at start-up.  The split-KV partial results go to a fixed DSA_STATIC_SCRATCH_MAX-byte
 * array inside the library image instead of a caller workspace; the call itself allocates and
 * frees nothing.  The price: each GPU that loads the library carries those bytes until the
 * process exits, whether or not this entry point is ever used.
 *
 * diag == NULL runs the dense call, otherwise the sparse call; q, caches, out and lse are passed
 * exactly as above and results are identical to dsa_decode_attention_dense / _sparse.
 * Problems whose partials exceed the array are refused with DSA_ERR_WORKSPACE_TOO_SMALL and
 * nothing is launched; dsa_workspace_size() tells the size in advance.
 * The first call on each device (or dsa_prepare() before it) looks up the array's device address,
 * with that device current; let that happen before any stream capture begins.
 * All calls share the one array and it keeps whatever the last call left there; nothing in it
 * needs clearing between calls.  Two calls whose kernels can run at the same time on one GPU
 * (different streams, different host threads) would overwrite each other's partials: keep calls
 * of this entry point ordered on one stream per GPU.
 */
#define DSA_STATIC_SCRATCH_MAX (8u << 20)
DSA_API int32_t dsa_decode_attention_static_scratch(const dsa_problem *problem, const dsa_diag_params *diag,
                                                    void *out, float *lse, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* DSA_H */
