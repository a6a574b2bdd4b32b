// C-ABI entry points of the decode-attention library: argument checks, launch planning and
// kernel dispatch.  Everything here is host code except the kernels it instantiates.
#include "../../include/dsa.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <type_traits>

#include "dsa_aux.cuh"
#include "dsa_launch.cuh"

namespace {

using namespace dsa;

thread_local int g_last_cuda_error = 0;

int32_t cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return DSA_ERR_CUDA;
}

// SM count of the current device, asked for once per device (an idempotent cache: two threads that
// race on the first call store the same value).  Falls back to the B200's 148 if the query fails.
int sm_count() {
    static std::atomic<int> cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return 148;
    }
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n <= 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            return 148;
        }
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

constexpr uint32_t kKnownPlanFlags = DSA_PLAN_CUDA_CORES | DSA_PLAN_NO_ITEM_WARPS | DSA_PLAN_RING_DEEP |
                                     DSA_PLAN_RING_SHALLOW | DSA_PLAN_GROUP | DSA_PLAN_NO_GROUP |
                                     DSA_PLAN_GROUP_W4 | DSA_PLAN_HEADS_PER_WARP_MASK | DSA_PLAN_NO_CLUSTER |
                                     DSA_PLAN_CLUSTER2 | DSA_PLAN_CLUSTER4 | DSA_PLAN_GATHER | DSA_PLAN_NO_GATHER | DSA_PLAN_PRODUCERS |
                                     DSA_PLAN_NO_PRODUCERS | DSA_PLAN_METADATA_STABLE;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int kMaxSplits = 8192;                 // split weights of the combine kernel: 32 KB of shared memory

// The launch plan: how many kept rows one block takes, how many splits that makes.
struct Plan {
    int mode;            // MODE_*
    int window;          // N_r of the sparse call (0: dense)
    int G;
    bool headmask;
    bool select;
    int tile, stages;
    int chunk, n_split;
    int bitmap_words;
    bool mma;            // bf16: one warp per work item, tensor-core tiles
    int mma_warps;       // warps (= kv heads) per block that share one row list
    int mma_kw;          // warps that share one work item (small launches), 1 or kMmaItemWarps
    int mma_cl;          // and blocks of a thread-block cluster that share it (1: no cluster)
    int mma_stages;      // ring depth of the tensor-core kernel
    int group_w;         // head-group tensor-core kernel: warps per block (0: not that kernel)
    int group_u;         // and kv heads each warp streams through the block's one row list
    int group_stages;    // and its ring depth
    bool producers;      // and whether every ring has a producer warp beside its consumer warp
    bool copy_only;      // measuring form of the plain four-warp kernel (dsa_debug_copy_only)
    bool gather;         // and whether its tiles are staged by tensor-map gather copies; the 2-D cache view then:
    int gather_rows_per_stride_b;
    int64_t gather_rows; // its number of token rows
    bool heads;          // per-head-list tensor-core kernel (kHeadsWarps warps per block, group_u heads per warp)
    int dir_cap, kidx_cap;
    int64_t blocks;      // its grid
    int64_t grid;
    size_t smem;
    size_t ws_out_bytes, ws_lse_bytes, ws_sel_bytes, ws_total;
};

// The kernels live in translation units of their own, one per (element type, head_dim): only the
// declarations of kernel_shape / kernel_launch are visible here, their instantiations are linked in.

// Dispatch over (dtype, head_dim): f is called with a value of the element type and head_dim as
// an integral constant.
template <class F>
int32_t dispatch(int dtype, int D, F&& f) {
    if (dtype == DSA_BF16 && D == 64) return f(__nv_bfloat16{}, std::integral_constant<int, 64>{});
    if (dtype == DSA_BF16 && D == 128) return f(__nv_bfloat16{}, std::integral_constant<int, 128>{});
    if (dtype == DSA_F32 && D == 64) return f(float{}, std::integral_constant<int, 64>{});
    if (dtype == DSA_F32 && D == 128) return f(float{}, std::integral_constant<int, 128>{});
    return DSA_ERR_UNSUPPORTED;
}

KernelQuery kernel_query(const Plan& pl) {
    KernelQuery q;
    q.G = pl.G; q.headmask = pl.headmask; q.select = pl.select;
    q.mma = pl.mma; q.mma_warps = pl.mma_warps; q.mma_kw = pl.mma_kw; q.mma_stages = pl.mma_stages;
    q.mma_cl = pl.mma_cl;
    q.group_w = pl.group_w; q.group_stages = pl.group_stages; q.gather = pl.gather; q.producers = pl.producers; q.copy_only = pl.copy_only;
    q.heads = pl.heads; q.dir_cap = pl.dir_cap; q.kidx_cap = pl.kidx_cap; q.window = pl.window;
    return q;
}

// Tokens one request can hold: its logical maximum, or prompt + sinks + ring when bounded.
int64_t physical_capacity(const dsa_problem* p) {
    if (p->ring_size > 0)
        return std::min<int64_t>(p->max_seq_len, (int64_t)p->max_prompt_len + p->ring_sinks + p->ring_size);
    return p->max_seq_len;
}

int32_t check_problem(const dsa_problem* p) {
    if (!p) return DSA_ERR_INVALID_ARG;
    if (p->batch < 0 || p->num_q_heads < 1 || p->num_kv_heads < 1) return DSA_ERR_INVALID_ARG;
    if (p->num_q_heads % p->num_kv_heads) return DSA_ERR_INVALID_ARG;
    if (p->dtype != DSA_BF16 && p->dtype != DSA_F32) return DSA_ERR_UNSUPPORTED;
    if (p->head_dim != 64 && p->head_dim != 128) return DSA_ERR_UNSUPPORTED;
    const int G = p->num_q_heads / p->num_kv_heads;
    if (G != 1 && G != 2 && G != 4 && G != 8) return DSA_ERR_UNSUPPORTED;
    if (p->max_seq_len < 0 || p->max_prompt_len < 0 || p->split_tokens < 0) return DSA_ERR_INVALID_ARG;
    if (p->plan_flags & ~kKnownPlanFlags) return DSA_ERR_INVALID_ARG;
    if (!(p->sm_scale >= 0.f) || !std::isfinite(p->sm_scale)) return DSA_ERR_INVALID_ARG;
    if (p->batch == 0) return DSA_OK;
    if (!p->q || !p->k_cache || !p->v_cache || !p->seq_len || !p->prompt_len) return DSA_ERR_INVALID_ARG;
    if (!aligned16(p->q) || !aligned16(p->k_cache) || !aligned16(p->v_cache)) return DSA_ERR_INVALID_ARG;
    const int64_t vec = p->dtype == DSA_BF16 ? 8 : 4;          // elements per 16 bytes
    if (p->stride_batch < 0 || p->stride_token < p->head_dim || p->stride_head < 0) return DSA_ERR_INVALID_ARG;
    if (p->stride_batch % vec || p->stride_token % vec || p->stride_head % vec) return DSA_ERR_INVALID_ARG;
    if (p->ring_size < 0 || p->ring_sinks < 0) return DSA_ERR_INVALID_ARG;
    if (p->ring_size > 0 && p->max_prompt_len < 1) return DSA_ERR_INVALID_ARG;   // capacity needs the bound
    if (p->block_table) {
        if (p->block_size < 1 || p->max_blocks < 1 || p->num_blocks < 1) return DSA_ERR_INVALID_ARG;
        if ((int64_t)p->max_blocks * p->block_size < physical_capacity(p)) return DSA_ERR_INVALID_ARG;
    }
    return DSA_OK;
}

int32_t check_diag(const dsa_problem* p, const dsa_diag_params* d) {
    if (!d) return DSA_OK;
    if (d->mode != DSA_MASK_WINDOW && d->mode != DSA_MASK_GRID && d->mode != DSA_MASK_LIST)
        return DSA_ERR_INVALID_ARG;
    if (d->window < 1 || d->n_sink < 0) return DSA_ERR_INVALID_ARG;
    // a bounded cache holds the last ring_size decode tokens and the first ring_sinks: nothing else can be kept
    if (p->ring_size > 0 && (d->window > p->ring_size || d->n_sink > p->ring_sinks)) return DSA_ERR_INVALID_ARG;
    if (d->mode == DSA_MASK_WINDOW) return DSA_OK;
    if (d->n_att < 1 || d->n_att > d->window) return DSA_ERR_INVALID_ARG;
    if (d->mode == DSA_MASK_GRID) {
        if (d->grid_w < 1 || d->row_extra < 0) return DSA_ERR_INVALID_ARG;
        if ((int64_t)d->grid_w + d->row_extra > (1 << 30)) return DSA_ERR_INVALID_ARG;
        return DSA_OK;
    }
    if (d->mask_heads != 1 && d->mask_heads != p->num_kv_heads && d->mask_heads != p->num_q_heads)
        return DSA_ERR_INVALID_ARG;
    if (d->trace_len < d->window - d->n_att) return DSA_ERR_INVALID_ARG;
    if (d->window - d->n_att > 0 && p->batch > 0 && !d->skip_offsets) return DSA_ERR_INVALID_ARG;
    if (d->skip_bitmap && (reinterpret_cast<uintptr_t>(d->skip_bitmap) & 3u)) return DSA_ERR_INVALID_ARG;
    if (d->select && d->mask_heads != p->num_q_heads) return DSA_ERR_UNSUPPORTED;   // one selection per attention head
    if (d->select && d->n_sink >= d->n_att) return DSA_ERR_INVALID_ARG;             // no candidate would be left
    return DSA_OK;
}

int round_up(int x, int m) { return (x + m - 1) / m * m; }

// The K / V caches as a matrix [token rows][elements of one token row], which the tensor-map kernel
// gathers rows of.  It exists when tokens are the outer dimension of a page / request (every head of a
// token inside its token stride) and pages / requests start a whole number of token rows apart.
bool gather_view(const dsa_problem* p, int* rows_per_stride_b, int64_t* rows) {
    if (p->dtype != DSA_BF16 || p->head_dim % 64 != 0) return false;
    const int64_t st = p->stride_token;
    if (st <= 0 || (st * 2) % 16 != 0 || p->stride_batch % st != 0) return false;
    if ((int64_t)(p->num_kv_heads - 1) * p->stride_head + p->head_dim > st) return false;
    const int64_t rpb = p->stride_batch / st;
    const int64_t units = p->block_table ? p->num_blocks : p->batch;
    const int64_t last = p->block_table ? p->block_size : physical_capacity(p);
    const int64_t n = (units - 1) * rpb + last;
    if (units < 1 || last < 1 || rpb > 0x7fffffffLL || n < 1 || n >= 0x7fffffffLL) return false;
    if (st > 0xffffffffLL || st * 2 >= (1LL << 40)) return false;      // (limits of a tensor map's extent and pitch)
    *rows_per_stride_b = (int)rpb;
    *rows = n;
    return true;
}

// How many kv heads each warp of the head-group kernel should stream (a power of two), and with which
// ring depth.
//
// Measured on the paged workload (window 512 / N_att 208, 32 kv heads, W = 4, 296 blocks resident) and
// on the decode-loop shape (50 prompt tokens + N_att 52): whatever the batch, the best U is the one
// that makes the grid JUST FIT the device -- 0.86 of a wave at batch 32 / 64 / 128 / 256 with
// U = 1 / 2 / 4 / 8 (37 / 68 / 130 / 256 us against 39 / 72 / 142 / 268 us for two heads per block;
// decode loop at batch 64 / 128 / 256: 22.5 / 40.3 / 75.8 us against 24.9 / 47.9 / 85.2 us).  Every
// block is then resident from the start and every warp streams U heads without a block turning
// over.  A grid of 1.3 waves is the worst case (+25 %), 1.7 and 3.5 waves cost 5-10 %, and under one
// wave the time is that of one block: at half a wave a larger U doubles it.  The estimate below is
// that table: (list building + U heads of `tiles` tiles) x (waves, a partial one counted half-way
// between its size and a whole one) x (time per tile, which grows with the warps that share an SM).
// The shallow ring (one tile in flight per warp instead of two, about 3 % slower when the grid
// fits either way) holds half as many blocks again per SM: it is for grids that would otherwise
// spill a little into a second wave (batch 40: 46 us against 55 us).
// Split plans keep U = 1: most of their (request, split) blocks are empty or short, the real wave
// count is unknown, and long blocks make a long tail (dense, batch 256: 1380 us at U = 1, 1516 at U = 8).
int choose_heads_per_warp(const dsa_problem* p, const Plan& pl, int w, int64_t bound, size_t smem_deep,
                          size_t smem_shallow, int num_sms, int* stages) {
    const bool want_shallow = (p->plan_flags & DSA_PLAN_RING_SHALLOW) != 0 && smem_shallow != 0;
    const bool want_deep = (p->plan_flags & DSA_PLAN_RING_DEEP) != 0 && !want_shallow;
    *stages = want_shallow ? kGroupStagesShallow : kGroupStages;
    if (pl.n_split > 1) return 1;
    const double tiles = std::max(1.0, (double)bound / std::max(pl.tile, 1));
    const double build = 3.0;                              // list building, in units of one 16-key tile
    int best = 0;
    double best_cost = 0;
    for (int shallow = 0; shallow < 2; ++shallow) {
        const size_t smem = shallow ? smem_shallow : smem_deep;
        if (shallow ? (smem == 0 || want_deep) : want_shallow) continue;
        const int64_t per_sm = std::max<int64_t>(1, (int64_t)(228 * 1024) / (int64_t)(smem + 1024));
        const double slots = (double)per_sm * num_sms;
        for (int u = 1; u * w <= p->num_kv_heads; u *= 2) {
            if (p->num_kv_heads % (u * w)) break;
            const double blocks = (double)p->batch * (p->num_kv_heads / (u * w));
            const double waves = blocks / slots;
            const double block_time = build + u * tiles;
            // how long a warp takes per tile depends on how many warps share its SM: 8 (the deep ring,
            // full) is the unit; fewer run up to a third faster, the shallow ring's 12 run 1.55 x slower
            const double full = (double)per_sm * w / 8.0;
            const double load = std::min(waves, 1.0) * full;
            const double per_tile = load <= 1.0 ? 0.67 + 0.33 * load : 1.0 + 1.1 * (load - 1.0);
            double cost = block_time * per_tile;
            if (waves > 1.0) cost *= waves * (1.0 + 0.5 * std::max(0.0, std::ceil(waves - 0.004) / waves - 1.0));
            if (shallow) cost *= 1.02;
            if (best == 0 || cost < best_cost * 1.005) {    // (ties go to the larger U: a grid that just fits has no turnover)
                best = u; best_cost = cost;
                *stages = shallow ? kGroupStagesShallow : kGroupStages;
            }
        }
    }
    return std::max(best, 1);
}

int32_t make_plan(const dsa_problem* p, const dsa_diag_params* d, Plan* pl) {
    int32_t rc = check_problem(p);
    if (rc != DSA_OK) return rc;
    rc = check_diag(p, d);
    if (rc != DSA_OK) return rc;
    if (!d && p->ring_size > 0) return DSA_ERR_INVALID_ARG;    // dense attention needs every token
    const int G = p->num_q_heads / p->num_kv_heads;
    pl->G = G;
    pl->mode = !d ? MODE_DENSE
                  : (d->mode == DSA_MASK_WINDOW ? MODE_WINDOW : (d->mode == DSA_MASK_GRID ? MODE_GRID : MODE_LIST));
    // per-query-head masks inside a group: rows of the union are read, heads mask individually
    pl->headmask = pl->mode == MODE_LIST && G > 1 && d->mask_heads == p->num_q_heads;
    pl->bitmap_words = pl->mode == MODE_LIST ? (d->window + 31) / 32 : 0;
    pl->select = pl->mode == MODE_LIST && d->select != 0;

    // upper bound of kept rows per (request, kv head)
    int64_t bound = p->max_seq_len;
    if (d) {
        const int64_t lp = p->max_prompt_len > 0 ? p->max_prompt_len : p->max_seq_len;
        int64_t dec = d->window;
        if (pl->mode != MODE_WINDOW) dec = std::min<int64_t>(d->window, (int64_t)d->n_att * (pl->headmask ? G : 1));
        bound = std::min<int64_t>(bound, lp + dec + d->n_sink);
    }
    if (bound < 1) bound = 1;

    const int kNumSMs = sm_count();
    // bf16 runs on the tensor-core kernel (one warp per work item); fp32 on the CUDA-core kernel.
    // DSA_PLAN_CUDA_CORES forces the latter for bf16 too (comparison runs).
    pl->mma = p->dtype == DSA_BF16 && !(p->plan_flags & DSA_PLAN_CUDA_CORES);
    pl->mma_warps = 1;
    pl->mma_kw = 1;
    pl->mma_cl = 1;
    pl->mma_stages = kMmaStages;
    pl->group_w = 0;
    pl->group_u = 0;
    pl->group_stages = kGroupStages;
    pl->gather = false;
    pl->producers = false;
    pl->copy_only = false;
    pl->gather_rows_per_stride_b = 0;
    pl->gather_rows = 0;
    pl->heads = false;
    pl->dir_cap = pl->kidx_cap = 0;
    pl->window = d ? d->window : 0;
    pl->blocks = 0;
    if (pl->mma) {
        const bool shared_mask = pl->mode != MODE_LIST || (d->mask_heads == 1 && !pl->select);
        // two kv heads per block (measured: 2 beats 1 and 4) when the row list can be shared
        if (shared_mask && p->num_kv_heads % 2 == 0) pl->mma_warps = 2;
    }
    // tile and ring depth of the kernel that will run (they do not depend on the row-list length)
    auto shape_of = [&](int chunk, KernelShape* shape) -> int32_t {
        return dispatch(p->dtype, p->head_dim, [&](auto t, auto dd) -> int32_t {
            using T = decltype(t);
            return kernel_shape<T, decltype(dd)::value>(kernel_query(*pl), chunk, pl->bitmap_words, shape)
                       ? DSA_OK : DSA_ERR_UNSUPPORTED;
        });
    };
    KernelShape shape = {};
    rc = shape_of(0, &shape);
    if (rc != DSA_OK) return rc;
    pl->tile = shape.tile;
    pl->stages = shape.stages;

    int chunk;
    if (p->split_tokens > 0) {
        chunk = std::min(MAX_CHUNK, round_up(p->split_tokens, pl->tile));
    } else {
        // One work item streams about 12 GB/s on its own, and a split costs the combine launch, so:
        // split only while fewer than ~6 warps (4 blocks of the CUDA-core kernel) per SM exist,
        // never below 96 (128) rows per item, and balance the splits (equal chunks rather than
        // full ones plus a short tail).
        const int64_t pairs = (int64_t)std::max(p->batch, 1) * p->num_kv_heads;
        const int64_t target = (pl->mma ? 6 : 4) * kNumSMs;        // a work item is a warp / a 4-warp block
        int64_t want_split = std::max<int64_t>(1, (target + pairs - 1) / pairs);
        // From half the warp slots on, one whole item per warp in a single wave beats two splits
        // that spill into a second wave (640-864 pairs of ~400 rows: 30-35 us against 36-43 us).
        if (pl->mma && pairs >= 4 * kNumSMs) want_split = 1;
        want_split = std::min<int64_t>(want_split, std::max<int64_t>(1, bound / (pl->mma ? 96 : 128)));
        int max_chunk = MAX_CHUNK;
        // Too few pairs to fill the device, and a request fits one (long) row list: the
        // tensor-core kernel puts kMmaItemWarps warps on one work item and merges them in shared
        // memory -- the same parallelism without partial results and, up to kMmaItemWarps pieces,
        // without the combine launch.  Those blocks hold four rings, so a list of twice the usual
        // length costs no occupancy, but only two of them fit an SM: not used where they would
        // make between one and two waves of short items (measured at 384 pairs of 408 rows:
        // 32.8 us against 29.7 us for three splits and the combine; with ~1000-row items the
        // single launch still wins there).  Requests beyond 2048 rows need the combine anyway;
        // there the merge on top of it measured as a small loss.
        // (a forced head-group kernel takes the place of the small-launch form as well)
        // (a forced cluster size brings this form with it: clusters exist only on top of it)
        const bool cluster_forced = (p->plan_flags & (DSA_PLAN_CLUSTER2 | DSA_PLAN_CLUSTER4)) != 0 &&
                                    !pl->headmask && !pl->select;
        if (pl->mma && (want_split >= 2 || cluster_forced) && bound <= 2 * MAX_CHUNK &&
            !(p->plan_flags & (DSA_PLAN_NO_ITEM_WARPS | DSA_PLAN_GROUP))) {
            const int64_t kw_blocks = pairs * ((want_split + kMmaItemWarps - 1) / kMmaItemWarps);
            if (cluster_forced || kw_blocks <= 2 * kNumSMs || kw_blocks >= 4 * kNumSMs || bound > MAX_CHUNK) {
                pl->mma_kw = kMmaItemWarps;
                pl->mma_warps = 1;
                want_split = (want_split + kMmaItemWarps - 1) / kMmaItemWarps;
                max_chunk = 2 * MAX_CHUNK;
            }
        }
        want_split = std::max<int64_t>(want_split, (bound + max_chunk - 1) / max_chunk);
        // Smaller launches still: a CLUSTER of 2 or 4 such blocks shares the item (8 or 16 warps with one
        // to three tiles each, all in flight at once) and block 0 collects the others' states through
        // distributed shared memory -- while every block of every cluster is resident at once (two
        // blocks per SM) and a block still gets a few tiles.  Head-independent masks, no HBM splits.
        // (Measured, single calls with a cold L2: GQA long-sequence configuration 18.4 -> 16.4 us, paged
        // workload at batch 1 / 2: 16.4 -> 14.3 us with clusters of four; clusters of two at batch 4: no
        // change; clusters that do not all fit at once lose: batch 8, 22.5 -> 26.7 / 38.9 us.)
        // Where the plan would otherwise cut the item into 2-4 splits with partials in HBM and a combine
        // launch, the cluster takes the place of those splits.
        int cluster = 1;
        if (pl->mma_kw > 1 && want_split <= 4 && !pl->headmask && !pl->select && !(p->plan_flags & DSA_PLAN_NO_CLUSTER)) {
            const int forced = (p->plan_flags & DSA_PLAN_CLUSTER4) ? 4 : ((p->plan_flags & DSA_PLAN_CLUSTER2) ? 2 : 0);
            if (forced) cluster = forced >= want_split ? forced : 1;
            else if (pairs * 4 <= 2 * kNumSMs && bound >= 4 * 96) cluster = 4;
            else if (want_split <= 2 && pairs * 2 <= 2 * kNumSMs && bound >= 2 * 96) cluster = 2;
        }
        if (cluster > 1) {
            pl->mma_cl = cluster;
            want_split = cluster;                             // (row ranges per block; the result is final: n_split is reset below)
        }
        // Requests too long for one row list are split anyway; when the (request, kv head) pairs
        // alone fill half the device's warp slots, ~512-row items balance better across the SMs
        // than ~900-row ones (measured on dense calls: +3-10 % at 640-4096 pairs, a loss below).
        if (pl->mma_kw == 1 && bound > MAX_CHUNK && pairs >= 4 * kNumSMs)
            want_split = std::max<int64_t>(want_split, (bound + 511) / 512);
        const int64_t c = (bound + want_split - 1) / want_split;
        chunk = std::min(max_chunk, round_up((int)c, pl->tile));
    }
    pl->chunk = chunk;
    pl->n_split = (int)((bound + chunk - 1) / chunk);
    if (pl->mma_cl > 1) {
        // the blocks of a cluster cover the row ranges [r chunk, (r + 1) chunk) and merge on chip
        if (pl->n_split > pl->mma_cl || p->split_tokens > 0) pl->mma_cl = 1;
        else pl->n_split = 1;
    }
    if (pl->n_split > kMaxSplits) return DSA_ERR_UNSUPPORTED;   // the combine kernel holds one weight per split
    pl->grid = (int64_t)p->batch * p->num_kv_heads * pl->n_split;
    if (pl->grid > 0x7fffffffLL) return DSA_ERR_UNSUPPORTED;

    // Head-group form: one row list per (request, split), built by a block of W warps and streamed by
    // each of them for U kv heads back to back.  Needs a mask that does not depend on the head.
    // With U = 1 it performs like the two-heads-per-block kernel (22.2 / 37.4 / 70.1 / 140 / 263 us
    // against 22.6 / 39.0 / 72.4 / 142 / 268 us on the paged workload at batch 16 ... 256); larger U
    // amortise the list over more heads and, more important, let the planner make the grid just
    // fit the device (see choose_heads_per_warp).
    if (pl->mma && pl->mma_kw == 1 && !(p->plan_flags & DSA_PLAN_NO_GROUP)) {
        const bool shared_mask = pl->mode != MODE_LIST || (d->mask_heads == 1 && !pl->select);
        const bool forced = (p->plan_flags & DSA_PLAN_GROUP) != 0;
        const int w = forced ? ((p->plan_flags & DSA_PLAN_GROUP_W4) ? 4 : 2) : 4;
        if (shared_mask && p->num_kv_heads % w == 0) {
            int u = (int)((p->plan_flags & DSA_PLAN_HEADS_PER_WARP_MASK) >> DSA_PLAN_HEADS_PER_WARP_SHIFT);
            int stages = (p->plan_flags & DSA_PLAN_RING_SHALLOW) ? kGroupStagesShallow : kGroupStages;
            if (!forced || u < 1) {
                Plan probe = *pl;
                probe.group_w = w;
                KernelShape gs[2] = {};
                int32_t rcg = DSA_OK;
                for (int sh = 0; sh < 2 && rcg == DSA_OK; ++sh) {
                    probe.group_stages = sh ? kGroupStagesShallow : kGroupStages;
                    rcg = dispatch(p->dtype, p->head_dim, [&](auto t, auto dd) -> int32_t {
                        using T = decltype(t);
                        return kernel_shape<T, decltype(dd)::value>(kernel_query(probe), pl->chunk, pl->bitmap_words, &gs[sh])
                                   ? DSA_OK : DSA_ERR_UNSUPPORTED;
                    });
                }
                u = rcg == DSA_OK ? choose_heads_per_warp(p, *pl, w, bound, gs[0].smem, gs[1].smem, kNumSMs, &stages) : 0;
            }
            if (u >= 1 && p->num_kv_heads % (w * u) == 0) {
                pl->group_w = w;
                pl->group_u = u;
                pl->group_stages = stages;
                if (w == 4 && (p->plan_flags & DSA_PLAN_GATHER) && !(p->plan_flags & DSA_PLAN_NO_GATHER))
                    pl->gather = gather_view(p, &pl->gather_rows_per_stride_b, &pl->gather_rows);
                // Producer warps pay where the grid is more than one wave of deep-ring blocks (measured on the
                // paged workload: batch 224 / 256, 1.5 / 1.7 waves: -3.5 % / -1.7 %; window 1024: -1.4 %), not
                // where all blocks are resident from the start (batch 32 ... 128: +2 ... 3 %), and with the
                // shallow ring they cannot run three blocks to an SM at all (registers).
                const int64_t n_blocks = (int64_t)p->batch * pl->n_split * (p->num_kv_heads / (w * u));
                const bool pays = stages == kGroupStages && pl->n_split == 1 && n_blocks > 2 * (int64_t)kNumSMs;
                if (w == 4 && !pl->gather && !(p->plan_flags & DSA_PLAN_NO_PRODUCERS) &&
                    ((p->plan_flags & DSA_PLAN_PRODUCERS) || pays))
                    pl->producers = true;
                pl->mma_warps = 1;
                pl->blocks = (int64_t)p->batch * pl->n_split * (p->num_kv_heads / (w * u));
            }
        }
    }
    // Per-head-list form (list masks per kv or query head, fused selection): the tables every head of a
    // request shares are built once per block, each head only derives which window candidates it keeps.
    if (pl->mma && pl->mma_kw == 1 && pl->group_w == 0 && !(p->plan_flags & DSA_PLAN_NO_GROUP) &&
        pl->mode == MODE_LIST && p->num_kv_heads % kHeadsWarps == 0) {
        const bool forced = (p->plan_flags & DSA_PLAN_GROUP) != 0;
        const int64_t lp = p->max_prompt_len > 0 ? p->max_prompt_len : p->max_seq_len;
        const int64_t dir_cap = std::min<int64_t>(p->max_seq_len, lp + d->n_sink);
        const int64_t kcap = std::min<int64_t>(d->window, (int64_t)d->n_att * (pl->headmask ? G : 1) + d->n_sink);
        Plan probe = *pl;
        probe.heads = true;
        probe.dir_cap = (int)std::max<int64_t>(dir_cap, 1);
        probe.kidx_cap = (int)std::max<int64_t>(kcap, 1);
        KernelShape hs = {};
        const int32_t rch = dispatch(p->dtype, p->head_dim, [&](auto t, auto dd) -> int32_t {
            using T = decltype(t);
            return kernel_shape<T, decltype(dd)::value>(kernel_query(probe), pl->chunk, pl->bitmap_words, &hs)
                       ? DSA_OK : DSA_ERR_UNSUPPORTED;
        });
        // two blocks per SM or nothing: with one, a block's set-up has nobody to hide behind
        if (rch == DSA_OK && hs.smem <= 112 * 1024 && d->window <= 65536 && (!forced || (p->plan_flags & DSA_PLAN_GROUP_W4))) {
            int u = (int)((p->plan_flags & DSA_PLAN_HEADS_PER_WARP_MASK) >> DSA_PLAN_HEADS_PER_WARP_SHIFT);
            if (!forced || u < 1) {
                int stages_unused = 0;
                u = choose_heads_per_warp(p, *pl, kHeadsWarps, bound, hs.smem, 0, kNumSMs, &stages_unused);
            }
            if (u >= 1 && p->num_kv_heads % (kHeadsWarps * u) == 0) {
                pl->heads = true;
                pl->dir_cap = probe.dir_cap;
                pl->kidx_cap = probe.kidx_cap;
                pl->group_u = u;
                pl->mma_warps = 1;
                pl->blocks = (int64_t)p->batch * pl->n_split * (p->num_kv_heads / (kHeadsWarps * u));
            }
        }
    }
    rc = shape_of(pl->chunk, &shape);                         // (the small-launch form may have been chosen since)
    if (rc != DSA_OK) return rc;
    pl->stages = shape.stages;

    // Ring depth of the two-heads-per-block kernel.  Shared memory decides how many blocks an SM
    // holds, and a launch of a few waves pays for every block beyond a whole number of them: a
    // last wave costs at least about half a full one, however few blocks it has (measured on the
    // paged workload, 32 heads: batch 36 -> 40 with the deep ring 43 -> 64 us).  The shallow ring
    // fits half as many blocks again per SM (and loses about 1 % when waves are many), so estimate
    // both and take the shallow one when it is clearly cheaper (batch 40 / 48 / 80: 48 / 55 / 94 us shallow against 64 / 67 / 102 deep;
    // batch 64 / 72: 73 / 79 deep against 88 / 91 shallow).
    // Only for unsplit plans: the splits of a long request differ so much in length (many are
    // empty) that their blocks pack into waves far better than the estimate assumes (measured: a
    // loss of 10 % on the dense calls at batch 1-8).
    const bool force_shallow = (p->plan_flags & DSA_PLAN_RING_SHALLOW) != 0;
    const bool force_deep = (p->plan_flags & DSA_PLAN_RING_DEEP) != 0 && !force_shallow;
    if (pl->mma && pl->group_w == 0 && !pl->heads && pl->mma_warps == 2 && pl->mma_kw == 1 && p->split_tokens == 0 &&
        (pl->n_split == 1 || force_shallow) && !force_deep) {
        Plan alt = *pl;
        alt.mma_stages = kMmaStagesShallow;
        KernelShape shallow = {};
        const int32_t rc2 = dispatch(p->dtype, p->head_dim, [&](auto t, auto dd) -> int32_t {
            using T = decltype(t);
            return kernel_shape<T, decltype(dd)::value>(kernel_query(alt), pl->chunk, pl->bitmap_words, &shallow)
                       ? DSA_OK : DSA_ERR_UNSUPPORTED;
        });
        auto cost = [&](size_t smem) {
            // blocks an SM holds: shared memory (1 KB of it reserved per block), at most 8 by registers
            const int64_t per_sm = std::min<int64_t>(8, (int64_t)(227 * 1024) / (int64_t)(smem + 1024));
            const double cap = (double)std::max<int64_t>(per_sm, 1) * kNumSMs;
            const double waves = (double)(pl->grid / 2) / cap;
            double whole = std::floor(waves), rest = waves - whole;
            if (rest < 0.05) rest = 0;                        // a few extra blocks ride on the shortest items
            if (rest > 0 && whole >= 1) rest = std::max(rest, 0.47);
            return (whole + rest) * cap;
        };
        if (rc2 == DSA_OK && shallow.stages == kMmaStagesShallow) {
            const bool forced = force_shallow;
            // (with many waves the two are within a few per cent either way: stay with the deep ring
            // unless the estimate is clearly better)
            const double margin = (double)(pl->grid / 2) < 3.0 * 4 * kNumSMs ? 1.0 : 0.97;
            if (forced || cost(shallow.smem) < margin * cost(shape.smem)) {
                pl->mma_stages = kMmaStagesShallow;
                pl->stages = shallow.stages;
                shape = shallow;
            }
        }
    }
    pl->smem = shape.smem;
    if (pl->smem > 200 * 1024) return DSA_ERR_UNSUPPORTED;     // window too large for LIST bitmaps

    if (pl->n_split > 1) {
        const size_t rows = (size_t)p->batch * p->num_q_heads * pl->n_split;
        pl->ws_out_bytes = (rows * p->head_dim * sizeof(float) + 255) / 256 * 256;
        pl->ws_lse_bytes = (rows * sizeof(float) + 255) / 256 * 256;
        // selection candidates per split (logit, distance) and the trace entry per (request, head)
        pl->ws_sel_bytes = pl->select ? pl->ws_lse_bytes : 0;
        const size_t k_bytes = pl->select ? ((size_t)p->batch * p->num_q_heads * sizeof(int) + 255) / 256 * 256 : 0;
        pl->ws_total = pl->ws_out_bytes + pl->ws_lse_bytes + 2 * pl->ws_sel_bytes + k_bytes;
    } else {
        pl->ws_out_bytes = pl->ws_lse_bytes = pl->ws_sel_bytes = 0;
        pl->ws_total = 0;
    }
    return DSA_OK;
}

void fill_args(const dsa_problem* p, const dsa_diag_params* d, const Plan& pl, AttnArgs* a) {
    *a = AttnArgs{};
    a->q = p->q; a->k = p->k_cache; a->v = p->v_cache;
    a->stride_b = p->stride_batch; a->stride_tok = p->stride_token; a->stride_head = p->stride_head;
    a->seq_len = p->seq_len; a->prompt_len = p->prompt_len;
    a->seq_len_rw = const_cast<int*>(p->seq_len);
    a->block_table = p->block_table;
    a->max_blocks = p->max_blocks; a->block_size = p->block_size; a->num_blocks = p->num_blocks;
    a->max_seq_len = p->max_seq_len;
    a->ring_size = p->ring_size; a->ring_sinks = p->ring_sinks;
    // the prompt length the kernels trust: with a bounded cache the region of a request holds
    // max_prompt_len + ring_sinks + ring_size tokens, so a longer device prompt_len is cut there
    a->prompt_cap = p->ring_size > 0 ? p->max_prompt_len : p->max_seq_len;
    a->B = p->batch; a->H_q = p->num_q_heads; a->H_kv = p->num_kv_heads;
    const float scale = p->sm_scale > 0.f ? p->sm_scale : 1.f / sqrtf((float)p->head_dim);
    a->scale_log2 = scale * LOG2E;
    a->mask.mode = pl.mode;
    a->mask.window = d ? d->window : 0;
    a->mask.n_att = d ? (pl.mode == MODE_WINDOW ? d->window : d->n_att) : 0;
    a->mask.stride = (d && pl.mode == MODE_GRID) ? d->grid_w + d->row_extra : 1;
    a->mask.n_sink = d ? d->n_sink : 0;
    a->mask.skip_offsets = (d && pl.mode == MODE_LIST) ? d->skip_offsets : nullptr;
    a->mask.select = pl.select ? 1 : 0;
    a->mask.mask_heads = (d && pl.mode == MODE_LIST) ? d->mask_heads : 1;
    a->mask.trace_len = (d && pl.mode == MODE_LIST) ? d->trace_len : 0;
    a->mask.bitmap_words = pl.bitmap_words;
    a->mask.skip_bitmap = (d && pl.mode == MODE_LIST) ? d->skip_bitmap : nullptr;
    a->chunk = pl.chunk; a->n_split = pl.n_split;
    a->heads_per_warp = pl.group_u;
    a->dir_cap = pl.dir_cap; a->kidx_cap = pl.kidx_cap;
    a->n_items = (int)pl.grid;
    a->out = nullptr; a->lse = nullptr; a->out_part = nullptr; a->lse_part = nullptr;
    a->sel_val_part = nullptr; a->sel_off_part = nullptr; a->sel_k = nullptr;
    a->step_append = 0; a->k_new = nullptr; a->v_new = nullptr;
    a->wait_timeouts = nullptr;
    a->early_list = (p->plan_flags & DSA_PLAN_METADATA_STABLE) ? 1 : 0;
}

// `after_attention`: the combine follows the attention kernel of the same call.  It is then
// launched with programmatic stream serialisation: its blocks may be scheduled while the last wave
// of the attention kernel is still running (the attention kernels signal early with
// griddepcontrol.launch_dependents) and wait inside the kernel (griddepcontrol.wait) until that
// grid has completed and its writes are visible -- the launch latency of the second kernel hides
// behind the first.
template <typename T>
cudaError_t launch_combine_t(const float* out_part, const float* lse_part, int64_t rows, int D, int n_split,
                             void* out, float* lse, cudaStream_t st, const float* sel_val, const int* sel_off,
                             const int* sel_k, int* trace, int trace_len, bool after_attention,
                             unsigned* skip_bitmap, int bitmap_words, int window) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)rows);
    cfg.blockDim = dim3((unsigned)((D + 31) / 32 * 32));    // whole warps: the block reductions shuffle with a full mask
    cfg.dynamicSmemBytes = (size_t)n_split * sizeof(float);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_attention ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, dsa_combine_kernel<T>, out_part, lse_part, D, n_split, out, lse, sel_val,
                              sel_off, sel_k, trace, trace_len, skip_bitmap, bitmap_words, window);
}

int32_t launch_combine(const float* out_part, const float* lse_part, int64_t rows, int D, int n_split,
                       void* out, float* lse, int dtype, cudaStream_t st, const float* sel_val = nullptr,
                       const int* sel_off = nullptr, const int* sel_k = nullptr, int* trace = nullptr,
                       int trace_len = 0, bool after_attention = false, unsigned* skip_bitmap = nullptr,
                       int bitmap_words = 0, int window = 0) {
    if (rows == 0) return DSA_OK;
    const cudaError_t e =
        dtype == DSA_BF16
            ? launch_combine_t<__nv_bfloat16>(out_part, lse_part, rows, D, n_split, out, lse, st, sel_val, sel_off,
                                              sel_k, trace, trace_len, after_attention, skip_bitmap, bitmap_words,
                                              window)
            : launch_combine_t<float>(out_part, lse_part, rows, D, n_split, out, lse, st, sel_val, sel_off, sel_k,
                                      trace, trace_len, after_attention, skip_bitmap, bitmap_words, window);
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}

int32_t launch_append(const dsa_problem* problem, const void* k_new, const void* v_new, bool advance,
                      cudaStream_t st);

// ---- tensor maps of the gather kernel --------------------------------------------------------------
// Bounded waits of the gather kernel that gave up, per device (dsa_wait_timeouts reads it).
__device__ int g_wait_timeouts;

cudaError_t wait_timeouts_address(int** out) {
    static std::atomic<int*> addr[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int* ptr = addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_wait_timeouts);
        if (e != cudaSuccess) return e;
        addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return cudaSuccess;
}

// cuTensorMapEncodeTiled, looked up through the runtime (the library does not link the driver).
using TensorMapEncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                       const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                       CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

TensorMapEncodeFn tensor_map_encoder() {
    static std::atomic<void*> cached{nullptr};
    void* fn = cached.load(std::memory_order_acquire);
    if (!fn) {
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess ||
            qr != cudaDriverEntryPointSuccess || !fn) {
            cudaGetLastError();
            return nullptr;
        }
        cached.store(fn, std::memory_order_release);
    }
    return reinterpret_cast<TensorMapEncodeFn>(fn);
}

// Views of the K and V caches for the plan's gather kernel: boxes of 64 elements (128 bytes) of one
// row, which the gather4 copy stacks four at a time; 128-byte swizzle, so that the 8 rows an
// ldmatrix reads lie in different banks.
int32_t build_gather_maps(const dsa_problem* p, const Plan& pl, GatherMaps* g) {
    const TensorMapEncodeFn encode = tensor_map_encoder();
    if (!encode) return DSA_ERR_UNSUPPORTED;
    const cuuint64_t dims[2] = {(cuuint64_t)((int64_t)(p->num_kv_heads - 1) * p->stride_head + p->head_dim),
                                (cuuint64_t)pl.gather_rows};
    const cuuint64_t pitch[1] = {(cuuint64_t)p->stride_token * 2};
    const cuuint32_t box[2] = {64u, 1u};
    const cuuint32_t step[2] = {1u, 1u};
    for (int kv = 0; kv < 2; ++kv) {
        const CUresult r = encode(kv ? &g->v : &g->k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                                  const_cast<void*>(kv ? p->v_cache : p->k_cache), dims, pitch, box, step,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return DSA_ERR_UNSUPPORTED;
    }
    g->rows_per_stride_b = pl.gather_rows_per_stride_b;
    g->oob_row = (int)pl.gather_rows;
    return DSA_OK;
}

// k_new / v_new non-NULL: the fused decode step -- seq_len counts the tokens already cached, the
// token being decoded is appended by this call and attended to as well.
int32_t run_attention(const dsa_problem* p, const dsa_diag_params* d, void* out, float* lse,
                      void* workspace, size_t workspace_bytes, void* stream, const void* k_new = nullptr,
                      const void* v_new = nullptr, bool copy_only = false) {
    Plan pl;
    int32_t rc = make_plan(p, d, &pl);
    if (rc != DSA_OK) return rc;
    if (copy_only) {
        // the measuring form exists for the plain four-warp head-group kernel: same grid, same lists, same copies
        if (pl.group_w != 4 || pl.heads || k_new) return DSA_ERR_UNSUPPORTED;
        pl.producers = false;
        pl.gather = false;
        pl.copy_only = true;
    }
    if (p->batch == 0) return DSA_OK;
    if (!out || !lse || !aligned16(out)) return DSA_ERR_INVALID_ARG;
    const bool step = k_new != nullptr;
    if (step && (!v_new || !aligned16(k_new) || !aligned16(v_new))) return DSA_ERR_INVALID_ARG;
    if (pl.ws_total > 0) {
        if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return DSA_ERR_INVALID_ARG;
        if (workspace_bytes < pl.ws_total) return DSA_ERR_WORKSPACE_TOO_SMALL;
    }
    AttnArgs a;
    fill_args(p, d, pl, &a);
    if (pl.n_split > 1) {
        a.out_part = reinterpret_cast<float*>(workspace);
        unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
        a.lse_part = reinterpret_cast<float*>(ws + pl.ws_out_bytes);
        if (pl.select) {
            a.sel_val_part = reinterpret_cast<float*>(ws + pl.ws_out_bytes + pl.ws_lse_bytes);
            a.sel_off_part = reinterpret_cast<int*>(ws + pl.ws_out_bytes + pl.ws_lse_bytes + pl.ws_sel_bytes);
            a.sel_k = reinterpret_cast<int*>(ws + pl.ws_out_bytes + pl.ws_lse_bytes + 2 * pl.ws_sel_bytes);
        }
    } else {
        a.out = out; a.lse = lse;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (step) {
        a.step_append = 1;
        if (pl.mma) {
            a.k_new = k_new; a.v_new = v_new;             // read and stored by the attention kernel itself
        } else {
            // CUDA-core kernel: the rows go to the cache in a launch of their own first
            rc = launch_append(p, k_new, v_new, false, st);
            if (rc != DSA_OK) return rc;
        }
    }
    if (pl.gather || pl.producers) {                  // (the kernels with bounded mbarrier waits)
        const cudaError_t e = wait_timeouts_address(&a.wait_timeouts);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    GatherMaps maps;
    if (pl.gather) {
        rc = build_gather_maps(p, pl, &maps);
        if (rc != DSA_OK) return rc;
    }
    cudaError_t err = cudaSuccess;
    rc = dispatch(p->dtype, p->head_dim, [&](auto t, auto dd) -> int32_t {
        using T = decltype(t);
        err = kernel_launch<T, decltype(dd)::value>(kernel_query(pl), step && pl.mma, a, pl.grid, pl.smem, st,
                                                    pl.blocks, pl.gather ? &maps : nullptr);
        return DSA_OK;
    });
    if (rc != DSA_OK) return rc;
    if (err != cudaSuccess) return cuda_fail(err);
    if (pl.n_split > 1)
        return launch_combine(a.out_part, a.lse_part, (int64_t)p->batch * p->num_q_heads, p->head_dim,
                              pl.n_split, out, lse, p->dtype, st, a.sel_val_part, a.sel_off_part, a.sel_k,
                              pl.select ? d->skip_offsets : nullptr, pl.select ? d->trace_len : 0, true,
                              pl.select ? d->skip_bitmap : nullptr, pl.bitmap_words, pl.select ? d->window : 0);
    return DSA_OK;
}

int32_t launch_append(const dsa_problem* problem, const void* k_new, const void* v_new, bool advance,
                      cudaStream_t st) {
    Plan pl = {};
    pl.mode = MODE_WINDOW;
    pl.chunk = 0; pl.n_split = 1;
    AttnArgs a;
    fill_args(problem, nullptr, pl, &a);
    const unsigned grid = (unsigned)problem->batch;
    const int cap = problem->max_seq_len;
    if (problem->dtype == DSA_BF16)
        dsa_append_kv_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(a, reinterpret_cast<const __nv_bfloat16*>(k_new),
                                                               reinterpret_cast<const __nv_bfloat16*>(v_new),
                                                               problem->head_dim, cap, advance);
    else
        dsa_append_kv_kernel<float><<<grid, 256, 0, st>>>(a, reinterpret_cast<const float*>(k_new),
                                                        reinterpret_cast<const float*>(v_new), problem->head_dim, cap,
                                                        advance);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}

}  // namespace

extern "C" {

int32_t dsa_version(void) { return DSA_VERSION; }

const char* dsa_status_string(int32_t status) {
    switch (status) {
        case DSA_OK: return "ok";
        case DSA_ERR_INVALID_ARG: return "invalid argument";
        case DSA_ERR_UNSUPPORTED: return "unsupported configuration";
        case DSA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case DSA_ERR_CUDA: return "CUDA runtime error";
        default: return "unknown status";
    }
}

int32_t dsa_last_cuda_error(void) { return g_last_cuda_error; }

int32_t dsa_debug_copy_only(const dsa_problem* problem, const dsa_diag_params* diag, void* out, float* lse,
                            void* workspace, size_t workspace_bytes, void* stream) {
    return run_attention(problem, diag, out, lse, workspace, workspace_bytes, stream, nullptr, nullptr, true);
}

int32_t dsa_build_skip_bitmap(const dsa_problem* problem, const dsa_diag_params* diag, void* stream) {
    if (!diag) return DSA_ERR_INVALID_ARG;
    Plan pl;
    const int32_t rc = make_plan(problem, diag, &pl);
    if (rc != DSA_OK) return rc;
    if (pl.mode != MODE_LIST || !diag->skip_bitmap) return DSA_ERR_INVALID_ARG;
    if (problem->batch == 0) return DSA_OK;
    AttnArgs a;
    fill_args(problem, diag, pl, &a);
    dsa_build_skip_bitmap_kernel<<<(unsigned)(problem->batch * diag->mask_heads), 128, 0,
                                   reinterpret_cast<cudaStream_t>(stream)>>>(a);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}

int32_t dsa_debug_wait_giveup(void* stream) {
    int* counter = nullptr;
    const cudaError_t e0 = wait_timeouts_address(&counter);
    if (e0 != cudaSuccess) return cuda_fail(e0);
    dsa_wait_giveup_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(counter);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}

int32_t dsa_wait_timeouts(int32_t* count_out) {
    if (!count_out) return DSA_ERR_INVALID_ARG;
    int n = 0;
    const cudaError_t e = cudaMemcpyFromSymbol(&n, g_wait_timeouts, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    *count_out = n;
    return DSA_OK;
}

static cudaError_t static_scratch_address(void** out);

int32_t dsa_prepare(void) {
    cudaError_t e = kernel_prepare<__nv_bfloat16, 64>();
    if (e == cudaSuccess) e = kernel_prepare<__nv_bfloat16, 128>();
    if (e == cudaSuccess) e = kernel_prepare<float, 64>();
    if (e == cudaSuccess) e = kernel_prepare<float, 128>();
    void* scratch = nullptr;
    if (e == cudaSuccess) e = static_scratch_address(&scratch);   // (and remember it for this device)
    int* counter = nullptr;
    if (e == cudaSuccess) e = wait_timeouts_address(&counter);    // (likewise: the give-up counter of the bounded waits)
    tensor_map_encoder();                                         // (and the driver entry point the tensor-map form needs)
    sm_count();
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}

int32_t dsa_workspace_size(const dsa_problem* problem, const dsa_diag_params* diag, size_t* bytes) {
    if (!bytes) return DSA_ERR_INVALID_ARG;
    Plan pl;
    const int32_t rc = make_plan(problem, diag, &pl);
    if (rc != DSA_OK) return rc;
    *bytes = pl.ws_total;
    return DSA_OK;
}

int32_t dsa_query_plan(const dsa_problem* problem, const dsa_diag_params* diag, dsa_plan_info* info) {
    if (!info) return DSA_ERR_INVALID_ARG;
    Plan pl;
    const int32_t rc = make_plan(problem, diag, &pl);
    if (rc != DSA_OK) return rc;
    info->split_tokens = pl.chunk;
    info->n_split = pl.n_split;
    info->launches = problem->batch == 0 ? 0 : (pl.n_split > 1 ? 2 : 1);
    const int block_warps = pl.heads ? kHeadsWarps : pl.group_w;        // (0: one of the one-block-per-item kernels)
    info->grid_blocks = (int32_t)(block_warps > 0 ? pl.blocks : (pl.mma ? pl.grid / pl.mma_warps : pl.grid));
    info->heads_per_block = block_warps * pl.group_u;
    info->block_warps = pl.mma ? (block_warps > 0 ? block_warps : pl.mma_warps * pl.mma_kw) : 4;
    info->per_head_lists = pl.heads ? 1 : 0;
    info->cluster_blocks = pl.mma_cl;
    info->tensor_map_copies = pl.gather ? 1 : 0;
    info->producer_warps = pl.producers ? pl.group_w : 0;
    if (pl.mma_cl > 1) info->grid_blocks = (int32_t)(pl.grid * pl.mma_cl);
    info->smem_bytes = (int32_t)pl.smem;
    info->tile_tokens = pl.tile;
    info->tensor_cores = pl.mma ? 1 : 0;
    info->work_items = (int32_t)pl.grid;
    info->item_warps = pl.mma ? pl.mma_kw : 1;
    info->stages = pl.stages;
    return DSA_OK;
}

int32_t dsa_decode_attention_dense(const dsa_problem* problem, void* out, float* lse, void* workspace,
                                   size_t workspace_bytes, void* stream) {
    return run_attention(problem, nullptr, out, lse, workspace, workspace_bytes, stream);
}

int32_t dsa_decode_attention_sparse(const dsa_problem* problem, const dsa_diag_params* diag, void* out,
                                    float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!diag) return DSA_ERR_INVALID_ARG;
    return run_attention(problem, diag, out, lse, workspace, workspace_bytes, stream);
}

int32_t dsa_decode_attention_host_io(const dsa_problem* problem, const dsa_diag_params* diag,
                                     const void* host_q, const int32_t* host_seq_len,
                                     const int32_t* host_prompt_len, const int32_t* host_block_table,
                                     void* dev_out, float* dev_lse, void* host_out, float* host_lse,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    const int32_t rc = check_problem(problem);
    if (rc != DSA_OK) return rc;
    if (problem->batch == 0) return DSA_OK;
    if (!host_q || !host_seq_len || !host_prompt_len || !host_out || !host_lse || !dev_out || !dev_lse)
        return DSA_ERR_INVALID_ARG;
    if ((problem->block_table != nullptr) != (host_block_table != nullptr)) return DSA_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t esize = problem->dtype == DSA_BF16 ? 2 : 4;
    const size_t n_q = (size_t)problem->batch * problem->num_q_heads * problem->head_dim;
    const size_t n_rows = (size_t)problem->batch * problem->num_q_heads;
    cudaError_t e = cudaMemcpyAsync(const_cast<void*>(problem->q), host_q, n_q * esize, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(const_cast<int32_t*>(problem->seq_len), host_seq_len, (size_t)problem->batch * 4,
                            cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(const_cast<int32_t*>(problem->prompt_len), host_prompt_len, (size_t)problem->batch * 4,
                            cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && host_block_table)
        e = cudaMemcpyAsync(const_cast<int32_t*>(problem->block_table), host_block_table,
                            (size_t)problem->batch * problem->max_blocks * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e);
    const int32_t rc2 = run_attention(problem, diag, dev_out, dev_lse, workspace, workspace_bytes, stream);
    if (rc2 != DSA_OK) return rc2;
    e = cudaMemcpyAsync(host_out, dev_out, n_q * esize, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(host_lse, dev_lse, n_rows * 4, cudaMemcpyDeviceToHost, st);
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}

// The address under which the device reaches a page-locked host buffer; nullptr when `host` is
// not such a buffer (pageable, device or unknown memory).
static void* mapped_alias(const void* host) {
    cudaPointerAttributes at = {};
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

int32_t dsa_decode_attention_host_mapped(const dsa_problem* problem, const dsa_diag_params* diag,
                                         const void* host_q, const int32_t* host_seq_len,
                                         const int32_t* host_prompt_len, const int32_t* host_block_table,
                                         void* host_out, float* host_lse, void* workspace,
                                         size_t workspace_bytes, void* stream) {
    Plan pl;
    const int32_t rc = make_plan(problem, diag, &pl);
    if (rc != DSA_OK) return rc;
    if (problem->batch == 0) return DSA_OK;
    if (!host_q || !host_seq_len || !host_prompt_len || !host_out || !host_lse) return DSA_ERR_INVALID_ARG;
    if ((problem->block_table != nullptr) != (host_block_table != nullptr)) return DSA_ERR_INVALID_ARG;
    void* q_dev = mapped_alias(host_q);
    void* out_dev = mapped_alias(host_out);
    float* lse_dev = reinterpret_cast<float*>(mapped_alias(host_lse));
    if (!q_dev || !out_dev || !lse_dev) return DSA_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t esize = problem->dtype == DSA_BF16 ? 2 : 4;
    cudaError_t e = cudaMemcpyAsync(const_cast<int32_t*>(problem->seq_len), host_seq_len,
                                    (size_t)problem->batch * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(const_cast<int32_t*>(problem->prompt_len), host_prompt_len, (size_t)problem->batch * 4,
                            cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && host_block_table)
        e = cudaMemcpyAsync(const_cast<int32_t*>(problem->block_table), host_block_table,
                            (size_t)problem->batch * problem->max_blocks * 4, cudaMemcpyHostToDevice, st);
    dsa_problem sub = *problem;
    if (pl.n_split > 1) {
        // every split of a (request, kv head) reads q: bring it over once
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(const_cast<void*>(problem->q), host_q,
                                (size_t)problem->batch * problem->num_q_heads * problem->head_dim * esize,
                                cudaMemcpyHostToDevice, st);
    } else {
        sub.q = q_dev;
    }
    if (e != cudaSuccess) return cuda_fail(e);
    return run_attention(&sub, diag, out_dev, lse_dev, workspace, workspace_bytes, stream);
}

int32_t dsa_combine_splits(const float* out_part, const float* lse_part, int32_t batch, int32_t num_q_heads,
                           int32_t head_dim, int32_t n_split, void* out, float* lse, int32_t out_dtype,
                           void* stream) {
    if (batch < 0 || num_q_heads < 1 || head_dim < 1 || head_dim > 1024 || n_split < 1) return DSA_ERR_INVALID_ARG;
    if (n_split > kMaxSplits) return DSA_ERR_UNSUPPORTED;        // weights live in 32 KB of shared memory
    if (out_dtype != DSA_BF16 && out_dtype != DSA_F32) return DSA_ERR_UNSUPPORTED;
    if (batch == 0) return DSA_OK;
    if (!out_part || !lse_part || !out) return DSA_ERR_INVALID_ARG;
    return launch_combine(out_part, lse_part, (int64_t)batch * num_q_heads, head_dim, n_split, out, lse,
                          out_dtype, reinterpret_cast<cudaStream_t>(stream));
}

int32_t dsa_append_kv(const dsa_problem* problem, const void* k_new, const void* v_new, int32_t advance,
                      void* stream) {
    const int32_t rc = check_problem(problem);
    if (rc != DSA_OK) return rc;
    if (problem->batch == 0) return DSA_OK;
    if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return DSA_ERR_INVALID_ARG;
    return launch_append(problem, k_new, v_new, advance != 0, reinterpret_cast<cudaStream_t>(stream));
}

int32_t dsa_decode_step(const dsa_problem* problem, const dsa_diag_params* diag, const void* k_new,
                        const void* v_new, void* out, float* lse, void* workspace, size_t workspace_bytes,
                        void* stream) {
    if (!k_new || !v_new) return DSA_ERR_INVALID_ARG;
    return run_attention(problem, diag, out, lse, workspace, workspace_bytes, stream, k_new, v_new);
}

int32_t dsa_advance_seq_len(int32_t* seq_len, int32_t batch, int32_t max_seq_len, void* stream) {
    if (batch < 0 || max_seq_len < 0 || (batch > 0 && !seq_len)) return DSA_ERR_INVALID_ARG;
    if (batch == 0) return DSA_OK;
    dsa_advance_seq_len_kernel<<<(unsigned)((batch + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        seq_len, batch, max_seq_len);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}

int32_t dsa_debug_kept_indices(const dsa_problem* problem, const dsa_diag_params* diag, int32_t* idx_out,
                               int32_t* count_out, int32_t max_kept, void* stream) {
    Plan pl;
    const int32_t rc = make_plan(problem, diag, &pl);
    if (rc != DSA_OK) return rc;
    if (max_kept < 0) return DSA_ERR_INVALID_ARG;
    if (problem->batch == 0) return DSA_OK;
    if (!count_out || (max_kept > 0 && !idx_out)) return DSA_ERR_INVALID_ARG;
    AttnArgs a;
    fill_args(problem, diag, pl, &a);
    const int mheads = pl.mode == MODE_LIST ? diag->mask_heads : 1;
    const size_t smem = (size_t)std::max(pl.bitmap_words, 4) * 4;
    if (smem > 48 * 1024) return DSA_ERR_UNSUPPORTED;
    dsa_kept_indices_kernel<<<(unsigned)(problem->batch * mheads), NT, smem,
                              reinterpret_cast<cudaStream_t>(stream)>>>(a, idx_out, count_out, max_kept);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA_OK : cuda_fail(e);
}


// ---- attention without caller-provided scratch ---------------------------------------------------
// Split-KV partial results normally live in the caller's workspace.  Some callers have nowhere to
// get one from: code that runs inside a region where device allocation is forbidden (a plugin
// called under a host framework's "no allocation" section, a real-time loop, a process whose memory
// pool was handed out completely at start-up).  For them the partials go to this fixed array, which
// is part of the library image: every GPU that loads the library holds these bytes until exit.
static __device__ __align__(256) unsigned char g_static_scratch[DSA_STATIC_SCRATCH_MAX];

// In host code `g_static_scratch` is only a handle for the symbol; the address kernels can use must
// be asked for, once per device and with that device current.  The per-device cache is idempotent
// (threads that race on the first call store the same address) and written atomically.
static cudaError_t static_scratch_address(void** out) {
    static std::atomic<void*> scratch_addr[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    void* ptr = scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return cudaSuccess;
}

int32_t dsa_decode_attention_static_scratch(const dsa_problem* problem, const dsa_diag_params* diag, void* out,
                                            float* lse, void* stream) {
    void* scratch = nullptr;
    const cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return cuda_fail(e);
    size_t need = 0;
    const int32_t rc = dsa_workspace_size(problem, diag, &need);
    if (rc != DSA_OK) return rc;
    if (need > DSA_STATIC_SCRATCH_MAX) return DSA_ERR_WORKSPACE_TOO_SMALL;   // problem too large for the fixed array
    // Nothing in the scratch has to start at zero: every split writes its own lse, and the output of
    // an empty split is never read, so leftovers of the previous call are harmless.
    return run_attention(problem, diag, out, lse, scratch, DSA_STATIC_SCRATCH_MAX, stream);
}

}  // extern "C"
