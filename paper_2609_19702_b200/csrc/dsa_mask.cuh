// In-kernel mask generator: turns (decode position, prompt length, window, N_att, grid stride or a
// skip trace) into the kept cache positions of one request, in ascending order, without touching
// global memory for anything but the trace.  Used by the attention kernel (to build the list of
// K/V rows it stages) and by the debug export (to write the positions out).
//
// Algorithm 1 of the paper in closed form.  A key chosen for skip_idx at step s with index j has
// distance o = s - j to the query and keeps it ("+1" shift every step), so with t = p - 1:
//   window distances  W_t = { 0 .. T },  T = min(t, N_r - 1)
//   active skips      the first n_act = clamp(t - (N_att - 1), 0, N_r - N_att) selections
//   kept              prompt [0, L_p)  u  { seq_len - 1 - o : o in W_t \ skips }
//                     u  the first n_sink decode tokens (attention sinks of the sink variants)
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace dsa {

enum : int { MODE_DENSE = 0, MODE_WINDOW = 1, MODE_GRID = 2, MODE_LIST = 3 };

struct MaskArgs {
    int mode;                  // MODE_*
    int window;                // N_r
    int n_att;                 // N_att
    int stride;                // grid_w + row_extra (GRID)
    int n_sink;                // first decode tokens that are always kept (attention sinks)
    int select;                // LIST: also run Algorithm 1's phase-2 selection and extend the trace
    int* skip_offsets;         // [B, mask_heads, trace_len] (LIST); written when select is set
    int mask_heads;
    int trace_len;
    int bitmap_words;          // 32-bit words per LIST bitmap = ceil(window / 32)
    unsigned* skip_bitmap;     // [B, mask_heads, bitmap_words] or NULL: the active entries of skip_offsets as bits
};

// The selection's result for trace slot k of mask row `row` (b * mask_heads + head): the list entry and,
// where the caller keeps one, the bit of the bitmap.
__device__ __forceinline__ void record_selection(const MaskArgs& a, int64_t row, int k, int off) {
    a.skip_offsets[row * a.trace_len + k] = off;
    if (a.skip_bitmap && off >= 0 && off < a.window)
        atomicOr(&a.skip_bitmap[row * a.bitmap_words + (off >> 5)], 1u << (off & 31));
}

// Per-request constants of the mask.
struct ReqMask {
    int S;        // clamped seq_len
    int L_p;      // clamped prompt length
    int p;        // decode tokens in the cache, current one included
    int T;        // largest window distance
    int n_win;    // window candidates = T + 1 (0 when p == 0)
    int w_lo;     // cache position of distance T
    int prefix;   // positions [0, prefix) are always kept: the prompt and the sinks older than the window
    int sink_end; // positions below this are sinks or prompt (kept even where the mask skips them)
    int n_act;    // LIST: active skip entries
    int sel_k;    // LIST with selection: trace entry this step appends (-1: no selection at this step)
    int dstar;    // GRID: column distance of the partly kept class (-1: keep none below T)
    int need;     // GRID: how many distances of class dstar are kept (lowest first)
    bool keep_all;// nothing skipped at this position
};

// Number of distances o in [0, T) whose column distance is <= x.
__device__ __forceinline__ int grid_count_le(int T, int stride, int x) {
    if (2 * x + 1 >= stride) return T;
    const int full = T / stride, rem = T - full * stride;
    const int hi_start = stride - x;                     // r >= stride - x  (and r > x here)
    const int part = min(rem, x + 1) + max(0, rem - hi_start);
    return full * (2 * x + 1) + part;
}

__device__ __forceinline__ ReqMask req_mask_setup(const MaskArgs& a, int seq_len, int prompt_len,
                                                  int max_seq_len) {
    ReqMask m;
    m.S = max(0, min(seq_len, max_seq_len));
    m.L_p = max(0, min(prompt_len, m.S));
    m.p = m.S - m.L_p;
    m.n_act = 0; m.dstar = -1; m.need = 0; m.keep_all = true; m.sel_k = -1;
    m.prefix = m.L_p; m.sink_end = m.L_p;
    if (a.mode == MODE_DENSE) {
        m.T = m.p - 1; m.n_win = m.p; m.w_lo = m.L_p;
        return m;
    }
    const int t = m.p - 1;
    m.T = min(t, a.window - 1);
    m.n_win = m.p > 0 ? m.T + 1 : 0;
    m.w_lo = m.S - m.n_win;
    m.sink_end = m.L_p + min(a.n_sink, m.p);
    m.prefix = min(m.sink_end, m.w_lo);
    if (a.mode == MODE_WINDOW || m.p == 0 || t < a.n_att - 1) return m;   // phase 1 / nothing to skip
    if (a.mode == MODE_LIST) {
        m.n_act = min(min(t - (a.n_att - 1), a.window - a.n_att), a.trace_len);
        m.keep_all = m.n_act <= 0;
        // phase 2 (t < N_r) with |skip_idx| < N_r - N_att: steps N_att-1 .. N_r-2 select entry t-(N_att-1)
        if (a.select && t <= a.window - 2 && t - (a.n_att - 1) < a.trace_len) m.sel_k = t - (a.n_att - 1);
        return m;
    }
    // GRID: keep the N_att - 1 best of [0, T) under (column distance, distance), plus T itself.
    m.keep_all = false;
    const int want = a.n_att - 1;
    if (want <= 0) { m.dstar = -1; m.need = 0; return m; }
    int lo = 0, hi = a.stride / 2;                       // smallest x with count_le(x) >= want
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (grid_count_le(m.T, a.stride, mid) >= want) hi = mid; else lo = mid + 1;
    }
    m.dstar = lo;
    m.need = want - (lo > 0 ? grid_count_le(m.T, a.stride, lo - 1) : 0);
    return m;
}

// LIST: set the bits of the active skip distances of one trace in a shared-memory bitmap
// (cleared by the caller).  Distances outside [0, window) are ignored.
template <int NT>
__device__ __forceinline__ void list_bitmap_fill(const MaskArgs& a, const ReqMask& m,
                                                 const int* trace, unsigned* bitmap) {
    for (int i = threadIdx.x; i < m.n_act; i += NT) {
        const int o = trace[i];
        if (o >= 0 && o < a.window) atomicOr(&bitmap[o >> 5], 1u << (o & 31));
    }
}

// LIST: which of the `slots` masks (one per head that shares this KV row) keep distance o.
template <int SLOTS>
__device__ __forceinline__ unsigned keep_bits(const MaskArgs& a, const ReqMask& m,
                                              const unsigned* bitmaps, int o) {
    constexpr unsigned ALL = (1u << SLOTS) - 1u;
    if (m.keep_all) return ALL;
    unsigned bits = 0;
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
        const unsigned w = bitmaps[s * a.bitmap_words + (o >> 5)];
        bits |= (((w >> (o & 31)) & 1u) ^ 1u) << s;
    }
    return bits;
}

// How the threads that build a list wait for each other: a whole block, or one warp.
struct BlockSync {
    __device__ static __forceinline__ void sync() { __syncthreads(); }
};
struct WarpSync {
    __device__ static __forceinline__ void sync() { __syncwarp(); }
};

// Exclusive scan of one int per thread over NT threads (threadIdx.x < NT, NT a multiple of 32).
template <int NT, class Sync>
__device__ __forceinline__ int block_excl_scan(int v, int& total, int* s_warp /* [NT/32] */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += n;
    }
    Sync::sync();                         // s_warp may still be read from a previous use
    if (lane == 31) s_warp[warp] = incl;
    Sync::sync();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) {
        const int c = s_warp[w];
        if (w < warp) base += c;
        tot += c;
    }
    total = tot;
    return base + incl - v;
}

// The kept positions are enumerated in two parts, both calling
//   sink(rank - r0, cache position, head bits)
// for the kept positions with union rank in [r0, r1).
//
// Part 1, "direct": the ranks whose position follows from the rank alone -- the prompt, the sinks
// that have left the window, and the whole window when nothing is skipped.  No scan, no barrier.
// Returns how many ranks of [r0, r1) it covered (they are the first ones of the split).
template <int NT, int SLOTS, class Sink>
__device__ __forceinline__ int enumerate_direct(const ReqMask& m, int r0, int r1, Sink sink) {
    constexpr unsigned ALL = (1u << SLOTS) - 1u;
    const int direct_end = m.keep_all ? m.prefix + m.n_win : m.prefix;
    const int hi = min(r1, direct_end);
    for (int r = r0 + (int)threadIdx.x; r < hi; r += NT)
        sink(r - r0, r < m.prefix ? r : m.w_lo + (r - m.prefix), ALL);
    return max(0, hi - r0);
}

// Part 2, "scanned": the window under a mask.  All NT threads must call it (it synchronises through
// Sync).  Returns the total number of kept positions of the request (direct ones included).
template <int NT, int SLOTS, class Sync, class Sink>
__device__ __forceinline__ int enumerate_scanned(const MaskArgs& a, const ReqMask& m,
                                                 const unsigned* bitmaps, int r0, int r1,
                                                 int* s_warp, Sink sink) {
    constexpr unsigned ALL = (1u << SLOTS) - 1u;
    if (m.keep_all) return m.prefix + m.n_win;
    // Each thread owns a contiguous run of window candidates (ascending position = descending
    // distance): count, scan, then emit.  The run is walked with the distance split as
    // o = k * stride + r kept up to date incrementally, so the GRID test needs no division.
    const int per = (m.n_win + NT - 1) / NT;
    const int c0 = min((int)threadIdx.x * per, m.n_win), c1 = min(c0 + per, m.n_win);
    const bool grid = a.mode == MODE_GRID;
    const int o_first = m.T - c0;
    const int k_first = grid ? o_first / a.stride : 0;
    const int r_first = grid ? o_first - k_first * a.stride : 0;
    auto bits_at = [&](int c, int o, int k, int r) -> unsigned {
        if (m.w_lo + c < m.sink_end) return ALL;        // a sink still inside the window is always kept
        if (grid) {
            if (o == m.T) return ALL;
            const int d = min(r, a.stride - r);
            if (d != m.dstar) return d < m.dstar ? ALL : 0u;
            const int rank = (m.dstar == 0 || 2 * m.dstar == a.stride) ? k : 2 * k + (r == m.dstar ? 0 : 1);
            return rank < m.need ? ALL : 0u;
        }
        return keep_bits<SLOTS>(a, m, bitmaps, o);
    };
    // Pass 1 counts and, for a single mask and a run of at most 32 candidates, remembers the
    // verdicts in a bit mask so that pass 2 only has to walk the set bits.
    const bool remember = SLOTS == 1 && per <= 32;
    unsigned verdicts = 0u;
    int cnt = 0;
    {
        int o = o_first, k = k_first, r = r_first;
        for (int c = c0; c < c1; ++c) {
            const bool keep = bits_at(c, o, k, r) != 0u;
            cnt += keep;
            if (remember && keep) verdicts |= 1u << (c - c0);
            --o;
            if (--r < 0) { r = a.stride - 1; --k; }
        }
    }
    int total;
    int rank = m.prefix + block_excl_scan<NT, Sync>(cnt, total, s_warp);
    if (rank < r1 && rank + cnt > r0) {
        if (remember) {
            while (verdicts) {
                const int j = __ffs(verdicts) - 1;
                verdicts &= verdicts - 1u;
                if (rank >= r0 && rank < r1) sink(rank - r0, m.w_lo + c0 + j, ALL);
                ++rank;
            }
        } else {
            int o = o_first, k = k_first, r = r_first;
            for (int c = c0; c < c1; ++c) {
                const unsigned bits = bits_at(c, o, k, r);
                if (bits) {
                    if (rank >= r0 && rank < r1) sink(rank - r0, m.w_lo + c, bits);
                    ++rank;
                }
                --o;
                if (--r < 0) { r = a.stride - 1; --k; }
            }
        }
    }
    return m.prefix + total;
}

}  // namespace dsa
