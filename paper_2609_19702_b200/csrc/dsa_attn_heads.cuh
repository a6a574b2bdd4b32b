// Split-KV decode attention for bf16 caches under PER-HEAD skip lists (the paper's own setting: every
// attention head selects its own diagonals, Section 4), with or without the fused phase-2 selection.
//
// What the heads of a request share although their masks differ: its lengths and mask constants,
// the rows that are always kept (prompt, sinks that left the window) and WHERE every window
// candidate lives (ring slot, block-table entry).  A block of W warps works that out once, with all
// its threads:
//   diroff[r]   byte offset of always-kept row r (kv head 0)            r in [0, prefix)
//   winoff[c]   byte offset of window candidate c = position w_lo + c    c in [0, n_win)
// What differs per head is only WHICH candidates it keeps, and that is cheap to derive from the
// head's skip trace without touching global memory again: the trace goes into a bitmap over window
// distances (16 distances per 32-bit word, so that the shared-memory atomics of a warp spread over
// twice as many words), and the kept candidates are enumerated 16 distances per lane (mask,
// popcount, one suffix scan across the warp, a handful of stores; where the caller also keeps the lists
// as bitmaps, MaskArgs::skip_bitmap, the head's row is copied instead of scattered) into
//   kidx[j]     candidate index of the j-th kept window row, ascending   (16 bits per row)
//   hbits[j]    which query heads of the group keep it                   (grouped queries only)
// Every warp streams U heads back to back through one ring that never drains in between: while the
// tiles of head u are in flight it builds kidx of head u + 1 into its second buffer; once the last
// tile of head u has been issued it turns that into woff[j] = winoff[kidx[j]], the byte offsets the
// copies are issued from (one shared-memory read per row, as in the other kernels: a second
// indirection on that path measured 15 % slower), and the first tiles of head u + 1 go into the slots
// that the last tiles of head u free.  Tile consumption is the tensor-core formulation of
// dsa_attn_mma.cuh; the selection candidates are tracked on the score fragment as there.
#pragma once
#include "dsa_attn_mma.cuh"

namespace dsa {

template <int D, int G, int STAGES, int W, bool HEADMASK>
struct HeadsCfg {
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int CPR = ROW_BYTES / 16;
    static constexpr int TILE_BYTES = MMA_KEYS * ROW_BYTES;
    static constexpr int SLOT_BYTES = 2 * TILE_BYTES;
    static constexpr int KSTEPS = D / 16;
    static constexpr int MTILES = D / 16;
    static constexpr int SLOTS = HEADMASK ? G : 1;
    __host__ __device__ static constexpr int align16(int x) { return (x + 15) / 16 * 16; }
    // one warp's private area: woff, two (kidx, hbits) buffers and its bitmaps
    __host__ __device__ static constexpr int kidx_bytes(int kcap) { return align16(kcap * 2) + (HEADMASK ? align16(kcap) : 0); }
    __host__ __device__ static constexpr int warp_bytes(int kcap, int words) {
        return kcap * 8 + 2 * kidx_bytes(kcap) + align16(SLOTS * 2 * words * 4);     // (bitmaps: 16 distances per word)
    }
    // dynamic shared memory: [W rings][diroff][winoff][W private areas]
    __host__ static size_t smem_bytes(int dir_cap, int window, int kcap, int words) {
        return (size_t)W * STAGES * SLOT_BYTES + (size_t)dir_cap * 8 + (size_t)window * 8 + (size_t)W * warp_bytes(kcap, words);
    }
};

// EARLY: the caller has promised that the launch before this one does not write the lengths, the block
// table or the skip lists (AttnArgs::early_list): the shared tables and the first head's kept rows are
// worked out before waiting for that launch; q, the new rows and the caches are touched after.
template <int D, int G, int STAGES, int W, bool HEADMASK, bool SELECT, bool APPEND, bool EARLY = false>
__global__ void __launch_bounds__(32 * W) dsa_attn_heads_kernel(const AttnArgs a) {
    using C = HeadsCfg<D, G, STAGES, W, HEADMASK>;
    using T = __nv_bfloat16;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr unsigned ALL = (1u << C::SLOTS) - 1u;
    constexpr int NTHR = 32 * W;

    asm volatile("griddepcontrol.launch_dependents;");
    if constexpr (!EARLY) asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* ring = smem + warp * (STAGES * C::SLOT_BYTES);
    int64_t* diroff = reinterpret_cast<int64_t*>(smem + W * STAGES * C::SLOT_BYTES);
    int64_t* winoff = diroff + a.dir_cap;
    unsigned char* mine = reinterpret_cast<unsigned char*>(winoff + a.mask.window) +
                          warp * C::warp_bytes(a.kidx_cap, a.mask.bitmap_words);
    const int kbuf_bytes = C::kidx_bytes(a.kidx_cap);
    int64_t* woff = reinterpret_cast<int64_t*>(mine);                 // byte offsets of the kept window rows of the head being issued
    unsigned char* kmem = mine + (size_t)a.kidx_cap * 8;
    unsigned* bitmaps = reinterpret_cast<unsigned*>(kmem + 2 * kbuf_bytes);
    auto kidx_of = [&](int buf) { return reinterpret_cast<unsigned short*>(kmem + buf * kbuf_bytes); };
    auto hbits_of = [&](int buf) { return kmem + buf * kbuf_bytes + C::align16(a.kidx_cap * 2); };
    const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.k);
    const unsigned char* vbase = reinterpret_cast<const unsigned char*>(a.v);

    const int U = a.heads_per_warp;
    const int hblocks = a.H_kv / (W * U);
    const int hb = blockIdx.x % hblocks;
    const int split = (blockIdx.x / hblocks) % a.n_split;
    const int b = blockIdx.x / (hblocks * a.n_split);
    const int kvh0 = hb * W * U + warp;               // this warp's heads: kvh0, kvh0 + W, ...

    const int seq_raw = a.seq_len[b], prompt_raw = req_prompt_len(a, b);
    const int hq = lane >> 2, qd = (lane & 3) * 2;
    unsigned qb[C::KSTEPS][2], qn[C::KSTEPS][2];
    auto load_q = [&](int kvh, unsigned (&dst)[C::KSTEPS][2]) {
        const T* qrow = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.H_q + kvh * G + (hq < G ? hq : 0)) * D;
#pragma unroll
        for (int kk = 0; kk < C::KSTEPS; ++kk) {
            const unsigned q0 = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd);
            const unsigned q1 = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd + 8);
            dst[kk][0] = hq < G ? q0 : 0u;
            dst[kk][1] = hq < G ? q1 : 0u;
        }
    };
    if constexpr (!EARLY) load_q(kvh0, qb);

    bool has_new = false;
    const int S_step = APPEND ? step_seq_len(a, seq_raw, has_new) : seq_raw;
    const ReqMask m = req_mask_setup(a.mask, S_step, prompt_raw, a.max_seq_len);
    const int64_t head_stride_bytes = a.stride_head * 2;
    const int prefix = min(m.prefix, a.dir_cap);      // always-kept rows (ranks [0, prefix) are their positions)
    const int n_win = min(m.n_win, a.mask.window);
    const int r_lo = split * a.chunk;                 // ranks [r_lo, r_lo + chunk) of the kept sequence are this split's rows

    // fused step: the token being decoded goes from k_new / v_new to the cache (split 0), per head
    auto store_new = [&]() {
        if (APPEND && has_new && split == 0 && lane < 2 * C::CPR) {
            const int64_t new_off = token_offset(a, b, m.L_p, m.S - 1) * 2;
            const bool is_k = lane < C::CPR;
            const int c = is_k ? lane : lane - C::CPR;
            const unsigned char* src0 = reinterpret_cast<const unsigned char*>(is_k ? a.k_new : a.v_new) + c * 16;
            unsigned char* dst0 = const_cast<unsigned char*>(is_k ? kbase : vbase) + new_off + c * 16;
            for (int u = 0; u < U; ++u) {
                const int kvh = kvh0 + u * W;
                *reinterpret_cast<uint4*>(dst0 + kvh * head_stride_bytes) =
                    *reinterpret_cast<const uint4*>(src0 + ((int64_t)b * a.H_kv + kvh) * C::ROW_BYTES);
            }
        }
    };
    if constexpr (!EARLY) store_new();

    // ---- shared by all heads of the block: where the always-kept rows and the window candidates live
    for (int r = threadIdx.x; r < prefix; r += NTHR)
        diroff[r] = token_offset(a, b, m.L_p, r) * 2;           // (prompt, then the old sinks: positions = ranks)
    __syncthreads();

    // ---- per head: which window candidates it keeps ------------------------------------------------
    // kept rows of a head, in ascending position: ranks [0, prefix) the always-kept rows, then its kept
    // window candidates.  Returns the number of those (all of them, whatever the split).
    const int words = 2 * a.mask.bitmap_words;                      // 16 distances per word
    const int n_sink_win = max(0, m.sink_end - m.w_lo);            // sinks still inside the window: candidates [0, n_sink_win)
    // The first PRE x 32 active trace entries of a head's first mask travel in registers: they are
    // fetched a whole head ahead (while the head before streams), so that their latency is off the path.
    constexpr int PRE = 12;
    auto trace_of = [&](int kvh, int s) {
        const int h = kvh * G + s;
        const int mh = a.mask.mask_heads == 1 ? 0 : (a.mask.mask_heads == a.H_kv ? kvh : h);
        return a.mask.skip_offsets + ((int64_t)b * a.mask.mask_heads + mh) * a.mask.trace_len;
    };
    // the same head's row of the caller's bitmap form of the lists (MaskArgs::skip_bitmap), if there is one
    auto bitmap_of = [&](int kvh, int s) {
        const int h = kvh * G + s;
        const int mh = a.mask.mask_heads == 1 ? 0 : (a.mask.mask_heads == a.H_kv ? kvh : h);
        return a.mask.skip_bitmap + ((int64_t)b * a.mask.mask_heads + mh) * a.mask.bitmap_words;
    };
    auto prefetch_trace = [&](int kvh, int (&pre)[PRE]) {
        if (a.mask.skip_bitmap) {                       // (then the words of the bitmap travel instead of list entries)
            const unsigned* src = bitmap_of(kvh, 0);
#pragma unroll
            for (int k = 0; k < PRE; ++k) {
                const int i = k * 32 + lane;
                pre[k] = (!m.keep_all && i < a.mask.bitmap_words) ? (int)src[i] : 0;
            }
            return;
        }
        const int* trace = trace_of(kvh, 0);
#pragma unroll
        for (int k = 0; k < PRE; ++k) {
            const int i = k * 32 + lane;
            pre[k] = (!m.keep_all && i < m.n_act) ? trace[i] : -1;
        }
    };
    auto build_kidx = [&](int kvh, int buf, const int (&pre)[PRE]) -> int {
        unsigned short* kidx = kidx_of(buf);
        unsigned char* hbits = hbits_of(buf);
        __syncwarp();
        if (!m.keep_all && a.mask.skip_bitmap) {
            // The caller keeps the lists as bitmaps, 32 distances per word: split every word into the two
            // 16-distance words of the layout used here.  Nothing to scatter, no atomics.
#pragma unroll
            for (int s = 0; s < C::SLOTS; ++s) {
                const unsigned* src = bitmap_of(kvh, s);
                for (int i0 = 0; i0 < a.mask.bitmap_words; i0 += 32) {
                    const int i = i0 + lane;
                    if (i < a.mask.bitmap_words) {
                        unsigned wd = 0u;
                        bool have = false;
                        if (s == 0) {
#pragma unroll
                            for (int k = 0; k < PRE; ++k)
                                if (i0 == k * 32) { wd = (unsigned)pre[k]; have = true; }
                        }
                        if (!have) wd = src[i];
                        bitmaps[s * words + 2 * i] = wd & 0xffffu;
                        bitmaps[s * words + 2 * i + 1] = wd >> 16;
                    }
                }
            }
            __syncwarp();
        } else if (!m.keep_all) {
            for (int i = lane; i < C::SLOTS * words; i += 32) bitmaps[i] = 0u;
            __syncwarp();
            auto mark = [&](int s, int o) {
                if (o >= 0 && o < a.mask.window) atomicOr(&bitmaps[s * words + (o >> 4)], 1u << (o & 15));
            };
#pragma unroll
            for (int k = 0; k < PRE; ++k) mark(0, pre[k]);
#pragma unroll
            for (int s = 0; s < C::SLOTS; ++s) {
                const int* trace = trace_of(kvh, s);
                // the rest, eight entries per lane at a time (the loads of a batch are in flight together)
                for (int i0 = s == 0 ? PRE * 32 : 0; i0 < m.n_act; i0 += 256) {
                    int o[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int i = i0 + k * 32 + lane;
                        o[k] = i < m.n_act ? trace[i] : -1;
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) mark(s, o[k]);
                }
            }
            __syncwarp();
        }
        // 16 distances per lane and round, the highest distances (= the oldest positions) first
        const int n_half = (n_win + 15) >> 4;
        int rank = 0;
        for (int base = ((n_half + 31) >> 5) * 32 - 32; base >= 0; base -= 32) {
            const int hw = base + lane;
            const int o_lo = hw * 16;
            unsigned valid = 0u;                                       // distances o_lo .. o_lo + 15 that exist (o <= T)
            if (o_lo <= m.T) valid = (m.T - o_lo >= 15) ? 0xffffu : ((1u << (m.T - o_lo + 1)) - 1u);
            unsigned sink = 0u;                                        // candidates below n_sink_win: distances above T - n_sink_win
            if (n_sink_win > 0) {
                const int lo = m.T - n_sink_win + 1;                   // first such distance
                if (lo <= o_lo) sink = 0xffffu;
                else if (lo <= o_lo + 15) sink = (0xffffu << (lo - o_lo)) & 0xffffu;
            }
            unsigned keep[C::SLOTS];
            unsigned uni = 0u;
#pragma unroll
            for (int s = 0; s < C::SLOTS; ++s) {
                unsigned skip = 0u;
                if (!m.keep_all && valid) skip = bitmaps[s * words + hw] & 0xffffu;
                keep[s] = (~skip | sink) & valid;
                uni |= keep[s];
            }
            const int cnt = __popc(uni);
            // ranks ascend with the position, i.e. descend with the distance: suffix sum over the lanes
            int incl = cnt;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int n = __shfl_down_sync(FULL, incl, off);
                if (lane + off < 32) incl += n;
            }
            int r = rank + incl - cnt;                                  // rank of this lane's highest kept distance
            rank += __shfl_sync(FULL, incl, 0);
            unsigned bitsleft = uni;
            while (bitsleft) {
                const int bit = 31 - __clz(bitsleft);
                bitsleft &= ~(1u << bit);
                if (r < a.kidx_cap) {
                    kidx[r] = (unsigned short)(m.T - (o_lo + bit));
                    if (HEADMASK) {
                        unsigned hbv = 0u;
#pragma unroll
                        for (int s = 0; s < C::SLOTS; ++s) hbv |= ((keep[s] >> bit) & 1u) << s;
                        hbits[r] = (unsigned char)hbv;
                    }
                }
                ++r;
            }
        }
        __syncwarp();
        return min(rank, a.kidx_cap);
    };

    // ---- staging --------------------------------------------------------------------------------
    // tile `tile` of head kvh (whose kept window rows are in woff): rows [16 tile, 16 tile + 16) of the split
    auto issue_tile = [&](int kvh, int tile, int slot, int n_rows, int new_r) {
        const int64_t head_bytes = kvh * head_stride_bytes;
        const int64_t knew_off = APPEND ? (reinterpret_cast<const unsigned char*>(a.k_new) - kbase) +
                                              ((int64_t)b * a.H_kv + kvh) * C::ROW_BYTES : 0;
        const int64_t vnew_off = APPEND ? (reinterpret_cast<const unsigned char*>(a.v_new) - vbase) +
                                              ((int64_t)b * a.H_kv + kvh) * C::ROW_BYTES : 0;
        unsigned char* ks = ring + slot * C::SLOT_BYTES;
        unsigned char* vs = ks + C::TILE_BYTES;
        const int row0 = tile * MMA_KEYS;
#pragma unroll
        for (int i = 0; i < MMA_KEYS * C::CPR / 32; ++i) {
            const int idx = i * 32 + lane;
            const int row = idx / C::CPR, c = idx % C::CPR;
            const int r = row0 + row;
            const bool valid = r < n_rows;
            const int dst = row * C::ROW_BYTES + ((c ^ (row & 7)) * 16);
            const int rg = r_lo + r;
            const int64_t* src = rg < prefix ? diroff + rg : woff + (rg - prefix);
            const int64_t off = valid ? *src + head_bytes + c * 16 : 0;
            const bool is_new = APPEND && r == new_r;    // (not in the cache yet: read it where the caller put it)
            cp_async16(ks + dst, kbase + (is_new ? knew_off + c * 16 : off), valid);
            cp_async16(vs + dst, vbase + (is_new ? vnew_off + c * 16 : off), valid);
        }
    };

    // The always-kept rows are the same for every head: the first tiles of the first head can be issued
    // before anything else is known, so that memory is streaming while the window table is built.
    int islot = 0;
    int inflight = 0;                                 // tiles issued and not yet consumed (one commit group each)
    const int dir_rows = max(0, min(prefix - r_lo, a.chunk));         // rows of this split that are always-kept rows
    int n_early = 0;
    {
        const int whole = dir_rows / MMA_KEYS;
        n_early = EARLY ? 0 : min(STAGES - 1, whole);       // (no cache reads before the wait)
        for (int s = 0; s < n_early; ++s) {
            issue_tile(kvh0, s, islot, dir_rows, -1);
            cp_async_commit();
            islot = islot + 1 == STAGES ? 0 : islot + 1;
            ++inflight;
        }
    }
    for (int c = threadIdx.x; c < n_win; c += NTHR) winoff[c] = token_offset(a, b, m.L_p, m.w_lo + c) * 2;
    __syncthreads();                                  // the last block barrier: from here on warps run free

    // rows of a head in this split, given how many window candidates it keeps
    auto rows_of = [&](int n_kept) { return max(0, min(prefix + n_kept - r_lo, a.chunk)); };
    // the token being decoded is candidate n_win - 1; kept positions ascend, so it can only be the head's last row
    auto new_row_of = [&](int buf, int n_kept, int n_rows) {
        if (!(APPEND && has_new) || n_kept <= 0) return -1;
        if (kidx_of(buf)[n_kept - 1] != (unsigned short)(n_win - 1)) return -1;
        const int r = prefix + n_kept - 1 - r_lo;     // its row in this split
        return (r >= 0 && r < n_rows) ? r : -1;
    };

    // kidx of a head -> woff (all lanes; the previous head's tiles have all been issued by then)
    auto convert = [&](int buf, int n_kept) {
        const unsigned short* kidx = kidx_of(buf);
        __syncwarp();
        for (int j = lane; j < n_kept; j += 32) woff[j] = winoff[kidx[j]];
        __syncwarp();
    };

    int cur_buf = 0;
    int pre[PRE];
    prefetch_trace(kvh0, pre);
    int cur_kept = build_kidx(kvh0, 0, pre);
    if (U > 1) prefetch_trace(kvh0 + W, pre);
    convert(0, cur_kept);
    if constexpr (EARLY) {                            // the first head's rows are known: now wait for the kernel before this one
        asm volatile("griddepcontrol.wait;" ::: "memory");
        load_q(kvh0, qb);
        store_new();
    }
    int cur_rows = rows_of(cur_kept);
    int cur_new = new_row_of(0, cur_kept, cur_rows);
    int cur_tiles = (cur_rows + MMA_KEYS - 1) / MMA_KEYS;
    int cur_issued = min(n_early, cur_tiles);         // (the early tiles were whole tiles of always-kept rows)
    int nxt_kvh = kvh0, nxt_rows = 0, nxt_tiles = 0, nxt_issued = 0, nxt_new = -1, nxt_kept = 0;
    bool nxt_valid = false, nxt_converted = false;

    // One ring step on the producer side, if a slot is free and a tile is known: the next tile of the
    // current head, else of the next one once its kept rows have been worked out.  Heads differ in
    // length and the next one is not always known yet, so no empty groups keep a fixed count here:
    // every commit group is a real tile, `inflight` counts them, and the consumer waits for
    // "all but the inflight - 1 newest groups", i.e. for its own tile.
    int cur_kvh = kvh0;
    auto try_issue = [&]() -> bool {
        if (inflight >= STAGES) return false;
        if (cur_issued < cur_tiles) {
            issue_tile(cur_kvh, cur_issued, islot, cur_rows, cur_new);
            ++cur_issued;
        } else if (nxt_valid && nxt_issued < nxt_tiles) {
            if (!nxt_converted) { convert(cur_buf ^ 1, nxt_kept); nxt_converted = true; }
            issue_tile(nxt_kvh, nxt_issued, islot, nxt_rows, nxt_new);
            ++nxt_issued;
        } else {
            return false;
        }
        cp_async_commit();
        islot = islot + 1 == STAGES ? 0 : islot + 1;
        ++inflight;
        return true;
    };
    while (inflight < STAGES - 1 && try_issue()) {}

    const int hc = (lane & 3) * 2, kr = lane >> 2;
    const int lm_row_k = (lane & 7) + ((lane >> 3) & 1) * 8, lm_chk_k = lane >> 4;
    const int lm_row_v = (lane & 7) + (lane >> 4) * 8, lm_chk_v = (lane >> 3) & 1;
    // Selection candidates are the kept decode keys that are no sinks.  Kept rows ascend in position, the
    // always-kept rows come first and the sinks still inside the window are the first window rows (all
    // kept), so "candidate" is a threshold on the row's rank, and the oldest of equal logits is the lowest
    // rank: the tile loop tracks ranks and only the winner is turned into a position.
    const int cand_row = prefix + min(max(0, m.L_p + a.mask.n_sink - m.w_lo), n_win);
    int cslot = 0;

#pragma unroll 1
    for (int u = 0; u < U; ++u) {
        const int kvh = kvh0 + u * W;
        cur_kvh = kvh;
        // the ring holds the first tiles of this head: work out the next head's rows while they fly.  No
        // tile is being consumed meanwhile, so the slot the last head's last tile has just left can fly too.
        nxt_valid = false;                              // (nothing of the next head is known yet)
        if (u + 1 < U) { while (inflight < STAGES && try_issue()) {} }
        nxt_valid = u + 1 < U;
        if (nxt_valid) {
            nxt_kvh = kvh + W;
            load_q(nxt_kvh, qn);
            nxt_kept = build_kidx(nxt_kvh, cur_buf ^ 1, pre);
            if (u + 2 < U) prefetch_trace(nxt_kvh + W, pre);        // (used a head from now)
            nxt_rows = rows_of(nxt_kept);
            nxt_new = new_row_of(cur_buf ^ 1, nxt_kept, nxt_rows);
            nxt_tiles = (nxt_rows + MMA_KEYS - 1) / MMA_KEYS;
            nxt_issued = 0;
            nxt_converted = false;
            while (inflight < STAGES - 1 && try_issue()) {}      // (a short head leaves room for the next one's tiles)
        }
        const unsigned short* kidx = kidx_of(cur_buf);
        const unsigned char* hbits = hbits_of(cur_buf);
        const int n_rows = cur_rows;

        float o[C::MTILES][4];
#pragma unroll
        for (int mt = 0; mt < C::MTILES; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
        float mrun[2] = {-INFINITY, -INFINITY}, lpart[2] = {0.f, 0.f};
        float bestv[2] = {INFINITY, INFINITY};
        int bestp[2] = {0x7fffffff, 0x7fffffff};

        for (int tile = 0; tile < cur_tiles; ++tile) {
            cp_async_wait_upto<STAGES - 2>(inflight - 1);   // the oldest tile in flight has landed (for this lane)
            __syncwarp();                                   // ... for every lane; the slot consumed last is free
            try_issue();
            const unsigned char* ks = ring + cslot * C::SLOT_BYTES;
            const unsigned char* vs = ks + C::TILE_BYTES;
            cslot = cslot + 1 == STAGES ? 0 : cslot + 1;

            float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kk = 0; kk < C::KSTEPS; ++kk) {
                unsigned af[4];
                const int chunk = kk * 2 + lm_chk_k;
                ldmatrix_x4(af, ks + lm_row_k * C::ROW_BYTES + ((chunk ^ (lm_row_k & 7)) * 16));
                mma_bf16_16816(s, af, qb[kk][0], qb[kk][1]);
            }
            const int r0 = tile * MMA_KEYS + kr, r1 = r0 + 8;
            const bool v0 = r0 < n_rows, v1 = r1 < n_rows;
            const int g0 = r_lo + r0 - prefix, g1 = r_lo + r1 - prefix;     // index among the kept window rows (< 0: always-kept row)
            unsigned bits0 = ALL, bits1 = ALL;
            if (HEADMASK) {
                bits0 = v0 ? (g0 < 0 ? ALL : (unsigned)hbits[g0]) : 0u;
                bits1 = v1 ? (g1 < 0 ? ALL : (unsigned)hbits[g1]) : 0u;
            }
            const int pos0 = r_lo + r0, pos1 = r_lo + r1;      // (ranks; see cand_row)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const bool on0 = v0 && (!HEADMASK || ((bits0 >> (hc + j)) & 1u));
                const bool on1 = v1 && (!HEADMASK || ((bits1 >> (hc + j)) & 1u));
                float x0 = on0 ? s[j] * a.scale_log2 : -INFINITY;
                float x1 = on1 ? s[2 + j] * a.scale_log2 : -INFINITY;
                if (SELECT) {
                    // keys arrive in ascending position: a strict "<" keeps the oldest of equal logits
                    if (on0 && pos0 >= cand_row && x0 < bestv[j]) { bestv[j] = x0; bestp[j] = pos0; }
                    if (on1 && pos1 >= cand_row && x1 < bestv[j]) { bestv[j] = x1; bestp[j] = pos1; }
                }
                float mx = fmaxf(x0, x1);
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 16));
                const float mnew = fmaxf(mrun[j], mx);
                const float msafe = mnew == -INFINITY ? 0.f : mnew;
                const float corr = fast_exp2(mrun[j] - msafe);
                x0 = fast_exp2(x0 - msafe);
                x1 = fast_exp2(x1 - msafe);
                lpart[j] = lpart[j] * corr + x0 + x1;
                mrun[j] = mnew;
                s[j] = x0; s[2 + j] = x1;
                if (corr != 1.f) {
#pragma unroll
                    for (int mt = 0; mt < C::MTILES; ++mt) { o[mt][j] *= corr; o[mt][2 + j] *= corr; }
                }
            }
            const unsigned pb0 = movmatrix_trans(pack_bf16x2(s[0], s[1]));
            const unsigned pb1 = movmatrix_trans(pack_bf16x2(s[2], s[3]));
#pragma unroll
            for (int mt = 0; mt < C::MTILES; ++mt) {
                unsigned af[4];
                const int chunk = mt * 2 + lm_chk_v;
                ldmatrix_x4_trans(af, vs + lm_row_v * C::ROW_BYTES + ((chunk ^ (lm_row_v & 7)) * 16));
                mma_bf16_16816(o[mt], af, pb0, pb1);
            }
            --inflight;
        }

        // ---- this head is done: sums over the key lanes, normalise, write ----------------------------
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            float l = lpart[j];
            l += __shfl_xor_sync(FULL, l, 4);
            l += __shfl_xor_sync(FULL, l, 8);
            l += __shfl_xor_sync(FULL, l, 16);
            float bv = bestv[j];
            int bp = bestp[j];
            if (SELECT) {
#pragma unroll
                for (int off = 4; off <= 16; off <<= 1) {
                    const float ov = __shfl_xor_sync(FULL, bv, off);
                    const int op = __shfl_xor_sync(FULL, bp, off);
                    if (ov < bv || (ov == bv && op < bp)) { bv = ov; bp = op; }
                }
            }
            const int h = hc + j;
            if (h < G) {
                const float inv = l > 0.f ? 1.f / l : 0.f;
                const float lse = l > 0.f ? (mrun[j] + log2f(l)) * LN2 : -INFINITY;
                const int64_t row = (int64_t)b * a.H_q + kvh * G + h;
#pragma unroll
                for (int mt = 0; mt < C::MTILES; ++mt) {
                    const int d0 = mt * 16 + kr;
                    if (a.n_split > 1) {
                        float* dst = a.out_part + (row * a.n_split + split) * D;
                        dst[d0] = o[mt][j] * inv;
                        dst[d0 + 8] = o[mt][2 + j] * inv;
                    } else {
                        T* dst = reinterpret_cast<T*>(a.out) + row * D;
                        dst[d0] = __float2bfloat16_rn(o[mt][j] * inv);
                        dst[d0 + 8] = __float2bfloat16_rn(o[mt][2 + j] * inv);
                    }
                }
                if (kr == 0) {
                    if (a.n_split > 1) a.lse_part[row * a.n_split + split] = lse;
                    else a.lse[row] = lse;
                    if (SELECT) {
                        // (rank -> position: a candidate is a window row)
                        const int off = bp == 0x7fffffff ? -1 : (m.S - 1) - (m.w_lo + (int)kidx[bp - prefix]);
                        if (a.n_split > 1) {
                            a.sel_val_part[row * a.n_split + split] = bv;
                            a.sel_off_part[row * a.n_split + split] = off;
                            a.sel_k[row] = m.sel_k;
                        } else if (m.sel_k >= 0) {
                            record_selection(a.mask, row, m.sel_k, off);
                        }
                    }
                }
            }
        }
        if (nxt_valid) {
#pragma unroll
            for (int kk = 0; kk < C::KSTEPS; ++kk) { qb[kk][0] = qn[kk][0]; qb[kk][1] = qn[kk][1]; }
            if (!nxt_converted) convert(cur_buf ^ 1, nxt_kept);        // (a head without tiles in between)
            cur_buf ^= 1;
            cur_rows = nxt_rows; cur_tiles = nxt_tiles; cur_issued = nxt_issued; cur_new = nxt_new;
        }
    }
    cp_async_wait<0>();
}

}  // namespace dsa
