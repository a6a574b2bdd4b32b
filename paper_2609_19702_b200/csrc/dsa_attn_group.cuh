// Split-KV decode attention for bf16 caches, head-group form: ONE row list per (request, split),
// built once by a whole block and used for W x U kv heads.
//
// Why: which rows a request keeps does not depend on the head whenever the mask does not (dense,
// window, grid, one shared skip list), yet the one-warp-per-item kernel (dsa_attn_mma.cuh) rebuilds
// the list for every pair of heads: lengths, mask constants, window scan, block-table lookups.  At
// ~400 kept rows that is a fifth of a warp's cycles; for the ~100-row items of a decode loop at the
// paper's shape (50 prompt tokens + N_att 52) it is as long as the streaming itself.  Here a block
// of W warps builds the list once with all its threads and every warp then streams U heads through
// it back to back: head kvh0 + u W of warp w's ring follows head kvh0 + (u - 1) W without the ring
// draining in between (the first tiles of the next head are issued into the slots that the last
// tiles of the current one free; its q is fetched a head ahead).  The W warps of a block read the
// same tokens of W neighbouring heads at the same time, i.e. neighbouring memory.
//
// Row-list entries are the 64-bit byte offsets of the rows of kv head 0 (a head adds its own offset
// when it issues a tile), so one list of up to 2048 rows costs 16 KB per block whatever W and U
// are.  Tile consumption is the tensor-core formulation of
// dsa_attn_mma.cuh: S^T = K . Q^T, online softmax on the accumulator fragment, O^T += V^T . P^T.
#pragma once
#include "dsa_attn_mma.cuh"

namespace dsa {

constexpr int GROUP_MAX_CHUNK = 2048;           // rows one shared list can hold

template <int D, int W, int STAGES>
struct GroupCfg {
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int CPR = ROW_BYTES / 16;
    static constexpr int TILE_BYTES = MMA_KEYS * ROW_BYTES;
    static constexpr int SLOT_BYTES = 2 * TILE_BYTES;
    static constexpr int KSTEPS = D / 16;
    static constexpr int MTILES = D / 16;
    // dynamic shared memory: [W rings][row list][one bitmap]
    __host__ static size_t smem_bytes(int chunk, int bitmap_words) {
        return (size_t)W * STAGES * SLOT_BYTES + (size_t)chunk * 8 + (size_t)bitmap_words * 4;
    }
};

// EARLY: the caller has promised that the launch before this one does not write the arrays the row
// list is made from (AttnArgs::early_list), so the list is built before waiting for that launch.
// COPY_ONLY: a measuring form (dsa_debug_copy_only): the same lists, the same copies into the same rings,
// but a landed tile is only read once and folded, no arithmetic; what it writes to out / lse is meaningless.
// Its time is what this launch's staging alone costs: the kernel's own speed of light.
template <int D, int G, int STAGES, int W, bool APPEND, bool EARLY = false, bool COPY_ONLY = false>
__global__ void __launch_bounds__(32 * W) dsa_attn_group_kernel(const AttnArgs a) {
    using C = GroupCfg<D, W, STAGES>;
    using IC = MmaItemCfg<D, G, false, false>;
    using T = __nv_bfloat16;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int NTHR = 32 * W;

    // may be scheduled early behind the previous kernel of the stream, and lets the next one in early
    asm volatile("griddepcontrol.launch_dependents;");
    constexpr bool early = EARLY;
    if constexpr (!EARLY) asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_warp[W];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* ring = smem + warp * (STAGES * C::SLOT_BYTES);
    int64_t* rowoff = reinterpret_cast<int64_t*>(smem + W * STAGES * C::SLOT_BYTES);   // bytes, kv head 0
    unsigned* bitmap = reinterpret_cast<unsigned*>(rowoff + a.chunk);
    const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.k);
    const unsigned char* vbase = reinterpret_cast<const unsigned char*>(a.v);

    // block -> (request, split, block of W x U heads); head blocks vary fastest, so blocks that run
    // together read the same tokens
    const int U = a.heads_per_warp;
    const int hblocks = a.H_kv / (W * U);
    const int hb = blockIdx.x % hblocks;
    const int split = (blockIdx.x / hblocks) % a.n_split;
    const int b = blockIdx.x / (hblocks * a.n_split);
    const int kvh0 = hb * W * U + warp;               // this warp's heads: kvh0, kvh0 + W, ...

    const int seq_raw = a.seq_len[b], prompt_raw = req_prompt_len(a, b);
    // Q^T fragment of the first head (see dsa_attn_mma.cuh); loaded first, used last
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

    // fused step: the token being decoded goes from k_new / v_new to the cache (split 0 only; nobody
    // reads that slot in this launch), for each of this warp's heads
    int64_t new_off = 0;
    int new_r = -1;
    if (APPEND && has_new) new_off = token_offset(a, b, m.L_p, m.S - 1) * 2;
    auto store_new = [&]() {
        if (APPEND && has_new && split == 0 && lane < 2 * C::CPR) {
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

    // ---- staging --------------------------------------------------------------------------------
    // tile `tile` of head u (rows [16 tile, 16 tile + 16) of the list, of which rows_ready exist)
    auto issue_tile = [&](int u, int tile, int slot, int rows_ready) {
        const int kvh = kvh0 + u * W;
        const int64_t head_bytes = kvh * head_stride_bytes;
        // fused step: the rows of the token being decoded, as offsets from the cache bases
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
            const bool valid = r < rows_ready;
            const int dst = row * C::ROW_BYTES + ((c ^ (row & 7)) * 16);
            const int64_t off = valid ? rowoff[r] + head_bytes + c * 16 : 0;
            const bool is_new = APPEND && r == new_r;   // (not in the cache yet: read it where the caller put it)
            cp_async16(ks + dst, kbase + (is_new ? knew_off + c * 16 : off), valid);
            cp_async16(vs + dst, vbase + (is_new ? vnew_off + c * 16 : off), valid);
        }
    };

    // ---- the row list, once for all heads of the block --------------------------------------------
    // Phase A: rows that need no scan (prompt, old sinks, an unmasked window); the first tiles of the
    // first head are issued from them right away, so that memory is already streaming while phase B
    // (mask bitmap, window scan, block-table lookups) is computed.
    const int r_lo = split * a.chunk, r_hi = r_lo + a.chunk;
    const int n_direct = enumerate_direct<NTHR, 1>(m, r_lo, r_hi, [&](int slot, int pos, unsigned) {
        rowoff[slot] = token_offset(a, b, m.L_p, pos) * 2;
    });
    __syncthreads();
    int islot = 0;                                    // ring slot of the next issue
    int i_u = 0, i_t = 0;                             // next tile to issue: head i_u, tile i_t
    {
        const int whole_a = (n_direct - (APPEND ? 1 : 0)) / MMA_KEYS;   // (never the newest row: it may not be in the cache)
        const int n_first = early ? 0 : min(STAGES - 1, max(whole_a, 0));          // (no cache reads before the wait)
        for (int s = 0; s < n_first; ++s) {
            issue_tile(0, s, islot, n_direct);
            cp_async_commit();
            islot = islot + 1 == STAGES ? 0 : islot + 1;
        }
        i_t = n_first;
    }
    const int n_early = i_t;
    int n_rows = n_direct;
    if (!m.keep_all && r_lo < m.prefix + m.n_win) {
        if (a.mask.mode == MODE_LIST) {
            for (int i = threadIdx.x; i < a.mask.bitmap_words; i += NTHR) bitmap[i] = 0u;
            __syncthreads();
            list_bitmap_fill<NTHR>(a.mask, m, a.mask.skip_offsets + (int64_t)b * a.mask.trace_len, bitmap);
            __syncthreads();
        }
        const int total = enumerate_scanned<NTHR, 1, BlockSync>(a.mask, m, bitmap, r_lo, r_hi, s_warp,
            [&](int slot, int pos, unsigned) { rowoff[slot] = pos; });
        n_rows = max(0, min(total - r_lo, a.chunk));
        __syncthreads();
        // positions -> byte offsets (independent block-table lookups, so they overlap)
#pragma unroll 4
        for (int i = n_direct + (int)threadIdx.x; i < n_rows; i += NTHR)
            rowoff[i] = token_offset(a, b, m.L_p, (int)rowoff[i]) * 2;
    }
    if constexpr (EARLY) {                            // the list is built: now wait for the kernel before this one
        asm volatile("griddepcontrol.wait;" ::: "memory");
        load_q(kvh0, qb);
        store_new();
    }
    if (n_rows <= 0) {
        for (int u = 0; u < U; ++u) write_empty_item<IC, 32>(a, m, b, kvh0 + u * W, split, lane);
        return;
    }
    __syncthreads();                                  // the last barrier: from here on warps run free
    // kept positions ascend, so the token being decoded can only be the list's last row
    if (APPEND && has_new && rowoff[n_rows - 1] == new_off) new_r = n_rows - 1;
    const int n_tiles = (n_rows + MMA_KEYS - 1) / MMA_KEYS;
    if (i_t >= n_tiles) { i_t = 0; i_u = 1; }         // (the early tiles were the whole first head)

    // One ring step on the producer side: the next tile of this warp's heads, or an empty group once
    // they are all issued (the group count per consumed tile stays fixed).
    auto issue_one = [&]() {
        if (i_u < U) {
            issue_tile(i_u, i_t, islot, n_rows);
            if (++i_t == n_tiles) { i_t = 0; ++i_u; }
        }
        cp_async_commit();
        islot = islot + 1 == STAGES ? 0 : islot + 1;
    };
    for (int s = n_early; s < STAGES - 1; ++s) issue_one();

    // accumulator-fragment coordinates: keys (or dims) lane/4 and lane/4 + 8, heads hc and hc + 1
    const int hc = (lane & 3) * 2, kr = lane >> 2;
    const int lm_row_k = (lane & 7) + ((lane >> 3) & 1) * 8, lm_chk_k = lane >> 4;
    const int lm_row_v = (lane & 7) + (lane >> 4) * 8, lm_chk_v = (lane >> 3) & 1;
    int cslot = 0;                                    // ring slot of the next tile to consume

#pragma unroll 1
    for (int u = 0; u < U; ++u) {
        const int kvh = kvh0 + u * W;
        if (u + 1 < U) load_q(kvh + W, qn);           // a head ahead: its latency hides behind this head's tiles
        float o[C::MTILES][4];
#pragma unroll
        for (int mt = 0; mt < C::MTILES; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
        float mrun[2] = {-INFINITY, -INFINITY}, lpart[2] = {0.f, 0.f};

        for (int tile = 0; tile < n_tiles; ++tile) {
            cp_async_wait<STAGES - 2>();
            __syncwarp();                               // the oldest tile landed for every lane; the slot before it is free
            issue_one();
            const unsigned char* ks = ring + cslot * C::SLOT_BYTES;
            const unsigned char* vs = ks + C::TILE_BYTES;
            cslot = cslot + 1 == STAGES ? 0 : cslot + 1;
            if constexpr (COPY_ONLY) {
                const uint4* p = reinterpret_cast<const uint4*>(ks);
                uint4 f = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int i = 0; i < C::SLOT_BYTES / 512; ++i) {
                    const uint4 x = p[i * 32 + lane];
                    f.x ^= x.x; f.y ^= x.y; f.z ^= x.z; f.w ^= x.w;
                }
                lpart[0] += __uint_as_float((f.x ^ f.y ^ f.z ^ f.w) & 0x007fffffu);    // (kept alive; tiny and finite)
                continue;
            }

            // S^T = K . Q^T
            float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kk = 0; kk < C::KSTEPS; ++kk) {
                unsigned af[4];
                const int chunk = kk * 2 + lm_chk_k;
                ldmatrix_x4(af, ks + lm_row_k * C::ROW_BYTES + ((chunk ^ (lm_row_k & 7)) * 16));
                mma_bf16_16816(s, af, qb[kk][0], qb[kk][1]);
            }
            // s[0]: (key kr, head hc)  s[1]: (kr, hc+1)  s[2]: (kr+8, hc)  s[3]: (kr+8, hc+1)
            const int r0 = tile * MMA_KEYS + kr, r1 = r0 + 8;
            const bool v0 = r0 < n_rows, v1 = r1 < n_rows;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float x0 = v0 ? s[j] * a.scale_log2 : -INFINITY;
                float x1 = v1 ? s[2 + j] * a.scale_log2 : -INFINITY;
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
            // P^T as B operand: accumulator layout [key][head] -> operand layout [head][key]
            const unsigned pb0 = movmatrix_trans(pack_bf16x2(s[0], s[1]));
            const unsigned pb1 = movmatrix_trans(pack_bf16x2(s[2], s[3]));
            // O^T += V^T . P^T
#pragma unroll
            for (int mt = 0; mt < C::MTILES; ++mt) {
                unsigned af[4];
                const int chunk = mt * 2 + lm_chk_v;
                ldmatrix_x4_trans(af, vs + lm_row_v * C::ROW_BYTES + ((chunk ^ (lm_row_v & 7)) * 16));
                mma_bf16_16816(o[mt], af, pb0, pb1);
            }
        }

        // ---- this head is done: sums over the key lanes, normalise, write ----------------------------
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            float l = lpart[j];
            l += __shfl_xor_sync(FULL, l, 4);
            l += __shfl_xor_sync(FULL, l, 8);
            l += __shfl_xor_sync(FULL, l, 16);
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
                }
            }
        }
        if (u + 1 < U) {
#pragma unroll
            for (int kk = 0; kk < C::KSTEPS; ++kk) { qb[kk][0] = qn[kk][0]; qb[kk][1] = qn[kk][1]; }
        }
    }
    cp_async_wait<0>();
}

}  // namespace dsa
