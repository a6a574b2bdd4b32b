// Split-KV decode attention for bf16 caches, head-group form with producer warps: every ring has a
// warp that only issues its copies and a warp that only consumes its tiles.
//
// In dsa_attn_group.cuh a warp alternates between issuing the 512 sixteen-byte copies of a tile
// (900-1500 cycles) and the two MMA chains with the softmax between them (~1100 cycles).  Here a
// block is W consumer warps and W producer warps on the same W rings: producer w + W issues the
// tiles of ring w as fast as slots come free, consumer w does nothing but wait for a tile, multiply
// and release the slot.  Same shared memory per block, twice the warps (16 per SM); the registers
// just fit (2 blocks x 256 threads x 128), which is also why this form cannot run three blocks to an
// SM with the shallow ring.
//
// What it buys is small, because a ring does not move a tile per max(issue, arithmetic) as hoped:
// a warp's copy instructions are accepted ~70 cycles apart whatever else the SM does (a copy-only
// probe: 2300 cycles per tile and warp with 2 or 5 tiles in flight, with 4 or 8 warps per SM), so
// the producer alone sets the pace and the consumer idles half the time.  Where the grid is more than
// one wave of deep-ring blocks it is 1.5-3.5 % faster than the plain form (paged workload, batch
// 224 / 256: 235.1 -> 226.8 / 250.8 -> 247.1 us; window 1024: 357.8 -> 352.8), where all blocks are
// resident from the start 2-3 % slower; the planner takes it for the former.  Two producer warps per ring (one for K, one
// for V; 12 warps per block, producers handing registers to consumers with setmaxnreg) ran at half
// the speed -- the consumer loop came out of the compiler with the block's 80 registers and spills.
//
// Hand-over: per ring slot a "full" mbarrier that the producer's 32 lanes arrive on asynchronously,
// each when its own copies of the tile have landed (cp.async.mbarrier.arrive.noinc), and an
// "empty" mbarrier that lane 0 of the consumer arrives on once the warp has read the tile.  Every
// wait is bounded: after about a second a warp counts the give-up (AttnArgs::wait_timeouts), stops
// waiting for the rest of the launch and runs to its end.
//
// The row list is built once per block by the consumer warps (a named barrier among them), while
// the producers wait at the two block barriers that publish it; list layout, work split, tile
// consumption and write-out are dsa_attn_group.cuh's.
#pragma once
#include "dsa_attn_gather.cuh"

namespace dsa {

// Barrier among the consumer warps only (threads [0, N)): they build the row list while the producer
// warps, which run on a few registers, wait for it at the block barriers.
template <int N>
struct ConsumerSync {
    __device__ static __forceinline__ void sync() { asm volatile("bar.sync 1, %0;" ::"n"(N) : "memory"); }
};

template <int D, int G, int STAGES, int W, bool APPEND>
__global__ void __launch_bounds__(64 * W, 2) dsa_attn_group_ws_kernel(const AttnArgs a) {
    using C = GroupCfg<D, W, STAGES>;
    using IC = MmaItemCfg<D, G, false, false>;
    using T = __nv_bfloat16;
    using CSync = ConsumerSync<32 * W>;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int NCONS = 32 * W;                     // consumer threads: they also build the list

    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_warp[W];
    __shared__ int s_info[4];                         // n_direct, n_rows, new_r: from the builders to the producers
    __shared__ __align__(8) unsigned long long s_full[W * STAGES], s_empty[W * STAGES];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool producer = warp >= W;
    const int rw = warp % W;                          // the ring this warp works on, and its head offset
    unsigned char* ring = smem + rw * (STAGES * C::SLOT_BYTES);
    int64_t* rowoff = reinterpret_cast<int64_t*>(smem + W * STAGES * C::SLOT_BYTES);   // bytes, kv head 0
    unsigned* bitmap = reinterpret_cast<unsigned*>(rowoff + a.chunk);
    unsigned long long* full = s_full + rw * STAGES;
    unsigned long long* empty = s_empty + rw * STAGES;
    if (!producer && lane == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full + s, 32); mbar_init(empty + s, 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.k);
    const unsigned char* vbase = reinterpret_cast<const unsigned char*>(a.v);

    const int U = a.heads_per_warp;
    const int hblocks = a.H_kv / (W * U);
    const int hb = blockIdx.x % hblocks;
    const int split = (blockIdx.x / hblocks) % a.n_split;
    const int b = blockIdx.x / (hblocks * a.n_split);
    const int kvh0 = hb * W * U + rw;                 // this ring's heads: kvh0, kvh0 + W, ...
    const int64_t head_stride_bytes = a.stride_head * 2;

    if (producer) {
        // ---- producer: wait for the list, then tile k goes into slot k mod STAGES as soon as the consumer
        // has released the slot's previous use ------------------------------------------------------------
        bool gave_up = false;
        int new_r = -1;
        auto issue_tile = [&](int u, int tile, int slot, int rows_ready) {
            const int kvh = kvh0 + u * W;
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
                const bool valid = r < rows_ready;
                const int dst = row * C::ROW_BYTES + ((c ^ (row & 7)) * 16);
                const int64_t off = valid ? rowoff[r] + head_bytes + c * 16 : 0;
                const bool is_new = APPEND && r == new_r;   // (not in the cache yet: read it where the caller put it)
                cp_async16(ks + dst, kbase + (is_new ? knew_off + c * 16 : off), valid);
                cp_async16(vs + dst, vbase + (is_new ? vnew_off + c * 16 : off), valid);
            }
            cp_async_arrive_on(full + slot);
        };
        __syncthreads();                              // A: the rows that needed no scan are listed
        const int n_direct = s_info[0];
        const int whole_a = (n_direct - (APPEND ? 1 : 0)) / MMA_KEYS;   // (never the newest row: it may not be in the cache)
        const int n_early = min(STAGES, max(whole_a, 0));
        for (int s = 0; s < n_early; ++s) issue_tile(0, s, s, n_direct);
        __syncthreads();                              // B: the list is complete
        const int n_rows = s_info[1];
        new_r = s_info[2];
        if (n_rows <= 0) return;                      // (then nothing was issued either)
        const int n_tiles = (n_rows + MMA_KEYS - 1) / MMA_KEYS;
        const int n_total = n_tiles * U;
        int slot = n_early % STAGES;
        int u = n_early / n_tiles, t = n_early % n_tiles;
        for (int k = n_early; k < n_total; ++k) {
            if (k >= STAGES) mbar_wait_bounded(empty + slot, (unsigned)((k / STAGES - 1) & 1), gave_up, a.wait_timeouts, lane);
            issue_tile(u, t, slot, n_rows);
            if (++t == n_tiles) { t = 0; ++u; }
            slot = slot + 1 == STAGES ? 0 : slot + 1;
        }
        cp_async_wait<0>();                             // (nothing of this thread's is in flight when it leaves)
        return;
    }

    // ---- consumers: lengths, mask, the fused step's store, the row list ----------------------------------
    const int seq_raw = a.seq_len[b], prompt_raw = req_prompt_len(a, b);
    bool has_new = false;
    const int S_step = APPEND ? step_seq_len(a, seq_raw, has_new) : seq_raw;
    const ReqMask m = req_mask_setup(a.mask, S_step, prompt_raw, a.max_seq_len);
    int64_t new_off = 0;
    if (APPEND && has_new) {
        new_off = token_offset(a, b, m.L_p, m.S - 1) * 2;
        if (split == 0 && lane < 2 * C::CPR) {
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
    }
    const int r_lo = split * a.chunk, r_hi = r_lo + a.chunk;
    const int n_direct = enumerate_direct<NCONS, 1>(m, r_lo, r_hi, [&](int slot, int pos, unsigned) {
        rowoff[slot] = token_offset(a, b, m.L_p, pos) * 2;
    });
    if (threadIdx.x == 0) s_info[0] = n_direct;
    __syncthreads();                                  // A (also: the barriers are initialised)
    int n_rows = n_direct;
    if (!m.keep_all && r_lo < m.prefix + m.n_win) {
        if (a.mask.mode == MODE_LIST) {
            for (int i = threadIdx.x; i < a.mask.bitmap_words; i += NCONS) bitmap[i] = 0u;
            CSync::sync();
            list_bitmap_fill<NCONS>(a.mask, m, a.mask.skip_offsets + (int64_t)b * a.mask.trace_len, bitmap);
            CSync::sync();
        }
        const int total = enumerate_scanned<NCONS, 1, CSync>(a.mask, m, bitmap, r_lo, r_hi, s_warp,
            [&](int slot, int pos, unsigned) { rowoff[slot] = pos; });
        n_rows = max(0, min(total - r_lo, a.chunk));
        CSync::sync();
#pragma unroll 4
        for (int i = n_direct + (int)threadIdx.x; i < n_rows; i += NCONS)
            rowoff[i] = token_offset(a, b, m.L_p, (int)rowoff[i]) * 2;
        CSync::sync();
    }
    if (threadIdx.x == 0) {
        s_info[1] = n_rows;
        // kept positions ascend, so the token being decoded can only be the list's last row
        s_info[2] = (APPEND && has_new && n_rows > 0 && rowoff[n_rows - 1] == new_off) ? n_rows - 1 : -1;
    }
    __syncthreads();                                  // B: the last block barrier, from here on warps run free
    if (n_rows <= 0) {
        for (int u = 0; u < U; ++u) write_empty_item<IC, 32>(a, m, b, kvh0 + u * W, split, lane);
        return;
    }
    const int n_tiles = (n_rows + MMA_KEYS - 1) / MMA_KEYS;
    bool gave_up = false;

    // ---- consumer ------------------------------------------------------------------------------------
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
    load_q(kvh0, qb);
    const int hc = (lane & 3) * 2, kr = lane >> 2;
    const int lm_row_k = (lane & 7) + ((lane >> 3) & 1) * 8, lm_chk_k = lane >> 4;
    const int lm_row_v = (lane & 7) + (lane >> 4) * 8, lm_chk_v = (lane >> 3) & 1;
    int cslot = 0;                                    // ring slot of the next tile to consume
    unsigned phases = 0u;                             // the "full" phase to wait for, one bit per slot

#pragma unroll 1
    for (int u = 0; u < U; ++u) {
        const int kvh = kvh0 + u * W;
        if (u + 1 < U) load_q(kvh + W, qn);           // a head ahead: its latency hides behind this head's tiles
        float o[C::MTILES][4];
#pragma unroll
        for (int mt = 0; mt < C::MTILES; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
        float mrun[2] = {-INFINITY, -INFINITY}, lpart[2] = {0.f, 0.f};

        for (int tile = 0; tile < n_tiles; ++tile) {
            mbar_wait_bounded(full + cslot, (phases >> cslot) & 1u, gave_up, a.wait_timeouts, lane);
            phases ^= 1u << cslot;
            const unsigned char* ks = ring + cslot * C::SLOT_BYTES;
            const unsigned char* vs = ks + C::TILE_BYTES;

            // S^T = K . Q^T
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
            __syncwarp();                               // every lane has read the tile: hand the slot back
            if (lane == 0) mbar_arrive(empty + cslot);
            cslot = cslot + 1 == STAGES ? 0 : cslot + 1;
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
}

}  // namespace dsa
