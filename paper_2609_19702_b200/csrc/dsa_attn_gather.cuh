// Split-KV decode attention for bf16 caches, head-group form with the tiles staged by the tensor
// memory accelerator: the rows a request keeps are scattered over the cache (skipped rows in
// between, pages anywhere), and sm_100's gather4 form of the tensor-map copy fetches four
// arbitrary rows of a 2-D view of the cache with ONE instruction of ONE lane, swizzles them on the
// way into shared memory and reports completion on an mbarrier.
//
// In dsa_attn_group.cuh every lane issues 16 sixteen-byte cp.async copies per 16-key tile (512 per
// warp), and a warp spends 900-1500 cycles per tile doing so.  Here a tile is 16 copies in all (4
// groups of 4 rows, x 2 128-byte halves of a row, x K and V), issued by lanes 0-15 in one
// instruction each.  A copy-only probe of the staging forms (8 warps per SM, the same scattered
// 256-byte rows, no arithmetic, GB/s moved) favoured it: cp.async 6350, one bulk copy per row 5320
// (the copy engine takes ~16 cycles per operation whatever its size), gather4 with swizzled
// 128-byte halves 7940.
//
// Inside the attention kernel the advantage does not survive: this form is 6-13 % SLOWER than the
// cp.async form on every shape measured (paged workload, batch 16 ... 256: 26.2 / 40.0 / 73.2 /
// 139.9 / 285.5 us against 22.4 / 37.7 / 68.3 / 130.6 / 252.0; decode loop at batch 128: 49.5
// against 40.6 us per layer-step).  The issue time that the copies save turns into waiting on the
// mbarrier (stall "wait" 2.44 against 1.67 per issue, 10 % more warp instructions because of the
// polling): with three slots per warp and 8 warps per SM the kernel is bound by how fast memory
// answers the two tiles a warp has in flight, not by issuing them, and the copy engine answers a
// little later than the load/store path.  A six-slot ring (five tiles in flight, one block per SM)
// made it 70 % slower still.  So the planner never chooses this kernel by itself: it runs only under
// DSA_PLAN_GATHER, for comparison runs and as the tested tensor-map path of the library.
//
// The cache is viewed as a matrix [token rows][elements of one token row]: row = offset of the
// token / stride_token, column = kv_head * stride_head (+ 64 for the second half of a 128-wide
// head).  The planner takes this kernel only when that view exists (see gather_view in dsa_api.cu).
// The row list holds 32-bit row numbers (the head-group kernel's holds 64-bit byte offsets).
// Everything else -- one list per (request, split) for W x U heads, the continuous ring across
// heads, S^T = K . Q^T / online softmax / O^T += V^T . P^T -- is dsa_attn_group.cuh's.
#pragma once
#include "dsa_attn_group.cuh"

namespace dsa {

// rows r.x, r.y, r.z, r.w of the view, columns [x, x + box width), to 4 consecutive box rows at dst
__device__ __forceinline__ void tma_gather4(void* dst, const CUtensorMap* map, int x, int4 r, unsigned long long* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile::gather4.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w), "r"(smem_u32(bar)) : "memory");
}

template <int D, int W, int STAGES>
struct GatherCfg {
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int CPR = ROW_BYTES / 16;
    static constexpr int HALVES = ROW_BYTES / 128;      // 128-byte pieces of a row: the widest box a 128B swizzle takes
    static constexpr int HALF_BYTES = MMA_KEYS * 128;   // one piece of all 16 rows: two 8-row swizzle atoms
    static constexpr int TILE_BYTES = MMA_KEYS * ROW_BYTES;
    static constexpr int SLOT_BYTES = 2 * TILE_BYTES;   // [K half 0][K half 1][V half 0][V half 1]
    static constexpr int COPIES = 2 * HALVES * 4;       // gather4 operations per tile, one lane each
    static constexpr int KSTEPS = D / 16;
    static constexpr int MTILES = D / 16;
    static constexpr int ALIGN = 1024;                  // swizzle atoms are 1 KB and must sit on 1 KB boundaries
    // dynamic shared memory: [slack to align][W rings][row list][one bitmap]
    __host__ static size_t smem_bytes(int chunk, int bitmap_words) {
        return (size_t)ALIGN + (size_t)W * STAGES * SLOT_BYTES + (size_t)chunk * 4 + (size_t)bitmap_words * 4;
    }
};

// The row of the 2-D view that holds token `pos` of request b (cf. token_offset).
__device__ __forceinline__ int token_row(const AttnArgs& a, const GatherMaps& g, int b, int L_p, int pos) {
    if (a.ring_size > 0) {
        const int first = L_p + a.ring_sinks;
        if (pos >= first) pos = first + (pos - first) % a.ring_size;
    }
    if (a.block_table) {
        const int bi = pos / a.block_size;
        int blk = a.block_table[(int64_t)b * a.max_blocks + min(bi, a.max_blocks - 1)];
        blk = max(0, min(blk, a.num_blocks - 1));
        return blk * g.rows_per_stride_b + (pos - bi * a.block_size);
    }
    return b * g.rows_per_stride_b + pos;
}

template <int D, int G, int STAGES, int W, bool APPEND>
__global__ void __launch_bounds__(32 * W) dsa_attn_gather_kernel(const AttnArgs a, const __grid_constant__ GatherMaps g) {
    using C = GatherCfg<D, W, STAGES>;
    using IC = MmaItemCfg<D, G, false, false>;
    using T = __nv_bfloat16;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int NTHR = 32 * W;

    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ int s_warp[W];
    __shared__ __align__(8) unsigned long long s_bar[W * STAGES];     // "tile landed", one per ring slot
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* smem = smem_raw + ((C::ALIGN - (smem_u32(smem_raw) & (C::ALIGN - 1))) & (C::ALIGN - 1));
    unsigned char* ring = smem + warp * (STAGES * C::SLOT_BYTES);
    int* rowid = reinterpret_cast<int*>(smem + W * STAGES * C::SLOT_BYTES);          // rows of the view
    unsigned* bitmap = reinterpret_cast<unsigned*>(rowid + a.chunk);
    unsigned long long* bars = s_bar + warp * STAGES;
    if (lane == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(bars + s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // (made visible to the copy engine; a barrier follows)

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
    load_q(kvh0, qb);

    bool has_new = false;
    const int S_step = APPEND ? step_seq_len(a, seq_raw, has_new) : seq_raw;
    const ReqMask m = req_mask_setup(a.mask, S_step, prompt_raw, a.max_seq_len);

    // Fused step: the token being decoded is not in the cache when the copies of this launch run, so
    // its slot of the list is fetched as an out-of-range row (zeros) and every lane keeps one 16-byte
    // piece of its K / V row (lanes [0, CPR): K, [CPR, 2 CPR): V) in a register, a head ahead, to put
    // it into the landed tile itself.  Split 0 also stores it to the cache for the launches to come.
    int new_row = -1, new_r = -1;
    uint4 newv = make_uint4(0u, 0u, 0u, 0u), newv_next = make_uint4(0u, 0u, 0u, 0u);
    const bool new_lane = lane < 2 * C::CPR, new_is_k = lane < C::CPR;
    const int new_c = new_is_k ? lane : lane - C::CPR;
    auto load_new = [&](int kvh) -> uint4 {
        const unsigned char* src = reinterpret_cast<const unsigned char*>(new_is_k ? a.k_new : a.v_new) +
                                   ((int64_t)b * a.H_kv + kvh) * C::ROW_BYTES + new_c * 16;
        return *reinterpret_cast<const uint4*>(src);
    };
    if (APPEND && has_new) {
        new_row = token_row(a, g, b, m.L_p, m.S - 1);
        if (new_lane) newv = load_new(kvh0);
        if (split == 0 && new_lane) {
            const int64_t new_off = token_offset(a, b, m.L_p, m.S - 1) * 2;
            unsigned char* dst0 = const_cast<unsigned char*>(reinterpret_cast<const unsigned char*>(new_is_k ? a.k : a.v)) +
                                  new_off + new_c * 16;
            const int64_t head_stride_bytes = a.stride_head * 2;
            *reinterpret_cast<uint4*>(dst0 + kvh0 * head_stride_bytes) = newv;
            for (int u = 1; u < U; ++u) {
                const int kvh = kvh0 + u * W;
                *reinterpret_cast<uint4*>(dst0 + kvh * head_stride_bytes) = load_new(kvh);
            }
        }
    }

    // ---- staging --------------------------------------------------------------------------------
    // tile `tile` of head u: lane l < COPIES fetches rows [16 tile + 4 (l & 3), + 4) of K or V, one
    // 128-byte piece of each, into its place of the slot
    const int cp_kv = lane / (C::HALVES * 4), cp_half = (lane >> 2) % C::HALVES, cp_g = lane & 3;
    const int col0 = (int)a.stride_head;              // columns of the view between neighbouring heads
    auto issue_tile = [&](int u, int tile, int slot) {
        if (lane == 0) mbar_expect_tx(bars + slot, C::SLOT_BYTES);
        __syncwarp();                                   // (the copies count down what lane 0 just counted up)
        if (lane < C::COPIES) {
            const int kvh = kvh0 + u * W;
            const int r0 = tile * MMA_KEYS + cp_g * 4;
            int4 r = *reinterpret_cast<const int4*>(rowid + r0);
            if (APPEND && new_r >= r0 && new_r < r0 + 4) {
                const int k = new_r - r0;
                if (k == 0) r.x = g.oob_row; else if (k == 1) r.y = g.oob_row; else if (k == 2) r.z = g.oob_row; else r.w = g.oob_row;
            }
            unsigned char* dst = ring + slot * C::SLOT_BYTES + cp_kv * C::TILE_BYTES + cp_half * C::HALF_BYTES + cp_g * 512;
            tma_gather4(dst, cp_kv ? &g.v : &g.k, kvh * col0 + cp_half * 64, r, bars + slot);
        }
    };

    // ---- the row list, once for all heads of the block --------------------------------------------
    const int r_lo = split * a.chunk, r_hi = r_lo + a.chunk;
    const int n_direct = enumerate_direct<NTHR, 1>(m, r_lo, r_hi, [&](int slot, int pos, unsigned) {
        rowid[slot] = token_row(a, g, b, m.L_p, pos);
    });
    __syncthreads();                                  // (also: every warp's barriers are initialised)
    int islot = 0;                                    // ring slot of the next issue
    int i_u = 0, i_t = 0;                             // next tile to issue: head i_u, tile i_t
    {
        const int whole_a = (n_direct - (APPEND ? 1 : 0)) / MMA_KEYS;   // (never the newest row: it is not in the cache)
        const int early = min(STAGES - 1, max(whole_a, 0));
        for (int s = 0; s < early; ++s) {
            issue_tile(0, s, islot);
            islot = islot + 1 == STAGES ? 0 : islot + 1;
        }
        i_t = early;
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
            [&](int slot, int pos, unsigned) { rowid[slot] = pos; });
        n_rows = max(0, min(total - r_lo, a.chunk));
        __syncthreads();
#pragma unroll 4
        for (int i = n_direct + (int)threadIdx.x; i < n_rows; i += NTHR)
            rowid[i] = token_row(a, g, b, m.L_p, rowid[i]);
    }
    if (n_rows <= 0) {
        for (int u = 0; u < U; ++u) write_empty_item<IC, 32>(a, m, b, kvh0 + u * W, split, lane);
        return;
    }
    const int n_tiles = (n_rows + MMA_KEYS - 1) / MMA_KEYS;
    // the last tile's missing rows are fetched out of range: zeros (their weights are zero as well)
    if ((int)threadIdx.x < n_tiles * MMA_KEYS - n_rows) rowid[n_rows + threadIdx.x] = g.oob_row;
    __syncthreads();                                  // the last barrier: from here on warps run free
    // kept positions ascend, so the token being decoded can only be the list's last row
    if (APPEND && has_new && rowid[n_rows - 1] == new_row) new_r = n_rows - 1;
    if (i_t >= n_tiles) { i_t = 0; i_u = 1; }         // (the early tiles were the whole first head)

    auto issue_one = [&]() {
        if (i_u < U) {
            issue_tile(i_u, i_t, islot);
            if (++i_t == n_tiles) { i_t = 0; ++i_u; }
        }
        islot = islot + 1 == STAGES ? 0 : islot + 1;
    };
    for (int s = n_early; s < STAGES - 1; ++s) issue_one();

    const int hc = (lane & 3) * 2, kr = lane >> 2;
    const int lm_row_k = (lane & 7) + ((lane >> 3) & 1) * 8, lm_chk_k = lane >> 4;
    const int lm_row_v = (lane & 7) + (lane >> 4) * 8, lm_chk_v = (lane >> 3) & 1;
    // byte offsets of this lane's ldmatrix rows inside a half, and the swizzle of their 16-byte pieces
    const int lm_off_k = lm_row_k * 128, lm_sw_k = lm_row_k & 7;
    const int lm_off_v = lm_row_v * 128, lm_sw_v = lm_row_v & 7;
    int cslot = 0;                                    // ring slot of the next tile to consume
    unsigned phases = 0u;                             // the phase to wait for, one bit per slot
    bool gave_up = false;

#pragma unroll 1
    for (int u = 0; u < U; ++u) {
        const int kvh = kvh0 + u * W;
        if (u + 1 < U) {
            load_q(kvh + W, qn);                       // a head ahead: its latency hides behind this head's tiles
            if (APPEND && new_r >= 0 && new_lane) newv_next = load_new(kvh + W);
        }
        float o[C::MTILES][4];
#pragma unroll
        for (int mt = 0; mt < C::MTILES; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
        float mrun[2] = {-INFINITY, -INFINITY}, lpart[2] = {0.f, 0.f};

        for (int tile = 0; tile < n_tiles; ++tile) {
            // Bounded wait for the tile: a copy that never lands is counted once, the kernel stops
            // waiting and runs to its end (its numbers are then wrong; dsa_wait_timeouts tells).
            mbar_wait_bounded(bars + cslot, (phases >> cslot) & 1u, gave_up, a.wait_timeouts, lane);
            phases ^= 1u << cslot;
            __syncwarp();                               // the slot consumed before this one is free for every lane
            issue_one();
            unsigned char* ks = ring + cslot * C::SLOT_BYTES;
            unsigned char* vs = ks + C::TILE_BYTES;
            cslot = cslot + 1 == STAGES ? 0 : cslot + 1;
            if (APPEND && new_r >= 0 && tile == n_tiles - 1) {
                if (new_lane) {
                    const int row = new_r & (MMA_KEYS - 1);
                    unsigned char* dst = (new_is_k ? ks : vs) + (new_c >> 3) * C::HALF_BYTES + row * 128 +
                                         (((new_c & 7) ^ (row & 7)) * 16);
                    *reinterpret_cast<uint4*>(dst) = newv;
                }
                __syncwarp();
            }

            // S^T = K . Q^T
            float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kk = 0; kk < C::KSTEPS; ++kk) {
                unsigned af[4];
                const int chunk = kk * 2 + lm_chk_k;
                ldmatrix_x4(af, ks + (chunk >> 3) * C::HALF_BYTES + lm_off_k + (((chunk & 7) ^ lm_sw_k) * 16));
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
                ldmatrix_x4_trans(af, vs + (chunk >> 3) * C::HALF_BYTES + lm_off_v + (((chunk & 7) ^ lm_sw_v) * 16));
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
            newv = newv_next;
        }
    }
}

}  // namespace dsa
