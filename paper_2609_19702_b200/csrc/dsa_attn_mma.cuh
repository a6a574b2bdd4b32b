// Split-KV decode attention for bf16 caches: ONE WARP per work item, tensor-core tiles.
//
// Why tensor cores in a bandwidth-bound kernel: with fp32 FMAs on the CUDA cores the scan costs
// about 0.14 warp instructions per byte; at 6.5-7 TB/s that is 80-90 % of the issue slots of the
// 148 SMs (measured), i.e. the kernel had become issue-bound.  mma.sync m16n8k16 brings it to
// about 0.02 instructions per byte; that most of each MMA multiplies padding is irrelevant.
//
// Formulation (transposed, so that the 16-row MMA dimension is filled with keys, not heads):
//   S^T[16 keys x 8 heads]  = K_tile[16 keys x D] . Q^T[D x 8 heads]          (D/16 MMAs)
//   O^T[D x 8 heads]       += V_tile^T[D x 16 keys] . P^T[16 keys x 8 heads]   (D/16 MMAs)
// The 8 "heads" are the G <= 8 query heads that share this kv head (GQA packing), the rest zero.
// K is the row-major A operand (ldmatrix), V^T comes from ldmatrix.trans on the same [key][dim]
// layout, P^T is moved from accumulator layout to B-operand layout with movmatrix.  Online
// softmax runs on the accumulator fragment: a thread owns two head columns and keys lane/4 and
// lane/4 + 8; column maxima take three shuffles, sums are kept per thread and reduced once.
//
// A work item belongs to a single warp, which streams it through its own 2-3 stage cp.async ring of
// 16-key tiles: no block barrier in the main loop, the hardware schedules and balances the warps,
// and ~10 of them per SM keep well over 100 KB in flight.  A block holds W warps that work on W
// neighbouring kv heads of the same (request, split): whenever the mask does not depend on the
// head (dense, window, grid, one shared list) the row list is the same for all of them, so the
// block builds it once with all its threads and every warp only adds its head's offset.  Masks
// per head run with W = 1.  Shared-memory tiles are XOR-swizzled in 16-byte chunks so that the
// ldmatrix row reads are conflict-free.
#pragma once
#include "dsa_tile.cuh"

namespace dsa {

constexpr int MMA_KEYS = 16;     // keys per tile

__device__ __forceinline__ void ldmatrix_x4(unsigned (&r)[4], const void* smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"((unsigned)__cvta_generic_to_shared(smem_row)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned (&r)[4], const void* smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"((unsigned)__cvta_generic_to_shared(smem_row)));
}
__device__ __forceinline__ unsigned movmatrix_trans(unsigned x) {
    unsigned y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// {lo, hi} -> packed bf16x2 (lo in the low half)
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {
    unsigned d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// ---- thread-block clusters: the CTAs of a cluster share one work item (see CL below) -------------
__device__ __forceinline__ unsigned cluster_ctarank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// split cluster barrier: every thread of every CTA arrives, and waits where it needs the others
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// a float of CTA `rank`'s shared memory, at the place where this CTA has `local` (distributed shared memory)
__device__ __forceinline__ float ld_cluster_f32(const float* local, unsigned rank) {
    unsigned remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                 : "=r"(remote) : "r"((unsigned)__cvta_generic_to_shared(local)), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

template <int D, int G, int STAGES, bool HEADMASK, bool SELECT, int W = 1>
struct MmaCfg {
    using T = __nv_bfloat16;
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int CPR = ROW_BYTES / 16;              // 16-byte chunks per row (8 or 16)
    static constexpr int TILE_BYTES = MMA_KEYS * ROW_BYTES; // one K (or V) tile
    static constexpr int SLOT_BYTES = 2 * TILE_BYTES;
    static constexpr int KSTEPS = D / 16;                   // MMAs of the score product
    static constexpr int MTILES = D / 16;                   // MMAs of the output product
    static constexpr int SLOTS = HEADMASK ? G : 1;
    __host__ __device__ static constexpr int list_bytes(int chunk) {
        return chunk * 8 + (SELECT ? chunk * 4 : 0) + (HEADMASK ? ((chunk + 15) / 16) * 16 : 0);
    }
    // dynamic shared memory: [W rings: STAGES x (K tile, V tile)][row list][bitmaps]
    __host__ static size_t smem_bytes(int chunk, int bitmap_words) {
        return (size_t)W * STAGES * SLOT_BYTES + list_bytes(chunk) + (size_t)SLOTS * bitmap_words * 4;
    }
};

// adapter with the member names the shared list-building code uses
template <int D_, int G_, bool HEADMASK_, bool SELECT_>
struct MmaItemCfg {
    using T = __nv_bfloat16;
    static constexpr int D = D_, G = G_;
    static constexpr bool HEADMASK = HEADMASK_, SELECT = SELECT_;
    static constexpr int SLOTS = HEADMASK ? G : 1;
};

// APPEND: fused decode step.  The token being decoded is not in the cache yet: its K/V rows are
// read from k_new / v_new wherever the row list names its position, and the warps of split 0
// write them to the cache (nobody reads that slot in this launch: with a bounded cache it belonged
// to a token that has left the window).
//
// KW > 1: small launches.  When the (request, kv head) pairs are too few to fill the device, KW
// warps share one work item instead of the item being cut into KW splits with a combine launch
// behind them: they build the row list together, warp k streams tiles k, k + KW, ... through its
// own ring, and the partial softmax states are merged through shared memory at the end.
//
// CL > 1: smaller launches still.  A thread-block CLUSTER of CL such blocks shares the work item:
// block r of the cluster builds and streams rows [r chunk, (r + 1) chunk) of the kept sequence (so
// CL x KW warps have one to three tiles each, all in flight at once), merges its warps as above, and
// block 0 then reads the other blocks' merged states straight out of their shared memory
// (ld.shared::cluster after a cluster barrier) and writes the result: no partials in HBM, no combine
// launch.  The launch carries the cluster dimension; plain per-thread loads only cross the cluster.
// EARLY: the caller has promised that no launch still running writes the arrays the row list is made
// from (AttnArgs::early_list): the list is built before waiting for the launch in front; q, the new rows
// and the caches are read after the wait.
template <int D, int G, int STAGES, bool HEADMASK, bool SELECT, int W, bool APPEND = false, int KW = 1, int CL = 1,
          bool EARLY = false>
__global__ void __launch_bounds__(32 * W * KW) dsa_attn_mma_kernel(const AttnArgs a) {
    using C = MmaCfg<D, G, STAGES, HEADMASK, SELECT, W * KW>;   // one ring per warp
    using IC = MmaItemCfg<D, G, HEADMASK, SELECT>;
    using T = __nv_bfloat16;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int NW = W * KW;                            // warps per block
    static_assert(W == 1 || (!HEADMASK && !SELECT), "a shared row list needs a head-independent mask");
    static_assert(W == 1 || KW == 1, "several warps per head only with one head per block");
    static_assert(CL == 1 || (KW > 1 && !SELECT), "clusters extend the several-warps-per-item form");

    // Programmatic launch on both sides: a combine kernel queued behind this grid may be scheduled
    // from now on (it waits for this grid to finish before it reads anything), and this grid may
    // itself have been scheduled early behind the append kernel of the same decode step: wait for
    // that kernel's writes (the new K/V rows, seq_len) before touching global memory.
    asm volatile("griddepcontrol.launch_dependents;");
    if constexpr (!EARLY) asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_warp[NW];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hw = KW == 1 ? warp : 0;                    // this warp's head within the block
    const int wk = KW == 1 ? 0 : warp;                    // its rank among the warps of that head
    unsigned char* ring = smem + warp * (STAGES * C::SLOT_BYTES);
    const RowList list = RowList::carve<IC>(smem + NW * STAGES * C::SLOT_BYTES, a.chunk);
    unsigned* bitmaps = reinterpret_cast<unsigned*>(smem + NW * STAGES * C::SLOT_BYTES + C::list_bytes(a.chunk));

    // kv heads vary fastest across the grid: the warps that run together read the same tokens
    // of neighbouring heads, i.e. neighbouring memory.
    const int hblocks = a.H_kv / W;
    // (cluster form: the CL blocks of a cluster are consecutive and take the "splits" of one pair;
    // a.n_split is 1 there, the result is final)
    const unsigned item_block = CL > 1 ? blockIdx.x / CL : blockIdx.x;
    const int kvh = (item_block % hblocks) * W + hw;
    const int split = CL > 1 ? (int)cluster_ctarank() : (item_block / hblocks) % a.n_split;
    const int b = CL > 1 ? item_block / hblocks : item_block / (hblocks * a.n_split);

    const int seq_raw = a.seq_len[b], prompt_raw = req_prompt_len(a, b);
    // ---- Q^T as B operand: head = lane / 4, dims 2*(lane%4)+{0,1} (+8) of every 16-dim step ----
    // Loaded first, used last: the loads depend on nothing but the work item, so their latency
    // hides behind the mask set-up and the row list (columns beyond the group are zeroed at use).
    const int hq = lane >> 2;                 // head column this thread feeds
    const int qd = (lane & 3) * 2;
    unsigned qb[C::KSTEPS][2];
    if constexpr (!EARLY) {
        const T* qrow = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.H_q + kvh * G + (hq < G ? hq : 0)) * D;
#pragma unroll
        for (int kk = 0; kk < C::KSTEPS; ++kk) {
            qb[kk][0] = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd);
            qb[kk][1] = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd + 8);
        }
    }
    bool has_new = false;
    const int S_step = APPEND ? step_seq_len(a, seq_raw, has_new) : seq_raw;
    const ReqMask m = req_mask_setup(a.mask, S_step, prompt_raw, a.max_seq_len);
    auto sync_builders = [&]() { if (NW == 1) __syncwarp(); else __syncthreads(); };
    // W > 1: one list for all the block's heads, built without a head offset (kv head "0")
    const int list_kvh = W == 1 ? kvh : 0;
    const int64_t head_bytes = W == 1 ? 0 : (int64_t)kvh * a.stride_head * 2;
    const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.k);
    const unsigned char* vbase = reinterpret_cast<const unsigned char*>(a.v);
    // fused step: where the current token's rows come from and where they go (kv head 0)
    const unsigned char* knew_row = nullptr;
    const unsigned char* vnew_row = nullptr;
    int64_t off_new = 0;
    int new_r = -1;                                       // its row in this item's list, once known
    uint4 new_chunk = make_uint4(0u, 0u, 0u, 0u);
    const bool store_new = APPEND && has_new && split == 0 && wk == 0 && lane < 2 * C::CPR;
    if (APPEND && has_new) {
        const int64_t row_bytes = ((int64_t)b * a.H_kv + kvh) * C::ROW_BYTES;
        knew_row = reinterpret_cast<const unsigned char*>(a.k_new) + row_bytes;
        vnew_row = reinterpret_cast<const unsigned char*>(a.v_new) + row_bytes;
        off_new = token_offset(a, b, m.L_p, m.S - 1);
        if constexpr (!EARLY) {
            if (store_new) {                              // lanes [0, CPR): K chunks, [CPR, 2 CPR): V chunks
                const unsigned char* src = lane < C::CPR ? knew_row + lane * 16 : vnew_row + (lane - C::CPR) * 16;
                new_chunk = *reinterpret_cast<const uint4*>(src);
            }
        }
    }

    // ---- staging: this warp's own ring of 16-key tiles ---------------------------------------
    // rows_ready: rows of the list that exist so far (tiles below it can be issued)
    // `tile` counts this warp's own tiles; it is tile wk + tile * KW of the item
    auto issue_tile = [&](int tile, int rows_ready) {
        const int row0 = (wk + tile * KW) * MMA_KEYS;
        if (row0 < rows_ready) {
            unsigned char* ks = ring + (tile % STAGES) * C::SLOT_BYTES;
            unsigned char* vs = ks + C::TILE_BYTES;
#pragma unroll
            for (int i = 0; i < MMA_KEYS * C::CPR / 32; ++i) {
                const int idx = i * 32 + lane;
                const int row = idx / C::CPR, c = idx % C::CPR;
                const int r = row0 + row;
                const bool valid = r < rows_ready;
                const int64_t off = valid ? list.rowoff[r] * 2 + head_bytes + c * 16 : 0;
                const int dst = row * C::ROW_BYTES + ((c ^ (row & 7)) * 16);       // swizzled chunk
                if (APPEND && r == new_r) {
                    cp_async16(ks + dst, knew_row + c * 16, valid);
                    cp_async16(vs + dst, vnew_row + c * 16, valid);
                } else {
                    cp_async16(ks + dst, kbase + off, valid);
                    cp_async16(vs + dst, vbase + off, valid);
                }
            }
        }
        cp_async_commit();
    };

    // Phase A of the row list: the rows that need no scan (prompt, old sinks, unmasked window).
    // The first tiles of the ring are issued from them right away, so that the memory stream is
    // already running while phase B (mask bitmaps, window scan, block-table lookups) is computed.
    const int n_direct = build_rows_direct<IC, 32 * NW>(a, m, b, list_kvh, split, list);
    sync_builders();
    // whole tiles inside phase A (fused step: never the newest row, which may not be in the cache)
    // that are this warp's
    const int whole_a = (n_direct - (APPEND ? 1 : 0)) / MMA_KEYS;
    const int early = EARLY ? 0 : min(STAGES - 1, whole_a > wk ? (whole_a - wk + KW - 1) / KW : 0);   // (EARLY: no cache reads yet)
    for (int s = 0; s < early; ++s) issue_tile(s, n_direct);
    const int n_rows = NW == 1
        ? build_rows_scanned<IC, WarpSync, 32>(a, m, b, list_kvh, split, list, bitmaps, s_warp, n_direct)
        : build_rows_scanned<IC, BlockSync, 32 * NW>(a, m, b, list_kvh, split, list, bitmaps, s_warp, n_direct);
    if constexpr (EARLY) {                             // the list is built: now wait for the launch in front
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const T* qrow = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.H_q + kvh * G + (hq < G ? hq : 0)) * D;
#pragma unroll
        for (int kk = 0; kk < C::KSTEPS; ++kk) {
            qb[kk][0] = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd);
            qb[kk][1] = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd + 8);
        }
        if (store_new) {
            const unsigned char* src = lane < C::CPR ? knew_row + lane * 16 : vnew_row + (lane - C::CPR) * 16;
            new_chunk = *reinterpret_cast<const uint4*>(src);
        }
    }
    if (store_new) {
        unsigned char* base = const_cast<unsigned char*>(lane < C::CPR ? kbase : vbase);
        const int c = lane < C::CPR ? lane : lane - C::CPR;
        *reinterpret_cast<uint4*>(base + (off_new + (int64_t)kvh * a.stride_head) * 2 + c * 16) = new_chunk;
    }
    if (CL == 1 && n_rows <= 0) {
        if (wk == 0) write_empty_item<IC, 32>(a, m, b, kvh, split, lane);
        return;
    }
    // (a block of a cluster that got no rows goes on with zero tiles: the others wait for it)
    sync_builders();                                   // the last barrier: from here on warps run free
    // kept positions ascend, so the token being decoded can only be this item's last row
    if (APPEND && has_new && (CL == 1 || n_rows > 0) && list.rowoff[n_rows - 1] == off_new + (int64_t)list_kvh * a.stride_head)
        new_r = n_rows - 1;
    const int item_tiles = (n_rows + MMA_KEYS - 1) / MMA_KEYS;
    const int n_tiles = item_tiles > wk ? (item_tiles - wk + KW - 1) / KW : 0;      // this warp's
    for (int s = early; s < STAGES - 1; ++s) issue_tile(s, n_rows);

    if (hq >= G) {
#pragma unroll
        for (int kk = 0; kk < C::KSTEPS; ++kk) { qb[kk][0] = 0u; qb[kk][1] = 0u; }
    }
    // accumulator-fragment coordinates: keys (or dims) lane/4 and lane/4 + 8, heads hc and hc + 1
    const int hc = (lane & 3) * 2;
    const int kr = lane >> 2;
    float o[C::MTILES][4];
#pragma unroll
    for (int mt = 0; mt < C::MTILES; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
    float mrun[2] = {-INFINITY, -INFINITY}, lpart[2] = {0.f, 0.f};
    float bestv[2] = {INFINITY, INFINITY};
    int bestp[2] = {0x7fffffff, 0x7fffffff};
    const int cand_lo = m.L_p + a.mask.n_sink;

    // per-lane ldmatrix row addresses inside a tile (swizzle applied per k-step / m-tile below)
    const int lm_row_k = (lane & 7) + ((lane >> 3) & 1) * 8;     // K as A: matrices (r0-7,c0) (r8-15,c0) (r0-7,c1) (r8-15,c1)
    const int lm_chk_k = lane >> 4;
    const int lm_row_v = (lane & 7) + (lane >> 4) * 8;           // V^T as A: (k0-7,d0) (k0-7,d1) (k8-15,d0) (k8-15,d1)
    const int lm_chk_v = (lane >> 3) & 1;

    for (int tile = 0; tile < n_tiles; ++tile) {
        cp_async_wait<STAGES - 2>();
        __syncwarp();                                   // tile landed for every lane; tile-1 fully consumed
        issue_tile(tile + STAGES - 1, n_rows);
        const unsigned char* ks = ring + (tile % STAGES) * C::SLOT_BYTES;
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
        // s[0]: (key kr, head hc)  s[1]: (kr, hc+1)  s[2]: (kr+8, hc)  s[3]: (kr+8, hc+1)
        const int r0 = (wk + tile * KW) * MMA_KEYS + kr, r1 = r0 + 8;
        const bool v0 = r0 < n_rows, v1 = r1 < n_rows;
        unsigned bits0 = 0xffu, bits1 = 0xffu;
        if (HEADMASK) { bits0 = v0 ? list.hbits[r0] : 0u; bits1 = v1 ? list.hbits[r1] : 0u; }
        int pos0 = 0, pos1 = 0;
        if (SELECT) { pos0 = v0 ? list.rowpos[r0] : 0; pos1 = v1 ? list.rowpos[r1] : 0; }
#pragma unroll
        for (int j = 0; j < 2; ++j) {                   // the thread's two head columns
            const bool on0 = v0 && (!HEADMASK || ((bits0 >> (hc + j)) & 1u));
            const bool on1 = v1 && (!HEADMASK || ((bits1 >> (hc + j)) & 1u));
            float x0 = on0 ? s[j] * a.scale_log2 : -INFINITY;
            float x1 = on1 ? s[2 + j] * a.scale_log2 : -INFINITY;
            if (SELECT) {
                // keys arrive in ascending position: a strict "<" keeps the oldest of equal logits
                if (on0 && pos0 >= cand_lo && x0 < bestv[j]) { bestv[j] = x0; bestp[j] = pos0; }
                if (on1 && pos1 >= cand_lo && x1 < bestv[j]) { bestv[j] = x1; bestp[j] = pos1; }
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
        // P^T as B operand: accumulator layout [key][head] -> operand layout [head][key]
        const unsigned pb0 = movmatrix_trans(pack_bf16x2(s[0], s[1]));     // keys 0-7
        const unsigned pb1 = movmatrix_trans(pack_bf16x2(s[2], s[3]));     // keys 8-15
        // O^T += V^T . P^T
#pragma unroll
        for (int mt = 0; mt < C::MTILES; ++mt) {
            unsigned af[4];
            const int chunk = mt * 2 + lm_chk_v;
            ldmatrix_x4_trans(af, vs + lm_row_v * C::ROW_BYTES + ((chunk ^ (lm_row_v & 7)) * 16));
            mma_bf16_16816(o[mt], af, pb0, pb1);
        }
    }
    cp_async_wait<0>();

    // ---- finish: sums over the key lanes, merge the warps of the item, normalise, write --------
    float ltot[2], bv[2];
    int bp[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        float l = lpart[j];
        l += __shfl_xor_sync(FULL, l, 4);
        l += __shfl_xor_sync(FULL, l, 8);
        l += __shfl_xor_sync(FULL, l, 16);
        ltot[j] = l;
        bv[j] = bestv[j];
        bp[j] = bestp[j];
        if (SELECT) {
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                const float ov = __shfl_xor_sync(FULL, bv[j], off);
                const int op = __shfl_xor_sync(FULL, bp[j], off);
                if (ov < bv[j] || (ov == bv[j] && op < bp[j])) { bv[j] = ov; bp[j] = op; }
            }
        }
    }
    if (KW > 1) {
        // Every warp holds its state in the same fragment layout, so the merge is element-wise:
        // warps 1.. leave theirs in shared memory (the rings are free now), warp 0 folds them in.
        constexpr int REC = C::MTILES * 4 + 8;            // floats per lane: o, m[2], l[2], best value[2], best position[2]
        float* rec = reinterpret_cast<float*>(smem);
        __syncthreads();                                  // all rings drained and consumed
        if (wk > 0) {
            float* mine = rec + (size_t)(wk - 1) * REC * 32 + lane;
#pragma unroll
            for (int mt = 0; mt < C::MTILES; ++mt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) mine[(mt * 4 + e) * 32] = o[mt][e];
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                mine[(C::MTILES * 4 + j) * 32] = mrun[j];
                mine[(C::MTILES * 4 + 2 + j) * 32] = ltot[j];
                mine[(C::MTILES * 4 + 4 + j) * 32] = bv[j];
                mine[(C::MTILES * 4 + 6 + j) * 32] = __int_as_float(bp[j]);
            }
        }
        __syncthreads();
        if (CL == 1) { if (wk > 0) return; }
        for (int w = 1; w < (CL == 1 || wk == 0 ? KW : 1); ++w) {
            const float* other = rec + (size_t)(w - 1) * REC * 32 + lane;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float m_o = other[(C::MTILES * 4 + j) * 32];
                const float l_o = other[(C::MTILES * 4 + 2 + j) * 32];
                const float mnew = fmaxf(mrun[j], m_o);
                const float msafe = mnew == -INFINITY ? 0.f : mnew;
                const float c0 = fast_exp2(mrun[j] - msafe), c1 = fast_exp2(m_o - msafe);
                ltot[j] = ltot[j] * c0 + l_o * c1;
                mrun[j] = mnew;
#pragma unroll
                for (int mt = 0; mt < C::MTILES; ++mt) {
                    o[mt][j] = o[mt][j] * c0 + other[(mt * 4 + j) * 32] * c1;
                    o[mt][2 + j] = o[mt][2 + j] * c0 + other[(mt * 4 + 2 + j) * 32] * c1;
                }
                if (SELECT) {
                    const float ov = other[(C::MTILES * 4 + 4 + j) * 32];
                    const int op = __float_as_int(other[(C::MTILES * 4 + 6 + j) * 32]);
                    if (ov < bv[j] || (ov == bv[j] && op < bp[j])) { bv[j] = ov; bp[j] = op; }
                }
            }
        }
    }
    if (CL > 1) {
        // Merge across the cluster.  Every thread of every block passes the same two barriers:
        //   blocks 1.. leave their merged state in their OWN shared memory   -> barrier 1 ->
        //   block 0 reads it there (distributed shared memory) and folds it in -> barrier 2 ->
        //   the other blocks may exit (their memory is no longer needed).
        constexpr int REC = C::MTILES * 4 + 8;
        float* rec = reinterpret_cast<float*>(smem) + lane;       // (warp 0 is done with the other warps' records)
        if (wk == 0 && split > 0) {
#pragma unroll
            for (int mt = 0; mt < C::MTILES; ++mt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) rec[(mt * 4 + e) * 32] = o[mt][e];
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                rec[(C::MTILES * 4 + j) * 32] = mrun[j];
                rec[(C::MTILES * 4 + 2 + j) * 32] = ltot[j];
            }
        }
        cluster_arrive();
        cluster_wait();
        if (wk == 0 && split == 0) {
            for (unsigned r = 1; r < (unsigned)CL; ++r) {
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const float m_o = ld_cluster_f32(rec + (C::MTILES * 4 + j) * 32, r);
                    const float l_o = ld_cluster_f32(rec + (C::MTILES * 4 + 2 + j) * 32, r);
                    const float mnew = fmaxf(mrun[j], m_o);
                    const float msafe = mnew == -INFINITY ? 0.f : mnew;
                    const float c0 = fast_exp2(mrun[j] - msafe), c1 = fast_exp2(m_o - msafe);
                    ltot[j] = ltot[j] * c0 + l_o * c1;
                    mrun[j] = mnew;
#pragma unroll
                    for (int mt = 0; mt < C::MTILES; ++mt) {
                        o[mt][j] = o[mt][j] * c0 + ld_cluster_f32(rec + (mt * 4 + j) * 32, r) * c1;
                        o[mt][2 + j] = o[mt][2 + j] * c0 + ld_cluster_f32(rec + (mt * 4 + 2 + j) * 32, r) * c1;
                    }
                }
            }
        }
        cluster_arrive();
        if (wk > 0 || split > 0) {
            cluster_wait();
            return;
        }
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const float l = ltot[j];
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
                    const int off = bp[j] == 0x7fffffff ? -1 : (m.S - 1) - bp[j];
                    if (a.n_split > 1) {
                        a.sel_val_part[row * a.n_split + split] = bv[j];
                        a.sel_off_part[row * a.n_split + split] = off;
                        a.sel_k[row] = m.sel_k;
                    } else if (m.sel_k >= 0) {
                        record_selection(a.mask, row, m.sel_k, off);
                    }
                }
            }
        }
    }
    if (CL > 1) cluster_wait();                           // (barrier 2, for form's sake: every arrival is waited for)
}

}  // namespace dsa
