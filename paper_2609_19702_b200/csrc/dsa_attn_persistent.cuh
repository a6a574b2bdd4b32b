// Split-KV decode attention with persistent, warp-specialised thread blocks.
//
// The grid is a few blocks per SM; block c takes work items c, c + gridDim.x, ...  (items are
// numbered with the kv head fastest, so co-resident blocks read neighbouring memory).  A block is
// 4 compute warps + 1 loader warp:
//   - the loader warp streams K/V rows into a ring of small tiles in shared memory with 1-D bulk
//     async copies (one copy per 128/256-byte row, completion counted on the tile's "full"
//     mbarrier), running straight on from the tiles of one item into those of the next;
//   - the compute warps build the row list of the NEXT item with the mask generator while the
//     loader is still streaming the current one, then consume tiles as they land (waiting on
//     "full", releasing through "empty"), merge, write the result and move on.
// So the memory stream never drains between work items: the per-item start-up (sequence lengths,
// mask generation, block-table lookups) and the merge hide behind tiles already in flight.
//
// Every wait on an mbarrier is bounded by a cycle budget.  A wait that runs out records a code in
// the device error flag and raises the block's abort flag, after which every wait of the block
// returns at once.  The compute warps then run their (finite) loops to the end without waiting --
// their results are garbage, but they keep meeting at their named barrier, so nothing can hang --
// and the loader stops issuing copies and waits, again bounded, for those in flight.
#pragma once
#include "dsa_tile.cuh"

namespace dsa {

constexpr int NT_PERSIST = NT + 32;             // compute threads + the loader warp
constexpr long long WAIT_CYCLES = 1ll << 31;    // about a second: far beyond any legitimate wait

enum : int { ERR_WAIT_FULL = 1, ERR_WAIT_EMPTY = 2, ERR_WAIT_READY = 3, ERR_WAIT_FREE = 4 };

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the cycle budget ran out or the block is aborting.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, volatile int* abort_flag, bool heed_abort) {
    if (heed_abort && *abort_flag) return false;
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (heed_abort && *abort_flag) return false;
        if (clock64() - t0 > WAIT_CYCLES) return false;
    }
}
// The same for a whole warp: lane 0 does the bounded wait and the verdict is broadcast, so the
// warp's control flow stays uniform even when a wait gives up; on success every lane then
// observes the completed phase itself.
__device__ __forceinline__ bool warp_mbar_wait(uint64_t* bar, unsigned parity, volatile int* abort_flag, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, true) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (ok) (void)mbar_try_wait(bar, parity);
    return ok != 0;
}
// One row: global -> shared, completion (in bytes) signalled on `bar`.
__device__ __forceinline__ void bulk_row_copy(void* smem_dst, const void* gmem_src, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

template <typename T, int D, int G, int TILE_N, bool HEADMASK, bool SELECT>
struct PersistCfg : ItemCfg<T, D, G, TILE_N, HEADMASK, SELECT> {
    using Base = ItemCfg<T, D, G, TILE_N, HEADMASK, SELECT>;
    __host__ __device__ static constexpr int list_stride(int chunk) { return (Base::list_bytes(chunk) + 15) / 16 * 16; }
    // dynamic shared memory:
    // [ring: slots x (K tile, V tile)][merge area][row list 0][row list 1][bitmaps][mbarriers][n_rows x 2]
    __host__ static size_t fixed_bytes(int chunk, int bitmap_words) {
        return (size_t)Base::MERGE_BYTES + 2 * (size_t)list_stride(chunk) +
               ((size_t)Base::SLOTS * bitmap_words * 4 + 15) / 16 * 16 + 64;
    }
    __host__ static size_t smem_bytes(int slots, int chunk, int bitmap_words) {
        return (size_t)slots * Base::SLOT_BYTES + 16 * (size_t)slots + fixed_bytes(chunk, bitmap_words);
    }
};

template <typename T, int D, int G, int TILE_N, bool HEADMASK, bool SELECT>
__global__ void __launch_bounds__(NT_PERSIST) dsa_attn_persistent_kernel(const AttnArgs a) {
    using C = PersistCfg<T, D, G, TILE_N, HEADMASK, SELECT>;
    using CSync = NamedSync<NT>;

    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_warp[NT / 32];
    __shared__ int s_abort;
    const int nslot = a.ring_slots;
    unsigned char* ring = smem;
    float* mg = reinterpret_cast<float*>(ring + (size_t)nslot * C::SLOT_BYTES);
    unsigned char* lbase = reinterpret_cast<unsigned char*>(mg) + C::MERGE_BYTES;
    const int lstride = C::list_stride(a.chunk);
    auto list_of = [&](int buf) { return RowList::carve<C>(lbase + buf * lstride, a.chunk); };
    unsigned* bitmaps = reinterpret_cast<unsigned*>(lbase + 2 * lstride);
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(bitmaps) +
                                                 ((size_t)C::SLOTS * a.mask.bitmap_words * 4 + 15) / 16 * 16);
    uint64_t* full = bars;                 // [nslot] tile landed            (1 arrival + bytes)
    uint64_t* empty = bars + nslot;        // [nslot] tile consumed          (4 compute warps)
    uint64_t* ready = bars + 2 * nslot;    // [2] row list written           (compute -> loader)
    uint64_t* lfree = ready + 2;           // [2] row list no longer needed  (loader -> compute)
    volatile int* n_rows_of = reinterpret_cast<volatile int*>(lfree + 2);   // [2]

    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int i = 0; i < nslot; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], NT / 32); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ready[i], 1); mbar_init(&lfree[i], 1); }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();                       // the only block-wide barrier: roles split below

    const int first = blockIdx.x, stride = gridDim.x;
    const int n_my = first < a.n_items ? (a.n_items - first + stride - 1) / stride : 0;
    volatile int* abortp = &s_abort;
    auto fail = [&](int code) {
        if (*abortp == 0) {
            *abortp = 1;
            if (a.error_flag) atomicCAS(a.error_flag, 0, code);
        }
    };

    if (tid >= NT) {
        // ------------------------------------------------------------------ loader warp
        const int lane = tid - NT;
        const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.k);
        const unsigned char* vbase = reinterpret_cast<const unsigned char*>(a.v);
        int slot = 0;
        unsigned phase = 0;
        long long issued = 0;
        bool ok = true;
        for (int i = 0; i < n_my && ok; ++i) {
            const int buf = i & 1;
            if (!warp_mbar_wait(&ready[buf], (unsigned)(i >> 1) & 1u, abortp, lane)) {
                if (lane == 0) fail(ERR_WAIT_READY);
                ok = false;
                break;
            }
            const int n_rows = n_rows_of[buf];
            const RowList list = list_of(buf);
            for (int row0 = 0; row0 < n_rows; row0 += TILE_N) {
                if (!warp_mbar_wait(&empty[slot], phase ^ 1u, abortp, lane)) {
                    if (lane == 0) fail(ERR_WAIT_EMPTY);
                    ok = false;
                    break;
                }
                const int rows_here = min(TILE_N, n_rows - row0);
                if (lane == 0) mbar_arrive_expect_tx(&full[slot], (unsigned)(2 * rows_here * C::ROW_BYTES));
                __syncwarp();
                unsigned char* sb = ring + (size_t)slot * C::SLOT_BYTES;
                for (int j = lane; j < 2 * rows_here; j += 32) {
                    const bool is_v = j >= rows_here;
                    const int row = is_v ? j - rows_here : j;
                    const int64_t off = list.rowoff[row0 + row] * (int64_t)sizeof(T);
                    bulk_row_copy(sb + (is_v ? C::TILE_BYTES : 0) + row * C::ROW_BYTES,
                                  (is_v ? vbase : kbase) + off, C::ROW_BYTES, &full[slot]);
                }
                ++issued;
                if (++slot == nslot) { slot = 0; phase ^= 1u; }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&lfree[buf]);
        }
        if (!ok) {
            // Leaving early: wait (bounded, ignoring the abort flag) until the copies already
            // issued have landed, so that nothing writes into this block's shared memory later.
            const long long back = issued < nslot ? issued : nslot;
            int s = slot;
            unsigned ph = phase;
            if (lane == 0) {
                for (long long n = 0; n < back; ++n) {
                    if (--s < 0) { s = nslot - 1; ph ^= 1u; }
                    if (!mbar_wait(&full[s], ph, abortp, false)) break;
                }
            }
            __syncwarp();
        }
        return;
    }

    // ---------------------------------------------------------------------- compute warps
    const int lane = tid & 31;
    auto decode = [&](int w, int& b, int& kvh, int& split) {
        kvh = w % a.H_kv;
        split = (w / a.H_kv) % a.n_split;
        b = w / (a.H_kv * a.n_split);
    };
    if (n_my == 0) return;
    int b, kvh, split, n_cur;
    decode(first, b, kvh, split);
    ReqMask m = req_mask_setup(a.mask, a.seq_len[b], a.prompt_len[b], a.max_seq_len);
    n_cur = build_row_list<C, CSync>(a, m, b, kvh, split, list_of(0), bitmaps, s_warp);
    CSync::sync();
    if (tid == 0) { n_rows_of[0] = n_cur; mbar_arrive(&ready[0]); }

    int slot = 0;
    unsigned phase = 0;
    for (int i = 0; i < n_my; ++i) {
        const int buf = i & 1;
        // the next item's row list, while the loader streams this item's tiles
        int nb = 0, nkvh = 0, nsplit = 0, n_next = 0;
        ReqMask m_next = m;
        if (i + 1 < n_my) {
            const int nbuf = buf ^ 1;
            // (a wait that gives up does not change the control flow: see the header comment)
            if (i + 1 >= 2 && !warp_mbar_wait(&lfree[nbuf], (unsigned)(((i + 1) >> 1) - 1) & 1u, abortp, lane))
                fail(ERR_WAIT_FREE);
            decode(first + (i + 1) * stride, nb, nkvh, nsplit);
            m_next = req_mask_setup(a.mask, a.seq_len[nb], a.prompt_len[nb], a.max_seq_len);
            n_next = build_row_list<C, CSync>(a, m_next, nb, nkvh, nsplit, list_of(nbuf), bitmaps, s_warp);
            CSync::sync();
            if (tid == 0) { n_rows_of[nbuf] = n_next; mbar_arrive(&ready[nbuf]); }
        }
        if (n_cur <= 0) {
            write_empty_item<C>(a, m, b, kvh, split);
        } else {
            ItemState<C> st;
            st.init(a, b, kvh);
            const int cand_lo = m.L_p + a.mask.n_sink;
            const RowList list = list_of(buf);
            for (int row0 = 0; row0 < n_cur; row0 += TILE_N) {
                if (!warp_mbar_wait(&full[slot], phase, abortp, lane)) fail(ERR_WAIT_FULL);
                const unsigned char* ks = ring + (size_t)slot * C::SLOT_BYTES;
                st.tile(ks, ks + C::TILE_BYTES, row0, n_cur, list, cand_lo);
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[slot]);
                if (++slot == nslot) { slot = 0; phase ^= 1u; }
            }
            st.template finish<CSync>(a, m, b, kvh, split, mg);
            CSync::sync();                    // merge area and this item's row list are free again
        }
        b = nb; kvh = nkvh; split = nsplit; n_cur = n_next; m = m_next;
    }
}

}  // namespace dsa
