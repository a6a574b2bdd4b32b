// Split-KV decode attention, one thread block per work item (request, kv head, split).
//
// 128 threads.  Preamble: the mask generator writes the element offsets of the kept K/V rows of
// this split into shared memory.  Main loop: tiles of TILE_N rows are staged with 16-byte cp.async
// copies into a STAGES-deep ring (K and V of a tile travel together) and consumed as they land.
// Tiles are small (a few KB) so that many blocks share an SM and overlap each other's start-up
// and merge phases.
#pragma once
#include "dsa_tile.cuh"

namespace dsa {

template <typename T, int D, int G, int TILE_N, int STAGES, bool HEADMASK, bool SELECT = false>
struct AttnCfg : ItemCfg<T, D, G, TILE_N, HEADMASK, SELECT> {
    using Base = ItemCfg<T, D, G, TILE_N, HEADMASK, SELECT>;
    static constexpr int PIPE_BYTES = STAGES * Base::SLOT_BYTES;
    __host__ __device__ static constexpr int big_bytes() {
        return PIPE_BYTES > Base::MERGE_BYTES ? PIPE_BYTES : Base::MERGE_BYTES;
    }
    // dynamic shared memory: [pipeline / merge area][row list][bitmaps]
    __host__ static size_t smem_bytes(int chunk, int bitmap_words) {
        return (size_t)big_bytes() + Base::list_bytes(chunk) + (size_t)Base::SLOTS * bitmap_words * 4;
    }
};

template <typename T, int D, int G, int TILE_N, int STAGES, bool HEADMASK, bool SELECT>
__global__ void __launch_bounds__(NT) dsa_attn_kernel(const AttnArgs a) {
    using C = AttnCfg<T, D, G, TILE_N, STAGES, HEADMASK, SELECT>;
    constexpr int LPR = C::LPR, VEC = C::VEC;

    // Programmatic launch on both sides: a combine kernel queued behind this grid may be scheduled
    // from now on (it waits for this grid to finish before it reads anything), and this grid may
    // itself have been scheduled early behind the append kernel of the same decode step: wait for
    // that kernel's writes (the new K/V rows, seq_len) before touching global memory.
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_warp[NT / 32];
    unsigned char* pipe = smem;
    const RowList list = RowList::carve<C>(smem + C::big_bytes(), a.chunk);
    unsigned* bitmaps = reinterpret_cast<unsigned*>(smem + C::big_bytes() + C::list_bytes(a.chunk));

    const int tid = threadIdx.x;
    // kv head varies fastest across the grid: the blocks that run together read the same tokens
    // of neighbouring heads, i.e. neighbouring memory.
    const int kvh = blockIdx.x % a.H_kv;
    const int split = (blockIdx.x / a.H_kv) % a.n_split;
    const int b = blockIdx.x / (a.H_kv * a.n_split);

    bool has_new;                                         // (the rows were appended by an earlier kernel)
    const ReqMask m = req_mask_setup(a.mask, step_seq_len(a, a.seq_len[b], has_new), req_prompt_len(a, b), a.max_seq_len);
    const int n_rows = build_row_list<C, BlockSync>(a, m, b, kvh, split, list, bitmaps, s_warp);
    if (n_rows <= 0) { write_empty_item<C>(a, m, b, kvh, split); return; }
    __syncthreads();

    // ---- staging ---------------------------------------------------------------------------
    const int n_tiles = (n_rows + TILE_N - 1) / TILE_N;
    const T* kbase = reinterpret_cast<const T*>(a.k);
    const T* vbase = reinterpret_cast<const T*>(a.v);
    auto issue_tile = [&](int tile) {
        if (tile < n_tiles) {
            unsigned char* ks = pipe + (tile % STAGES) * C::SLOT_BYTES;
            unsigned char* vs = ks + C::TILE_BYTES;
#pragma unroll
            for (int i = 0; i < TILE_N * LPR / NT; ++i) {
                const int idx = i * NT + tid;
                const int row = idx / LPR, c = idx % LPR;
                const int r = tile * TILE_N + row;
                const bool valid = r < n_rows;
                const int64_t off = valid ? list.rowoff[r] + c * VEC : 0;
                cp_async16(ks + row * C::ROW_BYTES + c * 16, kbase + off, valid);
                cp_async16(vs + row * C::ROW_BYTES + c * 16, vbase + off, valid);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) issue_tile(s);

    ItemState<C> st;
    st.init(a, b, kvh);
    const int cand_lo = m.L_p + a.mask.n_sink;

    for (int tile = 0; tile < n_tiles; ++tile) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();                      // tile `tile` landed; everyone is done with tile-1
        issue_tile(tile + STAGES - 1);        // refill the slot tile-1 used
        const unsigned char* ks = pipe + (tile % STAGES) * C::SLOT_BYTES;
        st.tile(ks, ks + C::TILE_BYTES, tile * TILE_N, n_rows, list, cand_lo);
    }
    cp_async_wait<0>();
    __syncthreads();                          // pipeline memory is free: reuse it for the merge
    st.template finish<BlockSync>(a, m, b, kvh, split, reinterpret_cast<float*>(pipe));
}

}  // namespace dsa
