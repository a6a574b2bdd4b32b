// Split-KV decode attention for bf16 caches, persistent form: every warp is a worker that streams
// MANY work items back to back through one cp.async ring that never drains between them.
//
// Why: a work item of the one-launch-per-item kernel (dsa_attn_mma.cuh) spends the start of its life
// with nothing in flight (lengths, mask, row list) and the end of it with the ring running empty.
// For items of ~400 kept rows that is a tenth of the item; for the ~100-row items of a decode loop
// at the paper's shape (50 prompt tokens + N_att 52) it is close to half, and the memory system sees
// correspondingly fewer bytes in flight.  Here the row list of item i+1 is built -- lengths, mask
// generator, block-table lookups, q loads -- while the tiles of item i are in flight, its first tiles
// are issued into the ring slots that item i's last tiles free, and the only bubbles left are one
// start-up and one drain per WARP instead of per item.
//
// Structure.  One warp per thread block (so nothing in the kernel is wider than __syncwarp), a grid
// of as many blocks as the device holds at once, worker w takes items w, w + grid, w + 2 grid, ...
// (kv heads vary fastest across items, so the workers read neighbouring heads of the same tokens at
// about the same time).  Per worker: a ring of STAGES slots (one 16-key K tile + V tile each) and
// TWO row lists, the one being consumed and the one being built.  Row-list entries are 32 bits
// (physical token position, or block id << 8 | token within the block for paged caches), turned
// into addresses when a tile is issued.  Tile consumption is the tensor-core formulation of
// dsa_attn_mma.cuh: S^T = K . Q^T, online softmax on the accumulator fragment, O^T += V^T . P^T.
// Items that keep nothing are answered while the list is built and never enter the ring.
#pragma once
#include "dsa_attn_mma.cuh"

namespace dsa {

template <int D, int G, bool HEADMASK, bool SELECT>
struct StreamCfg {
    using T = __nv_bfloat16;
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int CPR = ROW_BYTES / 16;
    static constexpr int TILE_BYTES = MMA_KEYS * ROW_BYTES;
    static constexpr int SLOT_BYTES = 2 * TILE_BYTES;
    static constexpr int KSTEPS = D / 16;
    static constexpr int MTILES = D / 16;
    static constexpr int SLOTS = HEADMASK ? G : 1;
    // one row list of `chunk` rows: entries, positions (selection), head bits (per-head masks)
    __host__ __device__ static constexpr int list_bytes(int chunk) {
        return chunk * 4 + (SELECT ? chunk * 4 : 0) + (HEADMASK ? ((chunk + 15) / 16) * 16 : 0);
    }
    // dynamic shared memory of a worker: [ring][list 0][list 1][bitmaps]
    __host__ static size_t smem_bytes(int stages, int chunk, int bitmap_words) {
        return (size_t)stages * SLOT_BYTES + 2 * (size_t)list_bytes(chunk) + (size_t)SLOTS * bitmap_words * 4;
    }
};

struct StreamList {
    unsigned* ent;          // where each kept row lives (see token_entry)
    int* rowpos;            // its logical cache position (selection only)
    unsigned char* hbits;   // which heads of the group keep it (per-head masks only)
    template <class C>
    __device__ static StreamList carve(unsigned char* base, int chunk) {
        StreamList l;
        l.ent = reinterpret_cast<unsigned*>(base);
        l.rowpos = reinterpret_cast<int*>(l.ent + chunk);
        l.hbits = reinterpret_cast<unsigned char*>(l.rowpos + (C::SELECT ? chunk : 0));
        return l;
    }
};

// What the worker keeps in registers about an item between building its list and writing its result.
template <int KSTEPS>
struct StreamItem {
    int b, kvh, split;
    int n_rows, n_tiles;
    int S, L_p, sel_k;                    // clamped lengths and the trace entry to append (selection)
    int new_r;                            // fused step: row of the token being decoded in this list, or -1
    int64_t base_bytes;                   // byte offset of the item's kv head (and request, if contiguous)
    int64_t new_bytes;                    // fused step: byte offset of k_new / v_new rows of this item
    unsigned qb[KSTEPS][2];               // Q^T fragment
};

template <int D, int G, int STAGES, bool HEADMASK, bool SELECT, bool APPEND>
__global__ void __launch_bounds__(32) dsa_attn_stream_kernel(const AttnArgs a) {
    using C = StreamCfg<D, G, HEADMASK, SELECT>;
    using IC = MmaItemCfg<D, G, HEADMASK, SELECT>;
    using T = __nv_bfloat16;
    using Item = StreamItem<C::KSTEPS>;
    constexpr unsigned FULL = 0xffffffffu;
    static_assert(STAGES >= 2, "the ring needs a slot in flight beside the one being consumed");

    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_warp[1];
    const int lane = threadIdx.x;
    unsigned char* ring = smem;
    const int lbytes = C::list_bytes(a.chunk);
    unsigned char* list_mem = smem + STAGES * C::SLOT_BYTES;
    unsigned* bitmaps = reinterpret_cast<unsigned*>(list_mem + 2 * lbytes);
    const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.k);
    const unsigned char* vbase = reinterpret_cast<const unsigned char*>(a.v);

    // fragment coordinates (see dsa_attn_mma.cuh)
    const int hq = lane >> 2, qd = (lane & 3) * 2;
    const int hc = (lane & 3) * 2, kr = lane >> 2;
    const int lm_row_k = (lane & 7) + ((lane >> 3) & 1) * 8, lm_chk_k = lane >> 4;
    const int lm_row_v = (lane & 7) + (lane >> 4) * 8, lm_chk_v = (lane >> 3) & 1;

    int next_item = blockIdx.x;                       // next item this worker will build

    // ---- build: the row list of the next non-empty item into list buffer `buf` --------------------
    // Returns false when the worker has no item left.  Items that keep nothing get their (empty)
    // result written here and are skipped.
    auto build_next = [&](int buf, Item& it) -> bool {
        const StreamList list = StreamList::carve<C>(list_mem + buf * lbytes, a.chunk);
        while (next_item < a.n_items) {
            const int item = next_item;
            next_item += gridDim.x;
            it.kvh = item % a.H_kv;
            const int rest = item / a.H_kv;
            it.split = rest % a.n_split;
            it.b = rest / a.n_split;
            const int b = it.b, kvh = it.kvh, split = it.split;
            const int seq_raw = a.seq_len[b], prompt_raw = req_prompt_len(a, b);
            {
                const T* qrow = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.H_q + kvh * G + (hq < G ? hq : 0)) * D;
#pragma unroll
                for (int kk = 0; kk < C::KSTEPS; ++kk) {
                    const unsigned q0 = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd);
                    const unsigned q1 = *reinterpret_cast<const unsigned*>(qrow + kk * 16 + qd + 8);
                    it.qb[kk][0] = hq < G ? q0 : 0u;
                    it.qb[kk][1] = hq < G ? q1 : 0u;
                }
            }
            bool has_new = false;
            const int S_step = APPEND ? step_seq_len(a, seq_raw, has_new) : seq_raw;
            const ReqMask m = req_mask_setup(a.mask, S_step, prompt_raw, a.max_seq_len);
            it.S = m.S; it.L_p = m.L_p; it.sel_k = m.sel_k;
            it.base_bytes = ((int64_t)kvh * a.stride_head + (a.block_table ? 0 : (int64_t)b * a.stride_b)) * 2;
            it.new_r = -1;
            it.new_bytes = ((int64_t)b * a.H_kv + kvh) * C::ROW_BYTES;
            unsigned new_ent = 0u;
            if (APPEND && has_new) {
                new_ent = token_entry(a, b, m.L_p, m.S - 1);
                if (split == 0 && lane < 2 * C::CPR) {
                    // the token being decoded goes to the cache: lanes [0, CPR) K chunks, [CPR, 2 CPR) V chunks
                    const bool is_k = lane < C::CPR;
                    const int c = is_k ? lane : lane - C::CPR;
                    const unsigned char* src = reinterpret_cast<const unsigned char*>(is_k ? a.k_new : a.v_new) +
                                               it.new_bytes + c * 16;
                    unsigned char* dst = const_cast<unsigned char*>(is_k ? kbase : vbase) + it.base_bytes +
                                         entry_bytes(a, new_ent) + c * 16;
                    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
                }
            }
            const int r0 = split * a.chunk, r1 = r0 + a.chunk;
            __syncwarp();                                  // the list buffer is free (its last reader was this warp)
            const int n_direct = enumerate_direct<32, C::SLOTS>(m, r0, r1, [&](int slot, int pos, unsigned bits) {
                list.ent[slot] = token_entry(a, b, m.L_p, pos);
                if (SELECT) list.rowpos[slot] = pos;
                if (HEADMASK) list.hbits[slot] = (unsigned char)bits;
            });
            int n_rows = n_direct;
            if (!m.keep_all && r0 < m.prefix + m.n_win) {
                if (a.mask.mode == MODE_LIST) {
                    for (int i = lane; i < C::SLOTS * a.mask.bitmap_words; i += 32) bitmaps[i] = 0u;
                    __syncwarp();
#pragma unroll
                    for (int s = 0; s < C::SLOTS; ++s) {
                        const int h = kvh * G + s;
                        const int mh = a.mask.mask_heads == 1 ? 0 : (a.mask.mask_heads == a.H_kv ? kvh : h);
                        const int* trace = a.mask.skip_offsets + ((int64_t)b * a.mask.mask_heads + mh) * a.mask.trace_len;
                        list_bitmap_fill<32>(a.mask, m, trace, bitmaps + s * a.mask.bitmap_words);
                    }
                    __syncwarp();
                }
                const int total = enumerate_scanned<32, C::SLOTS, WarpSync>(a.mask, m, bitmaps, r0, r1, s_warp,
                    [&](int slot, int pos, unsigned bits) {
                        list.ent[slot] = (unsigned)pos;
                        if (SELECT) list.rowpos[slot] = pos;
                        if (HEADMASK) list.hbits[slot] = (unsigned char)bits;
                    });
                n_rows = max(0, min(total - r0, a.chunk));
                __syncwarp();
                // positions -> entries (independent block-table lookups, so they overlap)
#pragma unroll 4
                for (int i = n_direct + lane; i < n_rows; i += 32)
                    list.ent[i] = token_entry(a, b, m.L_p, (int)list.ent[i]);
            }
            __syncwarp();
            if (n_rows <= 0) {
                write_empty_item<IC, 32>(a, m, b, kvh, split, lane);
                continue;
            }
            it.n_rows = n_rows;
            it.n_tiles = (n_rows + MMA_KEYS - 1) / MMA_KEYS;
            // kept positions ascend, so the token being decoded can only be the item's last row
            if (APPEND && has_new && list.ent[n_rows - 1] == new_ent) it.new_r = n_rows - 1;
            return true;
        }
        return false;
    };

    // ---- issue: tile `tile` of item `it` (list buffer `buf`) into ring slot `slot` ------------------
    auto issue_tile = [&](const Item& it, int buf, int tile, int slot) {
        const StreamList list = StreamList::carve<C>(list_mem + buf * lbytes, a.chunk);
        unsigned char* ks = ring + slot * C::SLOT_BYTES;
        unsigned char* vs = ks + C::TILE_BYTES;
        const int row0 = tile * MMA_KEYS;
#pragma unroll
        for (int i = 0; i < MMA_KEYS * C::CPR / 32; ++i) {
            const int idx = i * 32 + lane;
            const int row = idx / C::CPR, c = idx % C::CPR;
            const int r = row0 + row;
            const bool valid = r < it.n_rows;
            const int dst = row * C::ROW_BYTES + ((c ^ (row & 7)) * 16);
            if (APPEND && r == it.new_r) {
                cp_async16(ks + dst, reinterpret_cast<const unsigned char*>(a.k_new) + it.new_bytes + c * 16, true);
                cp_async16(vs + dst, reinterpret_cast<const unsigned char*>(a.v_new) + it.new_bytes + c * 16, true);
            } else {
                const int64_t off = valid ? it.base_bytes + entry_bytes(a, list.ent[r]) + c * 16 : 0;
                cp_async16(ks + dst, kbase + off, valid);
                cp_async16(vs + dst, vbase + off, valid);
            }
        }
    };

    Item cur, nxt;
    cur.n_tiles = 0; cur.n_rows = 0;
    bool cur_valid = false, nxt_valid = false;
    int cur_buf = 0;
    int cur_issued = 0, nxt_issued = 0;                // tiles of cur / nxt already in the ring
    int islot = 0, cslot = 0;                          // ring slot of the next issue / the next consume

    // One ring step on the producer side: the next tile of cur, else of nxt, else an empty group (the
    // group count per consumed tile stays fixed, so wait_group<STAGES - 2> always means "oldest tile").
    auto issue_one = [&]() {
        if (cur_valid && cur_issued < cur.n_tiles) {
            issue_tile(cur, cur_buf, cur_issued, islot);
            ++cur_issued;
        } else if (nxt_valid && nxt_issued < nxt.n_tiles) {
            issue_tile(nxt, cur_buf ^ 1, nxt_issued, islot);
            ++nxt_issued;
        }
        cp_async_commit();
        islot = islot + 1 == STAGES ? 0 : islot + 1;
    };

    nxt_valid = build_next(1, nxt);
#pragma unroll 1
    for (int s = 0; s < STAGES - 1; ++s) issue_one();

    // per-item accumulation state
    float o[C::MTILES][4];
    float mrun[2], lpart[2], bestv[2];
    int bestp[2];

#pragma unroll 1
    while (true) {
        // ---- the current item is done (or there was none yet): write it, move on to the next --------
        if (cur_valid) {
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
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float l = ltot[j];
                const int h = hc + j;
                if (h < G) {
                    const float inv = l > 0.f ? 1.f / l : 0.f;
                    const float lse = l > 0.f ? (mrun[j] + log2f(l)) * LN2 : -INFINITY;
                    const int64_t row = (int64_t)cur.b * a.H_q + cur.kvh * G + h;
#pragma unroll
                    for (int mt = 0; mt < C::MTILES; ++mt) {
                        const int d0 = mt * 16 + kr;
                        if (a.n_split > 1) {
                            float* dst = a.out_part + (row * a.n_split + cur.split) * D;
                            dst[d0] = o[mt][j] * inv;
                            dst[d0 + 8] = o[mt][2 + j] * inv;
                        } else {
                            T* dst = reinterpret_cast<T*>(a.out) + row * D;
                            dst[d0] = __float2bfloat16_rn(o[mt][j] * inv);
                            dst[d0 + 8] = __float2bfloat16_rn(o[mt][2 + j] * inv);
                        }
                    }
                    if (kr == 0) {
                        if (a.n_split > 1) a.lse_part[row * a.n_split + cur.split] = lse;
                        else a.lse[row] = lse;
                        if (SELECT) {
                            const int off = bp[j] == 0x7fffffff ? -1 : (cur.S - 1) - bp[j];
                            if (a.n_split > 1) {
                                a.sel_val_part[row * a.n_split + cur.split] = bv[j];
                                a.sel_off_part[row * a.n_split + cur.split] = off;
                                a.sel_k[row] = cur.sel_k;
                            } else if (cur.sel_k >= 0) {
                                a.mask.skip_offsets[row * a.mask.trace_len + cur.sel_k] = off;
                            }
                        }
                    }
                }
            }
        }
        if (!nxt_valid) break;
        cur = nxt;
        cur_valid = true;
        cur_buf ^= 1;
        cur_issued = nxt_issued;
        nxt_issued = 0;
        // The ring now holds the first tiles of the new current item: build the list of the one after
        // it while they are in flight.
        nxt_valid = build_next(cur_buf ^ 1, nxt);

#pragma unroll
        for (int mt = 0; mt < C::MTILES; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
        mrun[0] = mrun[1] = -INFINITY;
        lpart[0] = lpart[1] = 0.f;
        bestv[0] = bestv[1] = INFINITY;
        bestp[0] = bestp[1] = 0x7fffffff;
        const int cand_lo = cur.L_p + a.mask.n_sink;
        const StreamList list = StreamList::carve<C>(list_mem + cur_buf * lbytes, a.chunk);
        const int n_rows = cur.n_rows;

#pragma unroll 1
        for (int tile = 0; tile < cur.n_tiles; ++tile) {
            cp_async_wait<STAGES - 2>();
            __syncwarp();                               // the oldest tile landed for every lane; the slot before it is free
            issue_one();
            const unsigned char* ks = ring + cslot * C::SLOT_BYTES;
            const unsigned char* vs = ks + C::TILE_BYTES;
            cslot = cslot + 1 == STAGES ? 0 : cslot + 1;

            // S^T = K . Q^T
            float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kk = 0; kk < C::KSTEPS; ++kk) {
                unsigned af[4];
                const int chunk = kk * 2 + lm_chk_k;
                ldmatrix_x4(af, ks + lm_row_k * C::ROW_BYTES + ((chunk ^ (lm_row_k & 7)) * 16));
                mma_bf16_16816(s, af, cur.qb[kk][0], cur.qb[kk][1]);
            }
            const int r0 = tile * MMA_KEYS + kr, r1 = r0 + 8;
            const bool v0 = r0 < n_rows, v1 = r1 < n_rows;
            unsigned bits0 = 0xffu, bits1 = 0xffu;
            if (HEADMASK) { bits0 = v0 ? list.hbits[r0] : 0u; bits1 = v1 ? list.hbits[r1] : 0u; }
            int pos0 = 0, pos1 = 0;
            if (SELECT) { pos0 = v0 ? list.rowpos[r0] : 0; pos1 = v1 ? list.rowpos[r1] : 0; }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
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
            const unsigned pb0 = movmatrix_trans(pack_bf16x2(s[0], s[1]));
            const unsigned pb1 = movmatrix_trans(pack_bf16x2(s[2], s[3]));
#pragma unroll
            for (int mt = 0; mt < C::MTILES; ++mt) {
                unsigned af[4];
                const int chunk = mt * 2 + lm_chk_v;
                ldmatrix_x4_trans(af, vs + lm_row_v * C::ROW_BYTES + ((chunk ^ (lm_row_v & 7)) * 16));
                mma_bf16_16816(o[mt], af, pb0, pb1);
            }
        }
    }
    cp_async_wait<0>();
}

}  // namespace dsa
