// One work item = the kept rows of one (request, kv head, split).  This header holds what both
// attention kernels do with it: build its row list with the mask generator, consume staged K/V
// tiles (scores, online softmax, PV, phase-2 selection candidates), merge the lane groups and
// write the result.  How tiles get into shared memory is the kernels' business.
//
// Compute layout: LPR = row bytes / 16 lanes hold one 16-byte piece of a row each, so a warp
// reads 32/LPR whole rows per shared-memory instruction.  Every lane group keeps its own
// online-softmax state (running max, sum, fp32 accumulator slice) for each of the G query heads
// that share the kv head; the groups are merged once per item.  Logits are kept in base 2
// (q is pre-multiplied by sm_scale * log2 e) so that the exponentials are single ex2 instructions.
#pragma once
#include "dsa_common.cuh"

namespace dsa {

template <typename T_, int D_, int G_, int TILE_N_, bool HEADMASK_, bool SELECT_>
struct ItemCfg {
    using T = T_;
    static constexpr int D = D_, G = G_, TILE_N = TILE_N_;
    static constexpr bool HEADMASK = HEADMASK_, SELECT = SELECT_;
    static constexpr int VEC = Elem<T>::VEC;
    static constexpr int LPR = D / VEC;                 // lanes per row
    static constexpr int NG = NT / LPR;                 // lane groups per block
    static constexpr int R = TILE_N / NG;               // rows per group per tile
    static constexpr int ROW_BYTES = D * (int)sizeof(T);
    static constexpr int TILE_BYTES = TILE_N * ROW_BYTES;
    static constexpr int SLOT_BYTES = 2 * TILE_BYTES;   // K tile then V tile
    static constexpr int MSTRIDE = D + 4;               // merge record: acc[D], m, l, best logit, its position
    static constexpr int MERGE_BYTES = NG * G * MSTRIDE * 4;
    static constexpr int SLOTS = HEADMASK ? G : 1;      // masks evaluated per row
    static_assert(LPR <= 32 && TILE_N % NG == 0 && R >= 1, "bad tiling");
    // bytes of one row list of `chunk` rows: offsets, positions (selection), head bits
    __host__ __device__ static constexpr int list_bytes(int chunk) {
        return chunk * 8 + (SELECT ? chunk * 4 : 0) + (HEADMASK ? ((chunk + 15) / 16) * 16 : 0);
    }
};

struct RowList {
    int64_t* rowoff;        // element offset of every kept row (kv head included)
    int* rowpos;            // its logical cache position (selection only)
    unsigned char* hbits;   // which heads of the group keep it (per-head masks only)
    template <class C>
    __device__ static RowList carve(unsigned char* base, int chunk) {
        RowList l;
        l.rowoff = reinterpret_cast<int64_t*>(base);
        l.rowpos = reinterpret_cast<int*>(l.rowoff + chunk);
        l.hbits = reinterpret_cast<unsigned char*>(l.rowpos + (C::SELECT ? chunk : 0));
        return l;
    }
};

// Mask generator -> row list of split `split`, in two phases so that a kernel can start streaming
// the rows of phase A while phase B is still being computed.  All NTHR threads that work on the
// item call both.
//
// Phase A: the rows whose position needs no scan (prompt, old sinks, an unmasked window).  Writes
// their final element offsets and returns how many there are; they are rows [0, n) of the list.
// The caller synchronises before anyone reads them.
template <class C, int NTHR = NT>
__device__ __forceinline__ int build_rows_direct(const AttnArgs& a, const ReqMask& m, int b, int kvh, int split,
                                                 const RowList& list) {
    const int r0 = split * a.chunk, r1 = r0 + a.chunk;
    const int64_t head_off = (int64_t)kvh * a.stride_head;
    return enumerate_direct<NTHR, C::SLOTS>(m, r0, r1, [&](int slot, int pos, unsigned bits) {
        list.rowoff[slot] = token_offset(a, b, m.L_p, pos) + head_off;
        if (C::SELECT) list.rowpos[slot] = pos;
        if (C::HEADMASK) list.hbits[slot] = (unsigned char)bits;
    });
}

// Phase B: the window under a mask (rows [n_direct, n_rows) of the list).  Returns n_rows, the
// number of rows of the whole split.  The caller synchronises before anyone reads the new rows.
template <class C, class Sync, int NTHR = NT>
__device__ __forceinline__ int build_rows_scanned(const AttnArgs& a, const ReqMask& m, int b, int kvh, int split,
                                                  const RowList& list, unsigned* bitmaps, int* s_warp,
                                                  int n_direct) {
    const int tid = threadIdx.x;
    const int r0 = split * a.chunk, r1 = r0 + a.chunk;
    if (m.keep_all) return n_direct;
    if (r0 >= m.prefix + m.n_win) return n_direct;            // beyond anything a mask could keep
    if (a.mask.mode == MODE_LIST) {
        Sync::sync();                                     // bitmaps of a previous use are done with
        for (int i = tid; i < C::SLOTS * a.mask.bitmap_words; i += NTHR) bitmaps[i] = 0u;
        Sync::sync();
#pragma unroll
        for (int s = 0; s < C::SLOTS; ++s) {
            const int h = kvh * C::G + s;
            const int mh = a.mask.mask_heads == 1 ? 0 : (a.mask.mask_heads == a.H_kv ? kvh : h);
            const int* trace = a.mask.skip_offsets + ((int64_t)b * a.mask.mask_heads + mh) * a.mask.trace_len;
            list_bitmap_fill<NTHR>(a.mask, m, trace, bitmaps + s * a.mask.bitmap_words);
        }
        Sync::sync();
    }
    // Pass 1: the kept positions (nothing but integer work and shared-memory stores).
    const int total = enumerate_scanned<NTHR, C::SLOTS, Sync>(a.mask, m, bitmaps, r0, r1, s_warp,
        [&](int slot, int pos, unsigned bits) {
            list.rowoff[slot] = pos;
            if (C::SELECT) list.rowpos[slot] = pos;
            if (C::HEADMASK) list.hbits[slot] = (unsigned char)bits;
        });
    const int n_rows = max(0, min(total - r0, a.chunk));
    Sync::sync();
    // Pass 2: positions -> element offsets.  The block-table lookups of different rows are
    // independent loads (neighbouring rows mostly hit the same table entries), so they overlap
    // instead of queueing behind one another as they would inside the scan.
    const int64_t head_off = (int64_t)kvh * a.stride_head;
#pragma unroll 4
    for (int i = n_direct + tid; i < n_rows; i += NTHR)
        list.rowoff[i] = token_offset(a, b, m.L_p, (int)list.rowoff[i]) + head_off;
    return n_rows;
}

// Both phases back to back.
template <class C, class Sync, int NTHR = NT>
__device__ __forceinline__ int build_row_list(const AttnArgs& a, const ReqMask& m, int b, int kvh, int split,
                                              const RowList& list, unsigned* bitmaps, int* s_warp) {
    const int n_direct = build_rows_direct<C, NTHR>(a, m, b, kvh, split, list);
    return build_rows_scanned<C, Sync, NTHR>(a, m, b, kvh, split, list, bitmaps, s_warp, n_direct);
}

// Nothing kept in this split: lse = -inf (and out = 0 when this item owns the result).
// Called by the NTHR threads that own the item; `tid` is the caller's index among them.
template <class C, int NTHR = NT>
__device__ __forceinline__ void write_empty_item(const AttnArgs& a, const ReqMask& m, int b, int kvh, int split,
                                                 int tid = threadIdx.x) {
    using T = typename C::T;
    if (a.n_split > 1) {
        if (tid < C::G) {
            const int64_t row = (int64_t)b * a.H_q + kvh * C::G + tid;
            a.lse_part[row * a.n_split + split] = -INFINITY;
            if (C::SELECT) {
                a.sel_val_part[row * a.n_split + split] = INFINITY;
                a.sel_off_part[row * a.n_split + split] = -1;
                a.sel_k[row] = m.sel_k;
            }
        }
    } else {
        for (int i = tid; i < C::G * C::D; i += NTHR)
            Elem<T>::store(a.out, ((int64_t)b * a.H_q + kvh * C::G) * C::D + i, 0.f);
        if (tid < C::G) a.lse[(int64_t)b * a.H_q + kvh * C::G + tid] = -INFINITY;
        if (C::SELECT && tid < C::G && m.sel_k >= 0)
            a.mask.skip_offsets[((int64_t)b * a.H_q + kvh * C::G + tid) * a.mask.trace_len + m.sel_k] = -1;
    }
}

// Per-thread state of one work item.
template <class C>
struct ItemState {
    using T = typename C::T;
    static constexpr int G = C::G, VEC = C::VEC, LPR = C::LPR, NG = C::NG, R = C::R, D = C::D;
    float qf[G][VEC];
    float acc[G][VEC], mrun[G], lrun[G];
    float bestv[G];       // selection: lowest logit among the attended decode keys that are not sinks
    int bestp[G];         // and its position
    int lr, gid;

    __device__ __forceinline__ void init(const AttnArgs& a, int b, int kvh) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        lr = lane % LPR;                                   // which 16 bytes of a row
        gid = warp * (32 / LPR) + lane / LPR;              // lane group
        const T* qb = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.H_q + kvh * G) * D + lr * VEC;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint4 raw = *reinterpret_cast<const uint4*>(qb + g * D);
            Elem<T>::unpack(raw, qf[g]);
#pragma unroll
            for (int e = 0; e < VEC; ++e) qf[g][e] *= a.scale_log2;
            bestv[g] = INFINITY; bestp[g] = 0x7fffffff;
            mrun[g] = -INFINITY; lrun[g] = 0.f;
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[g][e] = 0.f;
        }
    }

    // One staged tile: rows row0 .. row0 + TILE_N - 1 of the list (rows >= n_rows are not there;
    // their shared memory may hold anything).
    __device__ __forceinline__ void tile(const unsigned char* ks, const unsigned char* vs, int row0, int n_rows,
                                         const RowList& list, int cand_lo) {
        constexpr unsigned ALLBITS = (1u << C::SLOTS) - 1u;
        float s[G * R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = i * NG + gid;
            const uint4 raw = *reinterpret_cast<const uint4*>(ks + row * C::ROW_BYTES + lr * 16);
            float kf[VEC];
            Elem<T>::unpack(raw, kf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float d = 0.f;
#pragma unroll
                for (int e = 0; e < VEC; ++e) d = fmaf(qf[g][e], kf[e], d);
                s[g * R + i] = d;
            }
        }
        // reduce over the lanes of the group, in batches of at most LPR values
        constexpr int VB = (G * R) < LPR ? (G * R) : LPR;
#pragma unroll
        for (int v0 = 0; v0 < G * R; v0 += VB) {
            float tmp[VB];
#pragma unroll
            for (int j = 0; j < VB; ++j) tmp[j] = s[v0 + j];
            group_sum_all<VB, LPR>(tmp, lr);
#pragma unroll
            for (int j = 0; j < VB; ++j) s[v0 + j] = tmp[j];
        }
        // rows past the end of the list, and heads that do not keep a row, get -inf
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int r = row0 + i * NG + gid;
            const bool valid = r < n_rows;
            unsigned bits = ALLBITS;
            if (C::HEADMASK) bits = valid ? list.hbits[r] : 0u;
            int pos = 0;
            if (C::SELECT) pos = valid ? list.rowpos[r] : 0;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const bool on = valid && (!C::HEADMASK || ((bits >> g) & 1u));
                if (!on) s[g * R + i] = -INFINITY;
                // rows arrive in ascending position, so a strict "<" keeps the oldest of equal logits
                if (C::SELECT && on && pos >= cand_lo && s[g * R + i] < bestv[g]) {
                    bestv[g] = s[g * R + i]; bestp[g] = pos;
                }
            }
        }
        // online softmax update, then s becomes the weights p
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float mt = s[g * R];
#pragma unroll
            for (int i = 1; i < R; ++i) mt = fmaxf(mt, s[g * R + i]);
            const float mnew = fmaxf(mrun[g], mt);
            const float msafe = mnew == -INFINITY ? 0.f : mnew;
            const float corr = fast_exp2(mrun[g] - msafe);        // exp2(-inf) = 0
            float psum = 0.f;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                const float p = fast_exp2(s[g * R + i] - msafe);
                s[g * R + i] = p;
                psum += p;
            }
            lrun[g] = lrun[g] * corr + psum;
            mrun[g] = mnew;
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[g][e] *= corr;
        }
        // acc += p * v   (a missing row is skipped: its weight is 0 but its bytes may be NaN)
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = i * NG + gid;
            if (row0 + row < n_rows) {
                const uint4 raw = *reinterpret_cast<const uint4*>(vs + row * C::ROW_BYTES + lr * 16);
                float vf[VEC];
                Elem<T>::unpack(raw, vf);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float p = s[g * R + i];
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[g][e] = fmaf(p, vf[e], acc[g][e]);
                }
            }
        }
    }

    // Merge the lane groups through `mg` (MERGE_BYTES of shared memory nobody else is using) and
    // write the item's result.  Sync covers the NT compute threads.
    template <class Sync>
    __device__ __forceinline__ void finish(const AttnArgs& a, const ReqMask& m, int b, int kvh, int split, float* mg) {
        constexpr int MS = C::MSTRIDE;
        const int tid = threadIdx.x;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float* dst = mg + ((int64_t)gid * G + g) * MS;
#pragma unroll
            for (int e = 0; e < VEC; ++e) dst[lr * VEC + e] = acc[g][e];
            if (lr == 0) {
                dst[D] = mrun[g]; dst[D + 1] = lrun[g];
                if (C::SELECT) { dst[D + 2] = bestv[g]; dst[D + 3] = __int_as_float(bestp[g]); }
            }
        }
        Sync::sync();
        for (int i = tid; i < G * D; i += NT) {
            const int g = i / D, d = i - g * D;
            float M = -INFINITY;
#pragma unroll
            for (int j = 0; j < NG; ++j) M = fmaxf(M, mg[((int64_t)j * G + g) * MS + D]);
            float num = 0.f, den = 0.f;
            if (M != -INFINITY) {
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    const float* src = mg + ((int64_t)j * G + g) * MS;
                    const float w = fast_exp2(src[D] - M);
                    num = fmaf(w, src[d], num);
                    den = fmaf(w, src[D + 1], den);
                }
            }
            const float o = den > 0.f ? num / den : 0.f;
            const float l = den > 0.f ? (M + log2f(den)) * LN2 : -INFINITY;
            const int64_t row = (int64_t)b * a.H_q + kvh * G + g;
            if (a.n_split > 1) {
                a.out_part[(row * a.n_split + split) * D + d] = o;
                if (d == 0) a.lse_part[row * a.n_split + split] = l;
            } else {
                Elem<T>::store(a.out, row * D + d, o);
                if (d == 0) a.lse[row] = l;
            }
            if (C::SELECT && d == 0) {
                // lowest logit over the lane groups; equal logits go to the oldest key
                float bv = INFINITY;
                int bp = 0x7fffffff;
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    const float* src = mg + ((int64_t)j * G + g) * MS;
                    const float v = src[D + 2];
                    const int pp = __float_as_int(src[D + 3]);
                    if (v < bv || (v == bv && pp < bp)) { bv = v; bp = pp; }
                }
                const int off = bp == 0x7fffffff ? -1 : (m.S - 1) - bp;
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
};

}  // namespace dsa
