// Split-KV decode attention over the kept rows of one (request, kv head, split).
//
// One thread block = 128 threads.  Preamble: the mask generator writes the element offsets of the
// kept K/V rows of this split into shared memory.  Main loop: tiles of TILE_N rows are staged
// with 16-byte cp.async copies into a STAGES-deep ring (K and V of a tile travel together), and
// consumed by "lane groups": LPR = row bytes / 16 lanes hold one 16-byte piece of a row each, so
// a warp reads 32/LPR whole rows per shared-memory instruction.  Every lane group keeps its own
// online-softmax state (running max, sum, fp32 accumulator slice) for each of the G query heads
// that share the kv head; the groups are merged once at the end.  Logits are kept in base 2
// (q is pre-multiplied by sm_scale * log2 e) so that the exponentials are single ex2 instructions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "dsa_mask.cuh"

namespace dsa {

constexpr int NT = 128;          // threads per block
constexpr int MAX_CHUNK = 1024;  // kept rows one block can hold in its row list
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

struct AttnArgs {
    const void* q;
    const void* k;
    const void* v;
    int64_t stride_b, stride_tok, stride_head;
    const int* seq_len;
    int* seq_len_rw;             // same array, for the append call that advances it
    const int* prompt_len;
    const int* block_table;
    int max_blocks, block_size, num_blocks;
    int max_seq_len;
    int ring_size, ring_sinks;   // bounded cache: decode tokens beyond the first ring_sinks live in a ring
    int B, H_q, H_kv;
    float scale_log2;            // sm_scale * log2(e)
    MaskArgs mask;
    int chunk;                   // kept rows per split (multiple of the tile, <= MAX_CHUNK)
    int n_split;
    void* out;                   // n_split == 1: [B, H_q, D] in T
    float* lse;                  //               [B, H_q]
    float* out_part;             // n_split > 1:  [B, H_q, n_split, D]
    float* lse_part;             //               [B, H_q, n_split]
    // phase-2 selection with n_split > 1: per-split candidates, reduced by the combine kernel
    float* sel_val_part;         // [B, H_q, n_split] lowest logit (base 2) among this split's candidates
    int* sel_off_part;           // [B, H_q, n_split] its distance behind the query, -1 if none
    int* sel_k;                  // [B, H_q] trace entry to write, -1 if this request selects nothing
};

// Where token `pos` (logical cache position) of request b lives, as an element offset of its kv
// head 0.  With a bounded cache (ring_size > 0) the prompt and the first ring_sinks decode tokens
// are stored in order and every later decode token j sits in ring slot (j - ring_sinks) mod
// ring_size behind them: the slot of the token it evicted ring_size steps earlier.
__device__ __forceinline__ int64_t token_offset(const AttnArgs& a, int b, int L_p, int pos) {
    if (a.ring_size > 0) {
        const int first = L_p + a.ring_sinks;
        if (pos >= first) pos = first + (pos - first) % a.ring_size;
    }
    if (a.block_table) {
        const int bi = pos / a.block_size;
        int blk = a.block_table[(int64_t)b * a.max_blocks + min(bi, a.max_blocks - 1)];
        blk = max(0, min(blk, a.num_blocks - 1));
        return (int64_t)blk * a.stride_b + (int64_t)(pos - bi * a.block_size) * a.stride_tok;
    }
    return (int64_t)b * a.stride_b + (int64_t)pos * a.stride_tok;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src, bool valid) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    const int src_size = valid ? 16 : 0;     // 0: nothing is read, the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(gmem_src), "r"(src_size));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static constexpr int VEC = 8;
    __device__ static __forceinline__ void unpack(const uint4& r, float (&f)[8]) {
        const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ static __forceinline__ void store(void* base, int64_t i, float x) {
        reinterpret_cast<__nv_bfloat16*>(base)[i] = __float2bfloat16_rn(x);
    }
};
template <> struct Elem<float> {
    static constexpr int VEC = 4;
    __device__ static __forceinline__ void unpack(const uint4& r, float (&f)[4]) {
        f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
    }
    __device__ static __forceinline__ void store(void* base, int64_t i, float x) {
        reinterpret_cast<float*>(base)[i] = x;
    }
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Sum V values per lane across the LPR lanes of a group; on return every lane holds all V sums.
// Halving exchange: at each step a lane hands half of its values to its partner and keeps the
// other half, so V values cost V - 1 + log2(LPR / V) shuffles instead of V * log2(LPR); a final
// V shuffles hand every sum to every lane.
template <int V, int LPR>
__device__ __forceinline__ void group_sum_all(float (&x)[V], int lr) {
    static_assert(V <= LPR && (V & (V - 1)) == 0, "V must be a power of two <= LPR");
    constexpr unsigned FULL = 0xffffffffu;
    int k = 0;
#pragma unroll
    for (int off = LPR / 2; off >= 1; off >>= 1, ++k) {
        const int cnt = (V >> k) > 1 ? (V >> k) : 1;
        if (cnt > 1) {
            const int half = cnt / 2;
            const bool up = (lr & off) != 0;
#pragma unroll
            for (int j = 0; j < half; ++j) {
                const float send = up ? x[j] : x[j + half];
                const float keep = up ? x[j + half] : x[j];
                x[j] = keep + __shfl_xor_sync(FULL, send, off);
            }
        } else {
            x[0] += __shfl_xor_sync(FULL, x[0], off);
        }
    }
    // lane lr now holds the sum of value lr / (LPR / V) in x[0]
    const float mine = x[0];
#pragma unroll
    for (int v = 0; v < V; ++v) x[v] = __shfl_sync(FULL, mine, v * (LPR / V), LPR);
}

template <typename T, int D, int G, int TILE_N, int STAGES, bool HEADMASK, bool SELECT = false>
struct AttnCfg {
    static constexpr int VEC = Elem<T>::VEC;
    static constexpr int LPR = D / VEC;                 // lanes per row
    static constexpr int NG = NT / LPR;                 // lane groups per block
    static constexpr int R = TILE_N / NG;               // rows per group per tile
    static constexpr int ROW_BYTES = D * (int)sizeof(T);
    static constexpr int TILE_BYTES = TILE_N * ROW_BYTES;
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;  // K tile then V tile
    static constexpr int PIPE_BYTES = STAGES * STAGE_BYTES;
    static constexpr int MSTRIDE = D + 4;               // merge record: acc[D], m, l, best logit, its position
    static constexpr int MERGE_BYTES = NG * G * MSTRIDE * 4;
    static constexpr int SLOTS = HEADMASK ? G : 1;
    static_assert(LPR <= 32 && TILE_N % NG == 0 && R >= 1, "bad tiling");
    __host__ __device__ static constexpr int big_bytes() {
        return PIPE_BYTES > MERGE_BYTES ? PIPE_BYTES : MERGE_BYTES;
    }
    // dynamic shared memory:
    // [pipeline / merge area][row offsets int64 x chunk][row positions int32 x chunk][head bits][bitmaps]
    __host__ static size_t smem_bytes(int chunk, int bitmap_words) {
        size_t b = big_bytes();
        b += (size_t)chunk * 8;
        if (SELECT) b += (size_t)chunk * 4;
        if (HEADMASK) b += (size_t)((chunk + 15) / 16) * 16;
        b += (size_t)SLOTS * bitmap_words * 4;
        return b;
    }
};

template <typename T, int D, int G, int TILE_N, int STAGES, bool HEADMASK, bool SELECT>
__global__ void __launch_bounds__(NT) dsa_attn_kernel(const AttnArgs a) {
    using C = AttnCfg<T, D, G, TILE_N, STAGES, HEADMASK, SELECT>;
    constexpr int VEC = C::VEC, LPR = C::LPR, NG = C::NG, R = C::R, SLOTS = C::SLOTS, MS = C::MSTRIDE;
    constexpr unsigned ALLBITS = (1u << SLOTS) - 1u;

    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_warp[NT / 32];
    unsigned char* pipe = smem;
    int64_t* rowoff = reinterpret_cast<int64_t*>(smem + C::big_bytes());
    int* rowpos = reinterpret_cast<int*>(rowoff + a.chunk);
    unsigned char* hbits = reinterpret_cast<unsigned char*>(rowpos + (SELECT ? a.chunk : 0));
    unsigned* bitmaps = reinterpret_cast<unsigned*>(hbits + (HEADMASK ? ((a.chunk + 15) / 16) * 16 : 0));

    const int tid = threadIdx.x;
    // kv head varies fastest across the grid: the blocks that run together read the same tokens
    // of neighbouring heads, i.e. neighbouring memory.
    const int kvh = blockIdx.x % a.H_kv;
    const int split = (blockIdx.x / a.H_kv) % a.n_split;
    const int b = blockIdx.x / (a.H_kv * a.n_split);

    const ReqMask m = req_mask_setup(a.mask, a.seq_len[b], a.prompt_len[b], a.max_seq_len);
    const int r0 = split * a.chunk, r1 = r0 + a.chunk;

    auto write_empty = [&]() {
        // nothing kept in this split: lse = -inf (and out = 0 when this block owns the result)
        if (a.n_split > 1) {
            if (tid < G) {
                const int64_t row = (int64_t)b * a.H_q + kvh * G + tid;
                a.lse_part[row * a.n_split + split] = -INFINITY;
                if (SELECT) {
                    a.sel_val_part[row * a.n_split + split] = INFINITY;
                    a.sel_off_part[row * a.n_split + split] = -1;
                    a.sel_k[row] = m.sel_k;
                }
            }
        } else {
            for (int i = tid; i < G * D; i += NT)
                Elem<T>::store(a.out, ((int64_t)b * a.H_q + kvh * G) * D + i, 0.f);
            if (tid < G) a.lse[(int64_t)b * a.H_q + kvh * G + tid] = -INFINITY;
            if (SELECT && tid < G && m.sel_k >= 0)
                a.mask.skip_offsets[((int64_t)b * a.H_q + kvh * G + tid) * a.mask.trace_len + m.sel_k] = -1;
        }
    };

    if (m.keep_all && r0 >= m.prefix + m.n_win) { write_empty(); return; }

    // ---- mask generator -> row list -------------------------------------------------------
    if (a.mask.mode == MODE_LIST && !m.keep_all) {
        for (int i = tid; i < SLOTS * a.mask.bitmap_words; i += NT) bitmaps[i] = 0u;
        __syncthreads();
#pragma unroll
        for (int s = 0; s < SLOTS; ++s) {
            const int h = kvh * G + s;
            const int mh = a.mask.mask_heads == 1 ? 0 : (a.mask.mask_heads == a.H_kv ? kvh : h);
            const int* trace = a.mask.skip_offsets + ((int64_t)b * a.mask.mask_heads + mh) * a.mask.trace_len;
            list_bitmap_fill<NT>(a.mask, m, trace, bitmaps + s * a.mask.bitmap_words);
        }
        __syncthreads();
    }
    const int64_t head_off = (int64_t)kvh * a.stride_head;
    const int total = enumerate_kept<NT, SLOTS>(a.mask, m, bitmaps, r0, r1, s_warp,
        [&](int slot, int pos, unsigned bits) {
            rowoff[slot] = token_offset(a, b, m.L_p, pos) + head_off;
            if (SELECT) rowpos[slot] = pos;
            if (HEADMASK) hbits[slot] = (unsigned char)bits;
        });
    const int n_rows = min(total - r0, a.chunk);
    if (n_rows <= 0) { write_empty(); return; }
    __syncthreads();

    // ---- staging ---------------------------------------------------------------------------
    const int n_tiles = (n_rows + TILE_N - 1) / TILE_N;
    const T* kbase = reinterpret_cast<const T*>(a.k);
    const T* vbase = reinterpret_cast<const T*>(a.v);
    auto issue_tile = [&](int tile) {
        if (tile < n_tiles) {
            unsigned char* ks = pipe + (tile % STAGES) * C::STAGE_BYTES;
            unsigned char* vs = ks + C::TILE_BYTES;
#pragma unroll
            for (int i = 0; i < TILE_N * LPR / NT; ++i) {
                const int idx = i * NT + tid;
                const int row = idx / LPR, c = idx % LPR;
                const int r = tile * TILE_N + row;
                const bool valid = r < n_rows;
                const int64_t off = valid ? rowoff[r] + c * VEC : 0;
                cp_async16(ks + row * C::ROW_BYTES + c * 16, kbase + off, valid);
                cp_async16(vs + row * C::ROW_BYTES + c * 16, vbase + off, valid);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) issue_tile(s);

    // ---- per-thread state ------------------------------------------------------------------
    const int lane = tid & 31, warp = tid >> 5;
    const int lr = lane % LPR;                           // which 16 bytes of a row
    const int gid = warp * (32 / LPR) + lane / LPR;      // lane group
    float qf[G][VEC];
    {
        const T* qb = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.H_q + kvh * G) * D + lr * VEC;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint4 raw = *reinterpret_cast<const uint4*>(qb + g * D);
            Elem<T>::unpack(raw, qf[g]);
#pragma unroll
            for (int e = 0; e < VEC; ++e) qf[g][e] *= a.scale_log2;
        }
    }
    // selection: lowest logit among the attended decode keys that are not sinks, per head
    float bestv[G];
    int bestp[G];
    const int cand_lo = m.L_p + a.mask.n_sink;
    float acc[G][VEC], mrun[G], lrun[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        bestv[g] = INFINITY; bestp[g] = 0x7fffffff;
        mrun[g] = -INFINITY; lrun[g] = 0.f;
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[g][e] = 0.f;
    }

    // ---- main loop -------------------------------------------------------------------------
    for (int tile = 0; tile < n_tiles; ++tile) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();                      // tile `tile` landed; everyone is done with tile-1
        issue_tile(tile + STAGES - 1);        // refill the slot tile-1 used

        const unsigned char* ks = pipe + (tile % STAGES) * C::STAGE_BYTES;
        const unsigned char* vs = ks + C::TILE_BYTES;

        // scores of this group's R rows for the G heads
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
            const int r = tile * TILE_N + i * NG + gid;
            const bool valid = r < n_rows;
            unsigned bits = ALLBITS;
            if (HEADMASK) bits = valid ? hbits[r] : 0u;
            int pos = 0;
            if (SELECT) pos = valid ? rowpos[r] : 0;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const bool on = valid && (!HEADMASK || ((bits >> g) & 1u));
                if (!on) s[g * R + i] = -INFINITY;
                // rows arrive in ascending position, so a strict "<" keeps the oldest of equal logits
                if (SELECT && on && pos >= cand_lo && s[g * R + i] < bestv[g]) {
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
        // acc += p * v
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = i * NG + gid;
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
    cp_async_wait<0>();
    __syncthreads();                          // pipeline memory is free: reuse it for the merge

    // ---- merge the lane groups ---------------------------------------------------------------
    float* mg = reinterpret_cast<float*>(pipe);           // [NG][G][MS]: acc, m, l, best logit, its position
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float* dst = mg + ((int64_t)gid * G + g) * MS;
#pragma unroll
        for (int e = 0; e < VEC; ++e) dst[lr * VEC + e] = acc[g][e];
        if (lr == 0) {
            dst[D] = mrun[g]; dst[D + 1] = lrun[g];
            if (SELECT) { dst[D + 2] = bestv[g]; dst[D + 3] = __int_as_float(bestp[g]); }
        }
    }
    __syncthreads();
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
        const int h = kvh * G + g;
        const int64_t row = (int64_t)b * a.H_q + h;
        if (a.n_split > 1) {
            a.out_part[(row * a.n_split + split) * D + d] = o;
            if (d == 0) a.lse_part[row * a.n_split + split] = l;
        } else {
            Elem<T>::store(a.out, row * D + d, o);
            if (d == 0) a.lse[row] = l;
        }
        if (SELECT && d == 0) {
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
                a.mask.skip_offsets[row * a.mask.trace_len + m.sel_k] = off;
            }
        }
    }
}

// ---- split combine: one block per (request, query head), one thread per output element -------
// With sel_k != nullptr it also finishes Algorithm 1's selection: the lowest candidate logit over
// the splits (equal logits: the oldest key, i.e. the largest distance) becomes trace entry sel_k.
template <typename T>
__global__ void dsa_combine_kernel(const float* __restrict__ out_part, const float* __restrict__ lse_part,
                                   int D, int n_split, void* out, float* lse,
                                   const float* __restrict__ sel_val_part = nullptr,
                                   const int* __restrict__ sel_off_part = nullptr,
                                   const int* __restrict__ sel_k = nullptr, int* trace = nullptr,
                                   int trace_len = 0) {
    const int64_t row = blockIdx.x;
    const float* lp = lse_part + row * n_split;
    float M = -INFINITY;
    for (int i = 0; i < n_split; ++i) M = fmaxf(M, lp[i]);
    float den = 0.f;
    if (M != -INFINITY)
        for (int i = 0; i < n_split; ++i) den += lp[i] == -INFINITY ? 0.f : expf(lp[i] - M);
    const float inv = den > 0.f ? 1.f / den : 0.f;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        float num = 0.f;
        if (den > 0.f) {
            for (int i = 0; i < n_split; ++i) {
                const float li = lp[i];
                if (li == -INFINITY) continue;            // empty part: its out_i is not read
                num = fmaf(expf(li - M), out_part[(row * n_split + i) * D + d], num);
            }
        }
        Elem<T>::store(out, row * D + d, num * inv);
    }
    if (threadIdx.x == 0 && lse) lse[row] = den > 0.f ? M + logf(den) : -INFINITY;
    if (threadIdx.x == 0 && sel_k != nullptr) {
        const int k = sel_k[row];
        if (k >= 0) {
            float bv = INFINITY;
            int bo = -1;
            for (int i = 0; i < n_split; ++i) {
                const float v = sel_val_part[row * n_split + i];
                const int o = sel_off_part[row * n_split + i];
                if (o >= 0 && (v < bv || (v == bv && o > bo))) { bv = v; bo = o; }
            }
            trace[row * trace_len + k] = bo;
        }
    }
}

// ---- K/V append: the new token of every request goes to logical position seq_len[b] --------------
// One block per request copies its H_kv rows of K and of V (16-byte pieces) and then, if asked,
// advances seq_len[b]; no other block reads that entry, so the update needs no further ordering.
// k_new / v_new are [B, H_kv, D].
template <typename T>
__global__ void dsa_append_kv_kernel(const AttnArgs a, const T* __restrict__ k_new, const T* __restrict__ v_new,
                                     int D, int capacity, bool advance) {
    const int b = blockIdx.x;
    const int S = a.seq_len[b];
    if (S < 0 || S >= capacity) return;                   // no room: the token is dropped
    const int L_p = max(0, min(a.prompt_len[b], S));
    const int64_t dst0 = token_offset(a, b, L_p, S);
    constexpr int VEC = 16 / (int)sizeof(T);
    T* kc = reinterpret_cast<T*>(const_cast<void*>(a.k));
    T* vc = reinterpret_cast<T*>(const_cast<void*>(a.v));
    const int per_row = D / VEC;
    for (int i = threadIdx.x; i < a.H_kv * per_row; i += blockDim.x) {
        const int kvh = i / per_row, c = (i - kvh * per_row) * VEC;
        const int64_t dst = dst0 + (int64_t)kvh * a.stride_head + c;
        const int64_t src = ((int64_t)b * a.H_kv + kvh) * D + c;
        *reinterpret_cast<uint4*>(kc + dst) = *reinterpret_cast<const uint4*>(k_new + src);
        *reinterpret_cast<uint4*>(vc + dst) = *reinterpret_cast<const uint4*>(v_new + src);
    }
    __syncthreads();                                       // every thread has read S
    if (advance && threadIdx.x == 0) a.seq_len_rw[b] = S + 1;
}

// ---- debug export of the kept positions: one block per (request, mask head) ------------------
__global__ void __launch_bounds__(NT) dsa_kept_indices_kernel(const AttnArgs a, int* idx_out, int* count_out,
                                                              int max_kept) {
    extern __shared__ __align__(16) unsigned bitmap[];
    __shared__ int s_warp[NT / 32];
    const int mheads = a.mask.mode == MODE_LIST ? a.mask.mask_heads : 1;
    const int mh = blockIdx.x % mheads, b = blockIdx.x / mheads;
    const ReqMask m = req_mask_setup(a.mask, a.seq_len[b], a.prompt_len[b], a.max_seq_len);
    if (a.mask.mode == MODE_LIST && !m.keep_all) {
        for (int i = threadIdx.x; i < a.mask.bitmap_words; i += NT) bitmap[i] = 0u;
        __syncthreads();
        const int* trace = a.mask.skip_offsets + ((int64_t)b * mheads + mh) * a.mask.trace_len;
        list_bitmap_fill<NT>(a.mask, m, trace, bitmap);
        __syncthreads();
    }
    int* dst = idx_out + (int64_t)blockIdx.x * max_kept;
    const int total = enumerate_kept<NT, 1>(a.mask, m, bitmap, 0, max_kept, s_warp,
                                            [&](int slot, int pos, unsigned) { dst[slot] = pos; });
    if (threadIdx.x == 0) count_out[blockIdx.x] = total;
}

}  // namespace dsa
