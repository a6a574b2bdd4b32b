// The small kernels around attention: split combine, K/V append, seq_len advance and the debug
// export of the kept positions.  Included by dsa_api.cu only (two of them are not templates).
#pragma once
#include "dsa_tile.cuh"

namespace dsa {

// ---- split combine: one block per (request, query head), one thread per output element -------
// Launch with n_split * 4 bytes of dynamic shared memory.
// With sel_k != nullptr it also finishes Algorithm 1's selection: the lowest candidate logit over
// the splits (equal logits: the oldest key, i.e. the largest distance) becomes trace entry sel_k.
template <typename T>
__global__ void dsa_combine_kernel(const float* __restrict__ out_part, const float* __restrict__ lse_part,
                                   int D, int n_split, void* out, float* lse,
                                   const float* __restrict__ sel_val_part = nullptr,
                                   const int* __restrict__ sel_off_part = nullptr,
                                   const int* __restrict__ sel_k = nullptr, int* trace = nullptr,
                                   int trace_len = 0, unsigned* skip_bitmap = nullptr, int bitmap_words = 0,
                                   int window = 0) {
    // launched behind an attention kernel with programmatic serialisation: wait for that grid
    // and its writes (returns at once after an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // Dynamic shared memory: n_split weights.  The lse values are loaded once, in parallel, the
    // maximum and the sum are block reductions, and the weighted sum then reads the partial
    // outputs with independent loads: no chain of dependent global loads as long as n_split.
    extern __shared__ float s_w[];
    __shared__ float s_red[32];
    const int64_t row = blockIdx.x;
    const float* lp = lse_part + row * n_split;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = (nthr + 31) >> 5;
    auto block_reduce = [&](float v, bool is_max) -> float {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            const float o = __shfl_xor_sync(0xffffffffu, v, off);
            v = is_max ? fmaxf(v, o) : v + o;
        }
        __syncthreads();                                 // s_red free again
        if (lane == 0) s_red[warp] = v;
        __syncthreads();
        float r = s_red[0];
        for (int w = 1; w < nwarp; ++w) r = is_max ? fmaxf(r, s_red[w]) : r + s_red[w];
        return r;
    };
    float mx = -INFINITY;
    for (int i = tid; i < n_split; i += nthr) {
        const float v = lp[i];
        s_w[i] = v;
        mx = fmaxf(mx, v);
    }
    const float M = block_reduce(mx, true);
    float part = 0.f;
    for (int i = tid; i < n_split; i += nthr) {          // each thread revisits the entries it wrote
        const float v = s_w[i];
        const float w = (v == -INFINITY || M == -INFINITY) ? 0.f : expf(v - M);
        s_w[i] = w;
        part += w;
    }
    const float den = block_reduce(part, false);         // (its barriers also publish s_w)
    const float inv = den > 0.f ? 1.f / den : 0.f;
    for (int d = tid; d < D; d += nthr) {
        float num = 0.f;
        const float* op = out_part + row * n_split * D + d;
#pragma unroll 4
        for (int i = 0; i < n_split; ++i) {
            const float w = s_w[i];
            if (w != 0.f) num = fmaf(w, op[(int64_t)i * D], num);   // an empty part's out_i is not read
        }
        Elem<T>::store(out, row * D + d, num * inv);
    }
    if (tid == 0 && lse) lse[row] = den > 0.f ? M + logf(den) : -INFINITY;
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
            if (skip_bitmap && bo >= 0 && bo < window)         // (the caller's bitmap form of the list, kept in step)
                atomicOr(&skip_bitmap[row * bitmap_words + (bo >> 5)], 1u << (bo & 31));
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
    // the attention kernel of this decode step may be scheduled behind this grid right away; it
    // waits for this grid's writes before it reads anything
    asm volatile("griddepcontrol.launch_dependents;");
    const int b = blockIdx.x;
    const int S = a.seq_len[b];
    if (S < 0 || S >= capacity) return;                   // no room: the token is dropped
    const int L_p = max(0, min(req_prompt_len(a, b), S));
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

// ---- the bitmap form of the skip lists (dsa_build_skip_bitmap): one block per (request, mask head) sets
// the bits of the head's first n_act entries and clears the rest of its row
__global__ void dsa_build_skip_bitmap_kernel(const AttnArgs a) {
    const int b = blockIdx.x / a.mask.mask_heads;
    const ReqMask m = req_mask_setup(a.mask, a.seq_len[b], req_prompt_len(a, b), a.max_seq_len);
    unsigned* row = a.mask.skip_bitmap + (int64_t)blockIdx.x * a.mask.bitmap_words;
    const int* trace = a.mask.skip_offsets + (int64_t)blockIdx.x * a.mask.trace_len;
    for (int i = threadIdx.x; i < a.mask.bitmap_words; i += blockDim.x) row[i] = 0u;
    __syncthreads();
    const int n_act = m.keep_all ? 0 : m.n_act;
    for (int i = threadIdx.x; i < n_act; i += blockDim.x) {
        const int o = trace[i];
        if (o >= 0 && o < a.mask.window) atomicOr(&row[o >> 5], 1u << (o & 31));
    }
}

// One warp waits, bounded, on an mbarrier that nobody ever arrives on: the wait runs out, the warp
// counts it and the kernel ends (what the attention kernels do when a tile never lands).
__global__ void dsa_wait_giveup_kernel(int* wait_timeouts) {
    __shared__ __align__(8) unsigned long long bar;
    const int lane = threadIdx.x & 31;
    if (lane == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    bool gave_up = false;
    mbar_wait_bounded(&bar, 0u, gave_up, wait_timeouts, lane);
}

// ---- seq_len[b] += 1 (not beyond the limit): once per decode step, after the last layer's fused step.
// A plain launch that does not signal early: everything queued behind it sees the new lengths.
__global__ void dsa_advance_seq_len_kernel(int* seq_len, int batch, int limit) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch && seq_len[b] >= 0 && seq_len[b] < limit) seq_len[b] += 1;
}

// ---- debug export of the kept positions: one block per (request, mask head) ------------------
__global__ void __launch_bounds__(NT) dsa_kept_indices_kernel(const AttnArgs a, int* idx_out, int* count_out,
                                                              int max_kept) {
    extern __shared__ __align__(16) unsigned bitmap[];
    __shared__ int s_warp[NT / 32];
    const int mheads = a.mask.mode == MODE_LIST ? a.mask.mask_heads : 1;
    const int mh = blockIdx.x % mheads, b = blockIdx.x / mheads;
    bool has_new;                                         // (the rows were appended by an earlier kernel)
    const ReqMask m = req_mask_setup(a.mask, step_seq_len(a, a.seq_len[b], has_new), req_prompt_len(a, b), a.max_seq_len);
    if (a.mask.mode == MODE_LIST && !m.keep_all) {
        for (int i = threadIdx.x; i < a.mask.bitmap_words; i += NT) bitmap[i] = 0u;
        __syncthreads();
        const int* trace = a.mask.skip_offsets + ((int64_t)b * mheads + mh) * a.mask.trace_len;
        list_bitmap_fill<NT>(a.mask, m, trace, bitmap);
        __syncthreads();
    }
    int* dst = idx_out + (int64_t)blockIdx.x * max_kept;
    auto write_pos = [&](int slot, int pos, unsigned) { dst[slot] = pos; };
    enumerate_direct<NT, 1>(m, 0, max_kept, write_pos);
    const int total = enumerate_scanned<NT, 1, BlockSync>(a.mask, m, bitmap, 0, max_kept, s_warp, write_pos);
    if (threadIdx.x == 0) count_out[blockIdx.x] = total;
}

}  // namespace dsa
