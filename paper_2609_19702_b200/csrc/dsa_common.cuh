// Shared by all kernels: the argument block, element types, cache addressing, small PTX wrappers.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "dsa_mask.cuh"

namespace dsa {

constexpr int NT = 128;          // compute threads per block (4 warps)
constexpr int MAX_CHUNK = 1024;  // kept rows one work item can hold in its row list (twice that when four warps share it)
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
    int prompt_cap;              // device prompt_len values above this are read as this (see req_prompt_len)
    int ring_size, ring_sinks;   // bounded cache: decode tokens beyond the first ring_sinks live in a ring
    int B, H_q, H_kv;
    float scale_log2;            // sm_scale * log2(e)
    MaskArgs mask;
    int heads_per_warp;          // head-group / per-head-list kernels: kv heads each warp streams back to back
    int dir_cap;                 // per-head-list kernel: capacity of the always-kept-row table (rows)
    int kidx_cap;                //                       and of a head's kept-candidate list (rows)
    int chunk;                   // kept rows per split (multiple of the tile; see MAX_CHUNK)
    int n_split;
    int n_items;                 // B * H_kv * n_split work items
    void* out;                   // n_split == 1: [B, H_q, D] in T
    float* lse;                  //               [B, H_q]
    float* out_part;             // n_split > 1:  [B, H_q, n_split, D]
    float* lse_part;             //               [B, H_q, n_split]
    // phase-2 selection with n_split > 1: per-split candidates, reduced by the combine kernel
    float* sel_val_part;         // [B, H_q, n_split] lowest logit (base 2) among this split's candidates
    int* sel_off_part;           // [B, H_q, n_split] its distance behind the query, -1 if none
    int* sel_k;                  // [B, H_q] trace entry to write, -1 if this request selects nothing
    // fused decode step: the cache holds seq_len[b] tokens and the call appends the token being
    // decoded itself (logical position seq_len[b]) before attending over seq_len[b] + 1 tokens
    int step_append;             // 0: seq_len counts the current token, nothing is appended
    const void* k_new;           // [B, H_kv, D] rows of the current token; NULL: already in the cache
    const void* v_new;
    int* wait_timeouts;          // device counter of bounded mbarrier waits that gave up (0 in a healthy run); may be NULL
    int early_list;              // 1: the caller promises that no launch still running when this kernel starts writes
                                 // seq_len, prompt_len, block_table or the skip lists, so the row list may be built BEFORE
                                 // waiting for the launch in front (programmatic dependent launch); q, the new rows and
                                 // the caches are still read after the wait only
};

// What the tensor-map (gather) kernel needs beyond AttnArgs: the K and V caches as 2-D views
// [token rows][elements of one token row] (boxes of 64 elements x 1 row, 128-byte swizzle).
struct GatherMaps {
    CUtensorMap k, v;
    int rows_per_stride_b;       // token rows between neighbouring pages (paged cache) or requests
    int oob_row;                 // a row index beyond the view: such a row reads as zeros
};

// The prompt length of request b as the kernels use it.  With a bounded cache a request's region
// holds max_prompt_len + ring_sinks + ring_size tokens, so a device value above max_prompt_len is
// cut there: every address derived from it then stays inside the region.
__device__ __forceinline__ int req_prompt_len(const AttnArgs& a, int b) {
    return min(a.prompt_len[b], a.prompt_cap);
}

// Number of tokens request b attends over.  In a fused decode step that is one more than the
// cache holds, unless the request is full (the token is then dropped, as by the append call).
__device__ __forceinline__ int step_seq_len(const AttnArgs& a, int S /* = seq_len[b] */, bool& has_new) {
    has_new = a.step_append != 0 && S >= 0 && S < a.max_seq_len;
    return has_new ? S + 1 : S;
}

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

// 16 bytes global -> shared, asynchronously; with !valid nothing is read and the 16 bytes are zeroed.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src, bool valid) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    const int src_size = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(gmem_src), "r"(src_size));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

// Wait until at most min(n, MAXN) of this thread's cp.async groups are still pending (n >= 0 known
// only at run time; the instruction takes an immediate).
template <int MAXN>
__device__ __forceinline__ void cp_async_wait_upto(int n) {
    if constexpr (MAXN > 0) {
        if (n >= MAXN) cp_async_wait<MAXN>();
        else cp_async_wait_upto<MAXN - 1>(n);
    } else {
        cp_async_wait<0>();
    }
}

// ---- mbarrier helpers (producer / consumer hand-over, tensor-map copies) ------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// one probe of phase `parity` of the barrier (the instruction itself blocks for a bounded time)
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
    unsigned done;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return done != 0;
}
constexpr long long kMbarWaitCycles = 1ll << 31;        // ~1 s: a wait that long gives up (see AttnArgs::wait_timeouts)
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// the barrier gets one arrival from this thread when all cp.async copies it has issued so far have landed
__device__ __forceinline__ void cp_async_arrive_on(unsigned long long* bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Wait for phase `parity` of `bar`, for kMbarWaitCycles at most.  `gave_up` is sticky: once a wait
// has run out the warp does not wait again.
__device__ __forceinline__ void mbar_wait_bounded(unsigned long long* bar, unsigned parity, bool& gave_up,
                                                  int* wait_timeouts, int lane) {
    if (gave_up || mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kMbarWaitCycles) { gave_up = true; break; }
    }
    if (gave_up && lane == 0 && wait_timeouts) atomicAdd(wait_timeouts, 1);
}


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

}  // namespace dsa
