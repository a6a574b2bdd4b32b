// Kernel selection and launch for one (element type, head_dim): included by the per-type
// translation units (dsa_kernels_*.cu), which instantiate kernel_shape / kernel_launch.
#pragma once
#include "dsa_attn.cuh"
#include "dsa_attn_mma.cuh"
#include "dsa_attn_gather.cuh"
#include "dsa_attn_group_ws.cuh"
#include "dsa_attn_group.cuh"
#include "dsa_attn_heads.cuh"
#include "dsa_launch.cuh"

#include <atomic>
#include <type_traits>

namespace dsa {

// Launch `kern` so that it may be scheduled before the kernel queued ahead of it on the stream has
// finished (programmatic stream serialisation).  Every kernel launched this way starts with
// griddepcontrol.wait, which holds it until that earlier grid has completed and its writes are
// visible; after a kernel that never signals early this is an ordinary serialised launch.
template <class Kern, class... Args>
cudaError_t launch_pdl(Kern kern, unsigned grid, unsigned block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

// The same with a thread-block cluster of `cluster` blocks along x (grid must be a multiple of it).
template <class Kern, class... Args>
cudaError_t launch_pdl_cluster(Kern kern, unsigned grid, unsigned block, size_t smem, cudaStream_t st, unsigned cluster,
                               Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

template <typename T, int D, int G, bool HM, bool SEL>
struct KernelPick {
    // Small tiles (2 KB of K + 2 KB of V) in a 4-deep ring: 16-20 KB of shared memory per block, so
    // 8 or more blocks share an SM and their start-up and merge phases overlap each other's
    // streaming.  (Measured on the paged batch-256 workload: 32-row tiles with 3 blocks/SM reach
    // 5.7 TB/s, these reach 6.6 TB/s; the dense call is flat at 7.2 TB/s either way.)
    static constexpr int TILE = 2048 / (D * (int)sizeof(T));
    static constexpr int STAGES = 4;
    using Cfg = AttnCfg<T, D, G, TILE, STAGES, HM, SEL>;
    static size_t smem(int chunk, int bw) { return Cfg::smem_bytes(chunk, bw); }
    // Tensor-core kernel (bf16 only).  W warps per block share one row list when the mask does not
    // depend on the head (never with per-head masks or selection).
    // The two-heads-per-block form also exists with a shallower ring (kMmaStagesShallow): more
    // blocks per SM, for launches that would otherwise spill a little into another wave.
    template <int W, int ST = kMmaStages>
    static size_t smem_mma_w(int chunk, int bw) { return MmaCfg<D, G, ST, HM, SEL, W>::smem_bytes(chunk, bw); }
    static size_t smem_mma(int w, int kw, int stages, int chunk, int bw) {
        if (kw > 1) return smem_mma_w<kMmaItemWarps>(chunk, bw);      // one ring per warp either way
        if constexpr (!HM && !SEL) {
            if (w == 2) return stages == kMmaStagesShallow ? smem_mma_w<2, kMmaStagesShallow>(chunk, bw)
                                                           : smem_mma_w<2>(chunk, bw);
        }
        return smem_mma_w<1>(chunk, bw);
    }
    // Kernels that use more than 48 KB of dynamic shared memory must be told so once per device.
    // The per-device flags are idempotent caches (configuring twice is harmless), kept atomic so
    // that host threads may make their first calls at the same time.
    using ConfiguredFlags = std::atomic<bool>;
    template <class Kern>
    static cudaError_t ensure_configured(Kern kern, ConfiguredFlags* done /* [kMaxDevices] */) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices || !done[dev].load(std::memory_order_acquire)) {
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < kMaxDevices) done[dev].store(true, std::memory_order_release);
        }
        return cudaSuccess;
    }
    template <int W, bool APPEND, int KW, int ST>
    static ConfiguredFlags* mma_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }
    template <bool APPEND, int CL, bool EARLY = false>
    static ConfiguredFlags* cluster_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }
    template <bool APPEND>
    static ConfiguredFlags* kw_early_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }
    // several warps per item, CL blocks of a cluster per item (head-independent masks only)
    template <bool APPEND, int CL>
    static cudaError_t launch_cluster_c(const AttnArgs& a, int64_t items, size_t smem_bytes, cudaStream_t st) {
        if constexpr (sizeof(T) == 2 && !HM && !SEL) {
            if (a.early_list) {                         // (row list before the dependency wait)
                auto kern = dsa_attn_mma_kernel<D, G, kMmaStages, HM, SEL, 1, APPEND, kMmaItemWarps, CL, true>;
                const cudaError_t e = ensure_configured(kern, cluster_configured<APPEND, CL, true>());
                if (e != cudaSuccess) return e;
                return launch_pdl_cluster(kern, (unsigned)(items * CL), 32 * kMmaItemWarps, smem_bytes, st, CL, a);
            }
            auto kern = dsa_attn_mma_kernel<D, G, kMmaStages, HM, SEL, 1, APPEND, kMmaItemWarps, CL>;
            const cudaError_t e = ensure_configured(kern, cluster_configured<APPEND, CL>());
            if (e != cudaSuccess) return e;
            return launch_pdl_cluster(kern, (unsigned)(items * CL), 32 * kMmaItemWarps, smem_bytes, st, CL, a);
        } else {
            return cudaErrorInvalidValue;
        }
    }
    static cudaError_t launch_cluster(int cl, bool append, const AttnArgs& a, int64_t items, size_t smem_bytes,
                                      cudaStream_t st) {
        if (cl == 4) return append ? launch_cluster_c<true, 4>(a, items, smem_bytes, st) : launch_cluster_c<false, 4>(a, items, smem_bytes, st);
        return append ? launch_cluster_c<true, 2>(a, items, smem_bytes, st) : launch_cluster_c<false, 2>(a, items, smem_bytes, st);
    }
    static ConfiguredFlags* cc_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }

    template <int W, bool APPEND, int KW, int ST = kMmaStages>
    static cudaError_t launch_mma_w(const AttnArgs& a, int64_t grid, size_t smem_bytes, cudaStream_t st) {
        auto kern = dsa_attn_mma_kernel<D, G, ST, HM, SEL, W, APPEND, KW>;
        const cudaError_t e = ensure_configured(kern, mma_configured<W, APPEND, KW, ST>());
        if (e != cudaSuccess) return e;
        return launch_pdl(kern, (unsigned)grid, 32 * W * KW, smem_bytes, st, a);
    }
    // Head-group tensor-core kernel (bf16, masks that do not depend on the head): blocks of W warps,
    // one row list per block; rings of kGroupStages slots, or kGroupStagesShallow for more blocks per SM.
    template <int W, int ST>
    static size_t smem_group_w(int chunk, int bw) { return GroupCfg<D, W, ST>::smem_bytes(chunk, bw); }
    static size_t smem_group(int w, int stages, int chunk, int bw) {
        if (stages == kGroupStagesShallow)
            return w == 4 ? smem_group_w<4, kGroupStagesShallow>(chunk, bw) : smem_group_w<2, kGroupStagesShallow>(chunk, bw);
        return w == 4 ? smem_group_w<4, kGroupStages>(chunk, bw) : smem_group_w<2, kGroupStages>(chunk, bw);
    }
    template <int W, bool APPEND, int ST, bool EARLY = false, bool COPY_ONLY = false>
    static ConfiguredFlags* group_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }
    template <int W, bool APPEND, int ST>
    static cudaError_t launch_group_w(const AttnArgs& a, int64_t blocks, size_t smem_bytes, cudaStream_t st,
                                      bool copy_only = false) {
        if constexpr (sizeof(T) == 2 && !HM && !SEL) {
            if constexpr (W == 4 && !APPEND) {
                if (copy_only) {                        // (the measuring form: dsa_debug_copy_only)
                    auto kern = dsa_attn_group_kernel<D, G, ST, 4, false, false, true>;
                    const cudaError_t e = ensure_configured(kern, group_configured<4, false, ST, false, true>());
                    if (e != cudaSuccess) return e;
                    return launch_pdl(kern, (unsigned)blocks, 32 * 4, smem_bytes, st, a);
                }
            }
            if (W == 4 && a.early_list) {               // (the early-list form exists for four-warp blocks)
                auto kern = dsa_attn_group_kernel<D, G, ST, 4, APPEND, true>;
                const cudaError_t e = ensure_configured(kern, group_configured<4, APPEND, ST, true>());
                if (e != cudaSuccess) return e;
                return launch_pdl(kern, (unsigned)blocks, 32 * 4, smem_bytes, st, a);
            }
            auto kern = dsa_attn_group_kernel<D, G, ST, W, APPEND>;
            const cudaError_t e = ensure_configured(kern, group_configured<W, APPEND, ST>());
            if (e != cudaSuccess) return e;
            return launch_pdl(kern, (unsigned)blocks, 32 * W, smem_bytes, st, a);
        } else {
            return cudaErrorInvalidValue;
        }
    }
    template <int ST>
    static cudaError_t launch_group_s(int w, bool append, const AttnArgs& a, int64_t blocks, size_t smem_bytes,
                                      cudaStream_t st, bool copy_only) {
        if (copy_only && (w != 4 || append)) return cudaErrorInvalidValue;
        if (w == 4) return append ? launch_group_w<4, true, ST>(a, blocks, smem_bytes, st)
                                  : launch_group_w<4, false, ST>(a, blocks, smem_bytes, st, copy_only);
        return append ? launch_group_w<2, true, ST>(a, blocks, smem_bytes, st)
                      : launch_group_w<2, false, ST>(a, blocks, smem_bytes, st);
    }
    static cudaError_t launch_group(int w, int stages, bool append, const AttnArgs& a, int64_t blocks,
                                    size_t smem_bytes, cudaStream_t st, bool copy_only) {
        return stages == kGroupStagesShallow
                   ? launch_group_s<kGroupStagesShallow>(w, append, a, blocks, smem_bytes, st, copy_only)
                   : launch_group_s<kGroupStages>(w, append, a, blocks, smem_bytes, st, copy_only);
    }
    // The same with tensor-map gather copies (four-warp blocks).
    static size_t smem_gather(int stages, int chunk, int bw) {
        return stages == kGroupStagesShallow ? GatherCfg<D, 4, kGroupStagesShallow>::smem_bytes(chunk, bw)
                                             : GatherCfg<D, 4, kGroupStages>::smem_bytes(chunk, bw);
    }
    template <bool APPEND, int ST>
    static ConfiguredFlags* gather_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }
    template <bool APPEND, int ST>
    static cudaError_t launch_gather_s(const AttnArgs& a, const GatherMaps& maps, int64_t blocks, size_t smem_bytes,
                                       cudaStream_t st) {
        if constexpr (sizeof(T) == 2 && !HM && !SEL) {
            auto kern = dsa_attn_gather_kernel<D, G, ST, 4, APPEND>;
            const cudaError_t e = ensure_configured(kern, gather_configured<APPEND, ST>());
            if (e != cudaSuccess) return e;
            return launch_pdl(kern, (unsigned)blocks, 32 * 4, smem_bytes, st, a, maps);
        } else {
            return cudaErrorInvalidValue;
        }
    }
    static cudaError_t launch_gather(int stages, bool append, const AttnArgs& a, const GatherMaps* maps, int64_t blocks,
                                     size_t smem_bytes, cudaStream_t st) {
        if (!maps) return cudaErrorInvalidValue;
        if (stages == kGroupStagesShallow)
            return append ? launch_gather_s<true, kGroupStagesShallow>(a, *maps, blocks, smem_bytes, st)
                          : launch_gather_s<false, kGroupStagesShallow>(a, *maps, blocks, smem_bytes, st);
        return append ? launch_gather_s<true, kGroupStages>(a, *maps, blocks, smem_bytes, st)
                      : launch_gather_s<false, kGroupStages>(a, *maps, blocks, smem_bytes, st);
    }
    // The same with a producer warp per ring (four consumer + four producer warps; the shared memory of
    // the plain four-warp form).
    template <bool APPEND, int ST>
    static ConfiguredFlags* ws_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }
    template <bool APPEND, int ST>
    static cudaError_t launch_ws_s(const AttnArgs& a, int64_t blocks, size_t smem_bytes, cudaStream_t st) {
        if constexpr (sizeof(T) == 2 && !HM && !SEL) {
            auto kern = dsa_attn_group_ws_kernel<D, G, ST, 4, APPEND>;
            const cudaError_t e = ensure_configured(kern, ws_configured<APPEND, ST>());
            if (e != cudaSuccess) return e;
            return launch_pdl(kern, (unsigned)blocks, 64 * 4, smem_bytes, st, a);
        } else {
            return cudaErrorInvalidValue;
        }
    }
    static cudaError_t launch_ws(int stages, bool append, const AttnArgs& a, int64_t blocks, size_t smem_bytes,
                                 cudaStream_t st) {
        if (stages == kGroupStagesShallow)
            return append ? launch_ws_s<true, kGroupStagesShallow>(a, blocks, smem_bytes, st)
                          : launch_ws_s<false, kGroupStagesShallow>(a, blocks, smem_bytes, st);
        return append ? launch_ws_s<true, kGroupStages>(a, blocks, smem_bytes, st)
                      : launch_ws_s<false, kGroupStages>(a, blocks, smem_bytes, st);
    }
    // Per-head-list tensor-core kernel (bf16, list masks per kv or query head, fused selection).
    static size_t smem_heads(int dir_cap, int window, int kidx_cap, int bw) {
        return HeadsCfg<D, G, kMmaStages, kHeadsWarps, HM>::smem_bytes(dir_cap, window, kidx_cap, bw);
    }
    template <bool APPEND, bool EARLY = false>
    static ConfiguredFlags* heads_configured() { static ConfiguredFlags done[kMaxDevices] = {}; return done; }
    template <bool APPEND>
    static cudaError_t launch_heads_a(const AttnArgs& a, int64_t blocks, size_t smem_bytes, cudaStream_t st) {
        if constexpr (sizeof(T) == 2) {
            if (a.early_list) {
                auto kern = dsa_attn_heads_kernel<D, G, kMmaStages, kHeadsWarps, HM, SEL, APPEND, true>;
                const cudaError_t e = ensure_configured(kern, heads_configured<APPEND, true>());
                if (e != cudaSuccess) return e;
                return launch_pdl(kern, (unsigned)blocks, 32 * kHeadsWarps, smem_bytes, st, a);
            }
            auto kern = dsa_attn_heads_kernel<D, G, kMmaStages, kHeadsWarps, HM, SEL, APPEND>;
            const cudaError_t e = ensure_configured(kern, heads_configured<APPEND>());
            if (e != cudaSuccess) return e;
            return launch_pdl(kern, (unsigned)blocks, 32 * kHeadsWarps, smem_bytes, st, a);
        } else {
            return cudaErrorInvalidValue;
        }
    }
    static cudaError_t launch_heads(bool append, const AttnArgs& a, int64_t blocks, size_t smem_bytes, cudaStream_t st) {
        return append ? launch_heads_a<true>(a, blocks, smem_bytes, st) : launch_heads_a<false>(a, blocks, smem_bytes, st);
    }
    // Configure every kernel of this variant for the current device (see dsa_prepare).
    static cudaError_t prepare() {
        cudaError_t e = ensure_configured(dsa_attn_kernel<T, D, G, TILE, STAGES, HM, SEL>, cc_configured());
        if constexpr (sizeof(T) == 2) {
            auto mma = [&](auto w, auto app, auto kw, auto stg) {
                constexpr int W = decltype(w)::value, KW = decltype(kw)::value, ST = decltype(stg)::value;
                constexpr bool APPEND = decltype(app)::value;
                if (e == cudaSuccess)
                    e = ensure_configured(dsa_attn_mma_kernel<D, G, ST, HM, SEL, W, APPEND, KW>,
                                          mma_configured<W, APPEND, KW, ST>());
            };
            if (e == cudaSuccess)
                e = ensure_configured(dsa_attn_heads_kernel<D, G, kMmaStages, kHeadsWarps, HM, SEL, false>, heads_configured<false>());
            if (e == cudaSuccess)
                e = ensure_configured(dsa_attn_heads_kernel<D, G, kMmaStages, kHeadsWarps, HM, SEL, true>, heads_configured<true>());
            if (e == cudaSuccess)
                e = ensure_configured(dsa_attn_heads_kernel<D, G, kMmaStages, kHeadsWarps, HM, SEL, false, true>, heads_configured<false, true>());
            if (e == cudaSuccess)
                e = ensure_configured(dsa_attn_heads_kernel<D, G, kMmaStages, kHeadsWarps, HM, SEL, true, true>, heads_configured<true, true>());
            using one = std::integral_constant<int, 1>;
            using two = std::integral_constant<int, 2>;
            using four = std::integral_constant<int, kMmaItemWarps>;
            using deep = std::integral_constant<int, kMmaStages>;
            using shallow = std::integral_constant<int, kMmaStagesShallow>;
            mma(one{}, std::false_type{}, one{}, deep{});
            mma(one{}, std::true_type{}, one{}, deep{});
            mma(one{}, std::false_type{}, four{}, deep{});
            mma(one{}, std::true_type{}, four{}, deep{});
            if (e == cudaSuccess)
                e = ensure_configured(dsa_attn_mma_kernel<D, G, kMmaStages, HM, SEL, 1, false, kMmaItemWarps, 1, true>,
                                      kw_early_configured<false>());
            if (e == cudaSuccess)
                e = ensure_configured(dsa_attn_mma_kernel<D, G, kMmaStages, HM, SEL, 1, true, kMmaItemWarps, 1, true>,
                                      kw_early_configured<true>());
            if constexpr (!HM && !SEL) {
                auto cluster = [&](auto app, auto cl) {
                    constexpr bool APPEND = decltype(app)::value;
                    constexpr int CL = decltype(cl)::value;
                    if (e == cudaSuccess)
                        e = ensure_configured(dsa_attn_mma_kernel<D, G, kMmaStages, HM, SEL, 1, APPEND, kMmaItemWarps, CL>,
                                              cluster_configured<APPEND, CL>());
                };
                auto cluster_early = [&](auto app, auto cl) {
                    constexpr bool APPEND = decltype(app)::value;
                    constexpr int CL = decltype(cl)::value;
                    if (e == cudaSuccess)
                        e = ensure_configured(dsa_attn_mma_kernel<D, G, kMmaStages, HM, SEL, 1, APPEND, kMmaItemWarps, CL, true>,
                                              cluster_configured<APPEND, CL, true>());
                };
                cluster_early(std::false_type{}, two{});
                cluster_early(std::true_type{}, two{});
                cluster_early(std::false_type{}, four{});
                cluster_early(std::true_type{}, four{});
                cluster(std::false_type{}, two{});
                cluster(std::true_type{}, two{});
                cluster(std::false_type{}, four{});
                cluster(std::true_type{}, four{});
                auto group = [&](auto w, auto app, auto stg) {
                    constexpr int W = decltype(w)::value, ST = decltype(stg)::value;
                    constexpr bool APPEND = decltype(app)::value;
                    if (e == cudaSuccess)
                        e = ensure_configured(dsa_attn_group_kernel<D, G, ST, W, APPEND>, group_configured<W, APPEND, ST>());
                    if constexpr (W == 4) {
                        if (e == cudaSuccess)
                            e = ensure_configured(dsa_attn_group_kernel<D, G, ST, 4, APPEND, true>,
                                                  group_configured<4, APPEND, ST, true>());
                    }
                };
                using gdeep = std::integral_constant<int, kGroupStages>;
                using gshallow = std::integral_constant<int, kGroupStagesShallow>;
                group(two{}, std::false_type{}, gdeep{});
                group(two{}, std::true_type{}, gdeep{});
                group(four{}, std::false_type{}, gdeep{});
                group(four{}, std::true_type{}, gdeep{});
                group(two{}, std::false_type{}, gshallow{});
                group(two{}, std::true_type{}, gshallow{});
                group(four{}, std::false_type{}, gshallow{});
                group(four{}, std::true_type{}, gshallow{});
                auto gather = [&](auto app, auto stg) {
                    constexpr int ST = decltype(stg)::value;
                    constexpr bool APPEND = decltype(app)::value;
                    if (e == cudaSuccess)
                        e = ensure_configured(dsa_attn_gather_kernel<D, G, ST, 4, APPEND>, gather_configured<APPEND, ST>());
                };
                auto ws = [&](auto app, auto stg) {
                    constexpr int ST = decltype(stg)::value;
                    constexpr bool APPEND = decltype(app)::value;
                    if (e == cudaSuccess)
                        e = ensure_configured(dsa_attn_group_ws_kernel<D, G, ST, 4, APPEND>, ws_configured<APPEND, ST>());
                };
                ws(std::false_type{}, gdeep{});
                ws(std::true_type{}, gdeep{});
                ws(std::false_type{}, gshallow{});
                ws(std::true_type{}, gshallow{});
                gather(std::false_type{}, gdeep{});
                gather(std::true_type{}, gdeep{});
                gather(std::false_type{}, gshallow{});
                gather(std::true_type{}, gshallow{});
                mma(two{}, std::false_type{}, one{}, deep{});
                mma(two{}, std::true_type{}, one{}, deep{});
                mma(two{}, std::false_type{}, one{}, shallow{});
                mma(two{}, std::true_type{}, one{}, shallow{});
            }
        }
        return e;
    }
    // `append`: the fused decode step (the kernel reads the current token from a.k_new / a.v_new)
    template <bool APPEND>
    static cudaError_t launch_mma_a(int w, int kw, int stages, const AttnArgs& a, int64_t items, size_t smem_bytes,
                                    cudaStream_t st) {
        if constexpr (sizeof(T) == 2) {
            if (kw > 1 && a.early_list) {               // (row list before the dependency wait)
                auto kern = dsa_attn_mma_kernel<D, G, kMmaStages, HM, SEL, 1, APPEND, kMmaItemWarps, 1, true>;
                const cudaError_t e = ensure_configured(kern, kw_early_configured<APPEND>());
                if (e != cudaSuccess) return e;
                return launch_pdl(kern, (unsigned)items, 32 * kMmaItemWarps, smem_bytes, st, a);
            }
            if (kw > 1) return launch_mma_w<1, APPEND, kMmaItemWarps>(a, items, smem_bytes, st);
            if constexpr (!HM && !SEL) {
                if (w == 2 && stages == kMmaStagesShallow)
                    return launch_mma_w<2, APPEND, 1, kMmaStagesShallow>(a, items / 2, smem_bytes, st);
                if (w == 2) return launch_mma_w<2, APPEND, 1>(a, items / 2, smem_bytes, st);
            }
            return launch_mma_w<1, APPEND, 1>(a, items, smem_bytes, st);
        } else {
            return cudaErrorInvalidValue;
        }
    }
    static cudaError_t launch_mma(int w, int kw, int stages, const AttnArgs& a, int64_t items, size_t smem_bytes,
                                  cudaStream_t st, bool append) {
        return append ? launch_mma_a<true>(w, kw, stages, a, items, smem_bytes, st)
                      : launch_mma_a<false>(w, kw, stages, a, items, smem_bytes, st);
    }
    static cudaError_t launch(const AttnArgs& a, int64_t grid, size_t smem_bytes, cudaStream_t st) {
        auto kern = dsa_attn_kernel<T, D, G, TILE, STAGES, HM, SEL>;
        const cudaError_t e = ensure_configured(kern, cc_configured());
        if (e != cudaSuccess) return e;
        return launch_pdl(kern, (unsigned)grid, NT, smem_bytes, st, a);
    }
};

// Dispatch over (group size, per-head masks, fused selection).  Selection needs one mask per query
// head, so it comes with per-head masks whenever the group is larger than one.
template <typename T, int D, class F>
bool dispatch_variant(const KernelQuery& q, F&& f) {
#define DSA_CASE_HM(GG)                                                                   \
    if (q.select) { f(KernelPick<T, D, GG, (GG > 1), true>{}); return true; }             \
    if (q.headmask) { f(KernelPick<T, D, GG, (GG > 1), false>{}); return true; }          \
    f(KernelPick<T, D, GG, false, false>{});                                              \
    return true;
    switch (q.G) {
        case 1: { DSA_CASE_HM(1) }
        case 2: { DSA_CASE_HM(2) }
        case 4: { DSA_CASE_HM(4) }
        case 8: { DSA_CASE_HM(8) }
        default: return false;
    }
#undef DSA_CASE_HM
}

template <typename T, int D>
bool kernel_shape(const KernelQuery& q, int chunk, int bitmap_words, KernelShape* out) {
    return dispatch_variant<T, D>(q, [&](auto pick) {
        using P = decltype(pick);
        out->tile = q.mma ? MMA_KEYS : P::TILE;
        if (q.mma && q.heads) {
            out->stages = kMmaStages;
            out->smem = P::smem_heads(q.dir_cap, q.window, q.kidx_cap, bitmap_words);
            return;
        }
        if (q.mma && q.group_w > 0) {
            out->stages = q.group_stages == kGroupStagesShallow ? kGroupStagesShallow : kGroupStages;
            out->smem = q.gather ? P::smem_gather(out->stages, chunk, bitmap_words)
                                 : P::smem_group(q.group_w, out->stages, chunk, bitmap_words);
            return;
        }
        const bool shallow = q.mma && q.mma_stages == kMmaStagesShallow && q.mma_warps == 2 && q.mma_kw == 1 &&
                             !q.headmask && !q.select;
        out->stages = q.mma ? (shallow ? kMmaStagesShallow : kMmaStages) : P::STAGES;
        out->smem = q.mma ? P::smem_mma(q.mma_warps, q.mma_kw, out->stages, chunk, bitmap_words)
                          : P::smem(chunk, bitmap_words);
    });
}

template <typename T, int D>
cudaError_t kernel_launch(const KernelQuery& q, bool append, const AttnArgs& a, int64_t items, size_t smem,
                          cudaStream_t st, int64_t blocks, const GatherMaps* maps) {
    cudaError_t err = cudaErrorInvalidValue;
    dispatch_variant<T, D>(q, [&](auto pick) {
        using P = decltype(pick);
        if (q.mma && q.mma_kw > 1 && q.mma_cl > 1) err = P::launch_cluster(q.mma_cl, append, a, items, smem, st);
        else if (q.mma && q.heads) err = P::launch_heads(append, a, blocks, smem, st);
        else if (q.mma && q.group_w > 0 && q.producers) err = P::launch_ws(q.group_stages, append, a, blocks, smem, st);
        else if (q.mma && q.group_w > 0 && q.gather) err = P::launch_gather(q.group_stages, append, a, maps, blocks, smem, st);
        else if (q.mma && q.group_w > 0) err = P::launch_group(q.group_w, q.group_stages, append, a, blocks, smem, st, q.copy_only);
        else
        err = q.mma ? P::launch_mma(q.mma_warps, q.mma_kw, q.mma_stages, a, items, smem, st, append)
                    : P::launch(a, items, smem, st);
    });
    return err;
}

template <typename T, int D>
cudaError_t kernel_prepare() {
    cudaError_t e = cudaSuccess;
    for (int g = 1; g <= 8 && e == cudaSuccess; g *= 2) {
        for (int variant = 0; variant < 3 && e == cudaSuccess; ++variant) {
            KernelQuery q = {};
            q.G = g; q.headmask = variant >= 1; q.select = variant == 2;
            if (g == 1 && variant == 1) continue;           // (a group of one has no per-head variant of its own)
            dispatch_variant<T, D>(q, [&](auto pick) { e = decltype(pick)::prepare(); });
        }
    }
    return e;
}

}  // namespace dsa
