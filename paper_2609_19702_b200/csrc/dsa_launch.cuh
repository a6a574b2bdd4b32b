// The seam between the host-side planner (dsa_api.cu) and the attention kernels: the kernels of
// each (element type, head_dim) are instantiated in a translation unit of their own, so that the
// library builds in parallel, and are reached through the two function templates declared here.
#pragma once
#include "dsa_common.cuh"

namespace dsa {

constexpr int kMaxDevices = 64;
constexpr int kMmaItemWarps = 4;                   // warps per work item in small launches
constexpr int kMmaStages = 3;                      // ring slots per warp: two 16-key tiles in flight, one being consumed
constexpr int kMmaStagesShallow = 2;
constexpr int kHeadsWarps = 4;                     // warps per block of the per-head-list kernel
constexpr int kGroupStagesShallow = 2;             // shallow form: half as many blocks again per SM
constexpr int kGroupStages = 3;                    // ring slots per warp of the head-group kernel (4 and 6 slots with
                                                   // fewer warps per SM measured 25-45 % slower: the warps, not the
                                                   // bytes in flight, carry the throughput)               // the shallow-ring form of the two-heads-per-block kernel

// Which kernel variant a call needs.
struct KernelQuery {
    int G;                   // query heads per kv head: 1, 2, 4 or 8
    bool headmask;           // one mask per query head inside a group
    bool select;             // fused phase-2 selection
    bool mma;                // tensor-core kernel (bf16) rather than the CUDA-core kernel
    int mma_warps;           // tensor-core kernel: kv heads per block that share one row list (1 or 2)
    int mma_kw;              // tensor-core kernel: warps that share one work item (1 or kMmaItemWarps)
    int mma_cl;              // tensor-core kernel, several warps per item: blocks of a cluster that share the item (1, 2 or 4)
    int mma_stages;          // tensor-core kernel: kMmaStages, or kMmaStagesShallow (two heads per block only)
    int group_w;             // head-group tensor-core kernel: warps per block that share one row list for
                             // group_w x heads_per_warp kv heads (2 or 4); 0: not that kernel
    int group_stages;        // its ring depth: kGroupStages or kGroupStagesShallow
    bool copy_only;          // head-group kernel (group_w 4, no fused step) in its measuring form: copies, no arithmetic
    bool gather;             // head-group kernel whose tiles are staged by tensor-map gather copies (group_w 4)
    bool producers;          // head-group kernel with a producer warp beside every consumer warp (group_w 4)
    bool heads;              // per-head-list tensor-core kernel (blocks of kHeadsWarps warps); sizes of its tables:
    int dir_cap, kidx_cap, window;
};

struct KernelShape {
    int tile;                // keys per staged tile
    int stages;              // tiles in flight (per warp for the tensor-core kernel)
    size_t smem;             // dynamic shared memory per block for a row list of `chunk` rows
};

// Shape of the variant `q` of element type T and head_dim D.  Returns false for an unsupported G.
template <typename T, int D>
bool kernel_shape(const KernelQuery& q, int chunk, int bitmap_words, KernelShape* out);

// Launch it: `items` (request, kv head, split) work items; `append`: the fused decode step (the
// kernel reads the current token's rows from a.k_new / a.v_new and stores them to the cache);
// `blocks`: thread blocks of the head-group kernel (ignored by the others); `maps`: the cache views
// of the tensor-map form of it (q.gather), NULL otherwise.
template <typename T, int D>
cudaError_t kernel_launch(const KernelQuery& q, bool append, const AttnArgs& a, int64_t items, size_t smem,
                          cudaStream_t st, int64_t blocks, const GatherMaps* maps);

// Configure every variant of (T, D) for the current device, so that no later launch has to (a
// launch inside a stream capture must not).
template <typename T, int D>
cudaError_t kernel_prepare();

}  // namespace dsa
