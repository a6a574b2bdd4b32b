// Attention kernels for bf16 caches with head_dim 128 (see dsa_launch.cuh).
#include "dsa_kernels.cuh"

namespace dsa {
template bool kernel_shape<__nv_bfloat16, 128>(const KernelQuery&, int, int, KernelShape*);
template cudaError_t kernel_launch<__nv_bfloat16, 128>(const KernelQuery&, bool, const AttnArgs&, int64_t, size_t, cudaStream_t, int64_t, const GatherMaps*);
template cudaError_t kernel_prepare<__nv_bfloat16, 128>();
}  // namespace dsa
