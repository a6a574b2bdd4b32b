// Attention kernels for float32 caches with head_dim 64 (see dsa_launch.cuh).
#include "dsa_kernels.cuh"

namespace dsa {
template bool kernel_shape<float, 64>(const KernelQuery&, int, int, KernelShape*);
template cudaError_t kernel_launch<float, 64>(const KernelQuery&, bool, const AttnArgs&, int64_t, size_t, cudaStream_t, int64_t, const GatherMaps*);
template cudaError_t kernel_prepare<float, 64>();
}  // namespace dsa
