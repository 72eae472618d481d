// Instantiation unit: block-per-plane kernels, bf16 activations.
#include "plane_kernels.cuh"
namespace wt {
namespace plane {
WT_PLANE_INSTANTIATE(__nv_bfloat16, )
}  // namespace plane
}  // namespace wt
