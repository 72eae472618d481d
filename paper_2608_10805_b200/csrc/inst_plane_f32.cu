// Instantiation unit: block-per-plane kernels, f32 activations.
#include "plane_kernels.cuh"
namespace wt {
namespace plane {
WT_PLANE_INSTANTIATE(float, )
}  // namespace plane
}  // namespace wt
