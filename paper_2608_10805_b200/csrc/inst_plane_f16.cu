// Instantiation unit: block-per-plane kernels, f16 activations.
#include "plane_kernels.cuh"
namespace wt {
namespace plane {
WT_PLANE_INSTANTIATE(__half, )
}  // namespace plane
}  // namespace wt
