// Instantiation unit: tiled kernels (k = 3, 5, 7), f32 activations.
#include "tiled_host.cuh"
namespace wt {
namespace host {
WT_TILED_INSTANTIATE(float, 3, )
WT_TILED_INSTANTIATE(float, 5, )
WT_TILED_INSTANTIATE(float, 7, )
}  // namespace host
}  // namespace wt
