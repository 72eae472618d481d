// Instantiation unit: tiled kernels (k = 3, 5, 7), f16 activations.
#include "tiled_host.cuh"
namespace wt {
namespace host {
WT_TILED_INSTANTIATE(__half, 3, )
WT_TILED_INSTANTIATE(__half, 5, )
WT_TILED_INSTANTIATE(__half, 7, )
}  // namespace host
}  // namespace wt
