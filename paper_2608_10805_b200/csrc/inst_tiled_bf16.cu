// Instantiation unit: tiled kernels (k = 3, 5, 7), bf16 activations.
#include "tiled_host.cuh"
namespace wt {
namespace host {
WT_TILED_INSTANTIATE(__nv_bfloat16, 3, )
WT_TILED_INSTANTIATE(__nv_bfloat16, 5, )
WT_TILED_INSTANTIATE(__nv_bfloat16, 7, )
}  // namespace host
}  // namespace wt
