// Instantiation unit: window kernels for large planes, bf16 activations.
#include "window_kernels.cuh"
namespace wt {
namespace window {
WT_WINDOW_INSTANTIATE(__nv_bfloat16, )
}  // namespace window
}  // namespace wt
