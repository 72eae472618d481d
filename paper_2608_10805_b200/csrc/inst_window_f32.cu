// Instantiation unit: window kernels for large planes, f32 activations.
#include "window_kernels.cuh"
namespace wt {
namespace window {
WT_WINDOW_INSTANTIATE(float, )
}  // namespace window
}  // namespace wt
