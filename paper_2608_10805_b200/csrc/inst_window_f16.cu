// Instantiation unit: window kernels for large planes, f16 activations.
#include "window_kernels.cuh"
namespace wt {
namespace window {
WT_WINDOW_INSTANTIATE(__half, )
}  // namespace window
}  // namespace wt
