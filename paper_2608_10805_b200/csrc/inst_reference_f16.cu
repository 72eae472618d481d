// Instantiation unit: reference-style comparator chain (k = 3, 5, 7), f16 activations.
#include "reference_chain.cuh"
namespace wt {
namespace refchain {
WT_REFCHAIN_INSTANTIATE(__half, 3, )
WT_REFCHAIN_INSTANTIATE(__half, 5, )
WT_REFCHAIN_INSTANTIATE(__half, 7, )
}  // namespace refchain
}  // namespace wt
