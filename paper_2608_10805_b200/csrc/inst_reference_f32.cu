// Instantiation unit: reference-style comparator chain (k = 3, 5, 7), f32 activations.
#include "reference_chain.cuh"
namespace wt {
namespace refchain {
WT_REFCHAIN_INSTANTIATE(float, 3, )
WT_REFCHAIN_INSTANTIATE(float, 5, )
WT_REFCHAIN_INSTANTIATE(float, 7, )
}  // namespace refchain
}  // namespace wt
