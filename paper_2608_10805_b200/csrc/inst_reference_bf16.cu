// Instantiation unit: reference-style comparator chain (k = 3, 5, 7), bf16 activations.
#include "reference_chain.cuh"
namespace wt {
namespace refchain {
WT_REFCHAIN_INSTANTIATE(__nv_bfloat16, 3, )
WT_REFCHAIN_INSTANTIATE(__nv_bfloat16, 5, )
WT_REFCHAIN_INSTANTIATE(__nv_bfloat16, 7, )
}  // namespace refchain
}  // namespace wt
