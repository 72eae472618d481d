// Instantiation unit: team kernels for small planes, bf16 activations.
#include "team_kernels.cuh"
namespace wt {
namespace team {
WT_TEAM_INSTANTIATE(__nv_bfloat16, )
}  // namespace team
}  // namespace wt
