// Instantiation unit: team kernels for small planes, f32 activations.
#include "team_kernels.cuh"
namespace wt {
namespace team {
WT_TEAM_INSTANTIATE(float, )
}  // namespace team
}  // namespace wt
