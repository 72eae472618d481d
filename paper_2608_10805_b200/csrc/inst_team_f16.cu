// Instantiation unit: team kernels for small planes, f16 activations.
#include "team_kernels.cuh"
namespace wt {
namespace team {
WT_TEAM_INSTANTIATE(__half, )
}  // namespace team
}  // namespace wt
