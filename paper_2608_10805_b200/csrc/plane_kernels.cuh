// Whole-plane shared-memory kernels (placeholder: not yet enabled; every shape takes the tiled path).
#pragma once
#include "common.cuh"
#include "tiled_kernels.cuh"

namespace wt {
namespace plane {

inline bool supported(int, int, int, int, int) { return false; }
inline size_t forward_workspace_bytes(int, int, int, int, int) { return 0; }
inline size_t backward_workspace_bytes(int, int, int, int, int) { return 0; }

template <typename T>
cudaError_t forward(int, int, int, int, int, const T *, const float *, const float *, const float *, const float *,
                    const float *, T *, char *, cudaStream_t) {
    return cudaErrorNotSupported;
}
template <typename T>
cudaError_t backward(int, int, int, int, int, const T *, const T *, const float *, const float *, const float *,
                     const float *, T *, char *, EpiloguePtrs *, cudaStream_t) {
    return cudaErrorNotSupported;
}

}  // namespace plane
}  // namespace wt
