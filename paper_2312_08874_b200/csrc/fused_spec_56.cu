// Fused persistent kernel specialised at compile time for the 56x56 token grid with 7x7 agents,
// both biases and the depthwise term present (a layer shape of the paper's App. G).
#include "fused_kernel.cuh"

namespace aa {
int fused_occupancy_s56(int dtype) { return fused_occupancy_dt<FusedShape<56, 56, 7>>(dtype); }
cudaError_t launch_fused_s56(int dtype, const FusedArgs& a, cudaStream_t st) {
    return fused_launch_dt<FusedShape<56, 56, 7>>(dtype, a, st);
}
// the same shape on tensors with strides (token-major or interleaved storage)
int fused_occupancy_s56s(int dtype) { return fused_occupancy_dt<FusedShape<56, 56, 7, false>>(dtype); }
cudaError_t launch_fused_s56s(int dtype, const FusedArgs& a, cudaStream_t st) {
    return fused_launch_dt<FusedShape<56, 56, 7, false>>(dtype, a, st);
}
}  // namespace aa
