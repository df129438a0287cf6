// Role-specialised fused kernel fixed at compile time to the 14x14 token grid with 7x7 agents, both
// biases and the depthwise term present (a layer shape of the paper's App. G).
#include "fused2_kernel.cuh"

namespace aa {
bool fused2_prepare_s14(int dtype) { return f2::fused2_prepare_dt<f2::Shape<14, 14, 7>>(dtype); }
cudaError_t launch_fused2_s14(int dtype, const FusedArgs& a, cudaStream_t st) {
    return f2::fused2_launch_dt<f2::Shape<14, 14, 7>>(dtype, a, st);
}
}  // namespace aa
