// Host-side launch interface between the C ABI (api.cu) and the kernel files.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace aa {

enum DType { kF32 = 0, kBF16 = 1, kF16 = 2 };

// Split-partial layout.  One partial per (slab, part): m[rows_pad], l[rows_pad],
// acc[rows_pad][dpad], all fp32, with m and the logits in log2 units (logit * log2(e)), so the
// merge weights are exp2(m_j - m).
__host__ __device__ inline size_t partial_floats(int rows_pad, int dpad) {
    return (size_t)rows_pad * (size_t)(dpad + 2);
}

// Agent pooling: A[slab][ay*pw+ax][:] = mean of Q over the window of pooled cell (ay, ax).
struct PoolArgs {
    const void* q;      // [slabs][H*W][d]
    void* a;            // [slabs][ph*pw][d]
    int slabs, H, W, d, ph, pw;
};
cudaError_t launch_pool(int dtype, const PoolArgs& p, cudaStream_t st);

// One softmax attention with an additive bias, out = softmax(scale * Qm Km^T + bias) Vm.
// Aggregation: rows = agents, cols = tokens (split over blocks, merged by the last block).
// Broadcast:   rows = tokens, cols = agents, plus the depthwise 3x3 term on `dwc_v`.
struct AttnArgs {
    const void* qm;       // [slabs][rows][d]
    const void* km;       // [slabs][cols][d]
    const void* vm;       // [slabs][cols][d]
    const void* bias;     // [heads][rows][cols] or nullptr
    void* out;            // [slabs][rows][d]
    float* partials;      // aggregation only: [slabs][parts][partial_floats(rows_pad, dpad)]
    unsigned* tickets;    // aggregation only: [slabs], zero on entry, zero on exit
    int slabs, heads, rows, cols, d;
    float scale;          // logit scale in natural units
    int splits;           // aggregation only: blocks per slab along the token axis
    const void* dwc_v;    // broadcast only: V [slabs][H*W][d] or nullptr
    const void* dwc_w;    // broadcast only: [heads][d][3][3] or nullptr
    int H, W;             // broadcast only: token grid
};

// Plan of the aggregation launch for a problem shape (used for workspace sizing too).
struct AggPlan {
    int rows_pad;     // agents padded to the kernel's row granularity
    int dpad;         // head dim padded to the kernel's column granularity
    int splits;       // blocks per slab along the token axis
    int parts;        // partial states per slab that the merge reads
    int row_blocks;   // blocks per slab along the agent axis (fp32 FMA path only)
};

// per-path planners and launchers (attn_simt.cu / aggregate_mma.cu / broadcast_mma.cu)
AggPlan plan_aggregate_simt(int slabs, int n_agents, int n_tokens, int d, int sm_count);
AggPlan plan_aggregate_mma(int slabs, int n_agents, int n_tokens, int d, int sm_count);
cudaError_t launch_aggregate_simt(int dtype, const AttnArgs& p, const AggPlan& plan, cudaStream_t st);
cudaError_t launch_broadcast_simt(int dtype, const AttnArgs& p, cudaStream_t st);
cudaError_t launch_aggregate_mma(int dtype, const AttnArgs& p, const AggPlan& plan, cudaStream_t st);
cudaError_t launch_broadcast_mma(int dtype, const AttnArgs& p, cudaStream_t st);

}  // namespace aa
