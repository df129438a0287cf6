// Host-side launch interface between the C ABI (api.cu) and the kernel files.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace aa {

enum DType { kF32 = 0, kBF16 = 1, kF16 = 2 };

// Strides of a [batch, head, token, d] tensor in elements (d contiguous).  Dense [B, h, N, d] is
// {h N d, N d, d}; the output of a fused projection kept as [B, N, h, d] is {N h d, d, h d}.
struct TokLayout {
    long long sb, sh, st;
};
inline TokLayout dense_layout(int heads, long long n_tokens, int d) {
    TokLayout l;
    l.sb = (long long)heads * n_tokens * d; l.sh = n_tokens * d; l.st = d;
    return l;
}
__host__ __device__ inline long long tok_offset(const TokLayout& l, int slab, int heads, long long tok) {
    return (long long)(slab / heads) * l.sb + (long long)(slab % heads) * l.sh + tok * l.st;
}


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
    int heads;          // slab = batch item * heads + head
    TokLayout lq;       // strides of q
};
cudaError_t launch_pool(int dtype, const PoolArgs& p, cudaStream_t st);

// Dense agent bias from column [heads][n][w], row [heads][n][h] and block [heads][n][h0][w0]
// components (any may be null); out is [heads][n][N] or, transposed, [heads][N][n].
struct ComposeArgs {
    const void *col, *row, *blk;
    void* out;
    int heads, n, h, w, h0, w0, transpose;
};
cudaError_t launch_compose_bias(int dtype, const ComposeArgs& p, cudaStream_t st);

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
    int* status;          // device status word for bounded waits (tensor-memory kernels), may be null
    // token-major tensors of the call ([batch, head, token, d] with strides): aggregation K and V; broadcast Q,
    // the V of the depthwise term, and out.  The agent-side tensors (A, V_A) are dense [slabs][n][d].
    TokLayout lin, lout;
    int strided;          // lin or lout is not the dense layout (only the kernels that read strides may run)
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
// tensor-memory (tcgen05) kernels for large agent counts (aggregate_umma.cu)
bool aggregate_umma_eligible(int dtype, int n_agents, int n_tokens, int d, bool has_bias);
AggPlan plan_aggregate_umma(int slabs, int n_agents, int n_tokens, int d, int sm_count);
cudaError_t launch_aggregate_umma(int dtype, const AttnArgs& p, const AggPlan& plan, cudaStream_t st);
bool broadcast_umma_eligible(int dtype, int n_agents, int n_tokens, int d);
cudaError_t launch_broadcast_umma(int dtype, const AttnArgs& p, int sm_count, cudaStream_t st);

// Whole module (Eq. 6) in one persistent kernel for small agent counts (n <= 64, d = 64,
// block pooling, W <= 64).  Blocks take tasks from a device-side queue: "G" tasks pool their token
// range of Q, publish those agent rows, wait for the slab's other G tasks, and aggregate their
// range of K/V; "B" tasks wait for the slab's merged V_A and do the broadcast + DWC for one
// 128-token tile.  A slab's B tasks follow its G tasks closely, so Q and V are re-read from L2.
struct FusedPlan {
    bool ok;            // shape is eligible
    int g_tasks;        // G tasks per slab
    int rows_per_g;     // grid rows per G task (a multiple of the pooling window height)
    int rows_per_b;     // grid rows per B task (rows_per_b * W <= 128 tokens)
    int b_tasks;        // B tasks per slab
    int lag;            // slabs between a slab's G tasks and its B tasks in the queue
    int grid;           // resident blocks
    int parts;          // partial states per slab
    int spec;           // 0 = generic kernel, else index of a kernel specialised for this shape
    size_t smem;        // dynamic shared memory per block
};
struct FusedArgs {
    const void *q, *k, *v, *b1, *b2, *dwc_w;
    void* out;
    void* a_ws;           // [slabs][n][d] agents (written by G tasks)
    void* va_ws;          // [slabs][n][d] agent features (written by the merging G task)
    float* partials;      // [slabs][parts][partial_floats(64, d)]
    unsigned* counters;   // zero on entry: a_count[slabs] | tickets[slabs] | va_ready[slabs] | queue[1]
    int* status;          // device status word: set when a bounded wait gives up
    unsigned poll_limit;  // polls of another block's counter before a wait gives up
    int slabs, heads, H, W, d, n, p;
    float scale1, scale2;
    TokLayout lin, lout;  // strides of Q, K, V and of out
    FusedPlan plan;
    // TMA descriptors (128-byte swizzle, 64-column boxes): K and V with 64-token boxes (any batch / head / token strides),
    // B1 as [heads*n][N] with 64x64 boxes, A and V_A workspaces as [slabs*n][d] with 64-row boxes
    int b1_tma;           // B1 tiles come through TMA (needs N % 8 == 0 and 8-aligned task ranges)
    alignas(64) CUtensorMap tm_k, tm_v, tm_b1, tm_a, tm_va;
    alignas(64) CUtensorMap tm_q;     // Q with 128-token boxes (A operand of the broadcast MMA)
    alignas(64) CUtensorMap tm_vrow;  // V with boxes of one grid row (W tokens), no swizzle: rows of the depthwise window
    int hf_k, hf_v, hf_q, hf_vrow;    // dimension order of the token-major maps (tma_load_tok)
    int v_rows_contiguous;            // token stride of V == d: a grid row of V is one contiguous run
    int dense_in;                     // Q, K, V are dense [B][heads][N][d]: their maps are 2-D over [slabs * N][d]
};
FusedPlan plan_fused(int dtype, int slabs, int H, int W, int d, int n_agents, int sm_count);
bool fused_make_maps(FusedArgs* a);     // encode the tensor maps from a's pointers and shape
cudaError_t launch_fused(int dtype, const FusedArgs& a, cudaStream_t st);
int fused_parts_per_slab(int dtype, int H, int W, int d, int n_agents);   // 0 if the shape is not eligible
inline size_t fused_counter_words(int slabs) { return 3 * (size_t)slabs + 4; }

// Whole module (Eq. 6) for small agent counts and long token grids (n <= 64, d = 64, N >= 1024, dense tensors)
// as three streaming kernels, phase by phase over the batch (the second reads of Q and V come from L2):
//   prep       agents A = Pooling(Q) (or the caller's A), scaled copies for the two logit products, biases
//              clamped to finite values (B2 also padded to 64 columns), arrival counters cleared
//   aggregate  V_A = softmax(scale1 A K^T + B1) V: grid (splits, slabs), tcgen05 with the agents and the
//              probabilities as tensor-memory operands, bias added inside the contraction
//   broadcast  O = softmax(scale2 Q A^T + B2) V_A + DWC(V): persistent blocks over runs of row tiles
struct StreamPlan {
    bool ok;
    int splits;          // aggregation blocks per slab
    int tiles_per_split; // 128-token tiles per aggregation block
    int rows_b;          // grid rows per broadcast tile (rows_b * W <= 128 tokens)
    int tiles_b;         // broadcast tiles per slab
    int grid_b;          // broadcast blocks (persistent)
    int halo_stages;     // ring depth of the depthwise window's V rows
    int smem_b;          // dynamic shared memory of a broadcast block
};
struct StreamArgs {
    const void *q, *k, *v, *a_user, *b1, *b2, *dwc_w;
    void* out;
    void *a_ws, *va_ws;        // [slabs][n][64] agents and agent features (element type)
    void *a1s, *a2s;           // [slabs][n][64] agents times scale1 / scale2
    void *b1c, *b2p;           // [heads][N][64] clamped, transposed, padded B1; [heads or 1][N][64] clamped, padded B2
    void* wt;                  // [heads][9][16][128 B] diagonal slices of the depthwise filter, as swizzled operand tiles
    float* partials;           // [slabs][splits][partial_floats(64, 64)]
    unsigned* tickets;         // [slabs]
    int* status;
    int slabs, heads, H, W, n, p;
    float scale1, scale2;
    int sm_count;
    StreamPlan plan;
    alignas(64) CUtensorMap tm_k, tm_v, tm_b1, tm_q, tm_b2, tm_h, tm_a2, tm_va;
};
StreamPlan plan_stream(int dtype, int slabs, int H, int W, int d, int n_agents, bool pooled, int sm_count);
// workspace beyond A and V_A: bytes of (a1s | a2s | b1c | b2p), each 256-byte aligned, in this order
size_t stream_extra_bytes(int slabs, int heads, int N, int n_agents);
bool stream_make_maps(StreamArgs* a);
cudaError_t launch_stream_prep(int dtype, const StreamArgs& a, cudaStream_t st);
cudaError_t launch_stream_aggregate(int dtype, const StreamArgs& a, cudaStream_t st);
cudaError_t launch_stream_broadcast(int dtype, const StreamArgs& a, cudaStream_t st);

// ------------------------------------------------------------------------------ backward pass
// Tiling of the backward kernels: tiles of `tile` tokens, `chunks` blocks per slab, each block
// walking `tiles_per_chunk` consecutive tiles; np = agents padded to a multiple of 32, plus 1.
struct BwdPlan {
    int tile, np, tiles, chunks, tiles_per_chunk;
};
// Arguments of one backward kernel (set per launch by launch_backward).
struct BwdArgs {
    const void *x, *y;        // token rows [slabs][N][d]: operand of the logits, second operand
    const void* bias;         // B1 [heads][n][N] or B2 [heads][N][n], or null
    const float *m0, *m1;     // fp32 [slabs][n][d]: A; V_A or dV_A
    const float *lse, *dot;   // fp32 [slabs][n]: log-sum-exp of the aggregation rows; dV_A . V_A
    float* part;              // fp32 [slabs][chunks][n][2]: per-block (max, sum) of the aggregation logits
    float *outer0, *outer1;   // fp32 [slabs][n][d]: sums over tokens (atomics)
    float *row0, *row1;       // fp32 [slabs][N][d]: per-token results
    float* dbias;             // fp32 in the layout of `bias` (atomics), or null
    int slabs, heads, N, H, W, d, n, ph, pw;
    int np, tile, tiles, chunks, tiles_per_chunk;
    float scale;
};
// One backward call: inputs in the handle's element type, gradients and workspace in fp32.
struct BwdCall {
    const void *q, *k, *v, *d_out, *b1, *b2, *wd;
    float *dq, *dk, *dv, *db1, *db2, *dwd;
    float *ws_a, *ws_va, *ws_dva, *ws_da;     // [slabs][n][d] each; V_A, dV_A, dA contiguous in this order
    float *ws_lse, *ws_dot;                   // [slabs][n]
    float* ws_part;                           // [slabs][chunks][n][2]
    int4* ws_tab;                             // [N][3]: pooling windows of each token
    size_t clear_bytes;                       // bytes from ws_va to the end of ws_da
    int slabs, heads, H, W, d, n, p, sm_count;
    float scale1, scale2;
    BwdPlan plan;
    int dtype;                                // element type of the inputs (kF32, kBF16, kF16)
    int use_mma;                              // the two gradient stages run on the tensor-core kernels
    BwdPlan plan_mma;                         // their tiling
};
bool plan_backward(int slabs, int n, int N, int d, int sm_count, BwdPlan* out);   // false: shape not supported
int backward_launch_count(bool use_mma);
cudaError_t launch_backward(int dtype, const BwdCall& c, cudaStream_t st);
// Tensor-core kernels of the two gradient stages (16-bit inputs, n <= 64, d = 64)
bool backward_mma_eligible(int dtype, int n, int d);
BwdPlan plan_backward_mma(int slabs, int N, int sm_count);
cudaError_t launch_backward_mma(int dtype, bool broadcast_stage, const BwdArgs& a, cudaStream_t st);
// aggregation stage recomputed: per-block partials into a.part, then V_A and the log-sum-exp per agent
cudaError_t launch_backward_fwd1_mma(int dtype, const BwdArgs& a, float* va, float* lse, cudaStream_t st);
size_t backward_mma_part_floats(int slabs, const BwdPlan& pl);

}  // namespace aa
