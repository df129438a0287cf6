// Host side of the fused persistent kernel (fused_kernel.cuh): eligibility and task plan, tensor
// maps, and dispatch between the generic kernel and the kernels specialised for the paper's layer
// shapes (App. G: 56x56 grid with 7x7 agents, 14x14 grid with 7x7 agents).
#include "fused_kernel.cuh"

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

namespace aa {

// defined in fused_spec_56.cu / fused_spec_14.cu
int fused_occupancy_s56(int dtype);
int fused_occupancy_s14(int dtype);
cudaError_t launch_fused_s56(int dtype, const FusedArgs& a, cudaStream_t st);
cudaError_t launch_fused_s14(int dtype, const FusedArgs& a, cudaStream_t st);
int fused_occupancy_s56s(int dtype);
int fused_occupancy_s14s(int dtype);
cudaError_t launch_fused_s56s(int dtype, const FusedArgs& a, cudaStream_t st);
cudaError_t launch_fused_s14s(int dtype, const FusedArgs& a, cudaStream_t st);

static int fused_spec_of(int H, int W, int n_agents) {
    if (H == 56 && W == 56 && n_agents == 49) return 1;
    if (H == 14 && W == 14 && n_agents == 49) return 2;
    return 0;
}


// Shape part of the plan (no CUDA calls): eligibility, task counts, partial states per slab.
static bool fused_shape_plan(int dtype, int H, int W, int d, int n_agents, FusedPlan* pl) {
    memset(pl, 0, sizeof(*pl));
    if (dtype != kBF16 && dtype != kF16) return false;
    if (d != DK) return false;
    if (n_agents < 1 || n_agents > RP || W > MAXW || W < MINW || H < 1) return false;
    int p = 1;
    while (p * p < n_agents) ++p;
    if (p * p != n_agents || H % p != 0 || W % p != 0) return false;
    const int win_h = H / p;
    // about 448 tokens per G task, in whole agent rows
    int k = (448 + win_h * W / 2) / (win_h * W);
    if (k < 1) k = 1;
    if (k > p) k = p;
    pl->rows_per_g = k * win_h;
    pl->g_tasks = (p + k - 1) / k;
    int R = QT / W;
    if (R > 16) R = 16;
    if (R > H) R = H;
    pl->rows_per_b = R;
    pl->b_tasks = (H + R - 1) / R;
    if ((R + 2) * (W + 2) > kHaloTokens) return false;
    pl->parts = pl->g_tasks;
    return pl->g_tasks <= 32;
}

int fused_parts_per_slab(int dtype, int H, int W, int d, int n_agents) {
    FusedPlan pl;
    return fused_shape_plan(dtype, H, W, d, n_agents, &pl) ? pl.parts : 0;
}

FusedPlan plan_fused(int dtype, int slabs, int H, int W, int d, int n_agents, int sm_count) {
    FusedPlan pl;
    if (!fused_shape_plan(dtype, H, W, d, n_agents, &pl)) { pl.ok = false; return pl; }
    if (!encode_tiled_fn()) return pl;            // no tensor-map encoder: use the per-step kernels
    pl.spec = fused_spec_of(H, W, n_agents);
    // (each query also raises that kernel's dynamic shared-memory limit; the generic kernel serves a
    // specialised shape whenever a bias or the depthwise filter is absent)
    int occ = fused_occupancy_dt<ShapeAny>(dtype);
    if (pl.spec == 1) occ = std::min(occ, std::min(fused_occupancy_s56(dtype), fused_occupancy_s56s(dtype)));
    if (pl.spec == 2) occ = std::min(occ, std::min(fused_occupancy_s14(dtype), fused_occupancy_s14s(dtype)));
    if (occ < 1) return pl;
    // The occupancy query counts a block that allocates tensor memory as taking all of it.  Two blocks
    // of 128 columns each fit the 512 columns of an SM, so where registers and shared memory allow a
    // second block the grid is sized for two (the queue only needs g_tasks resident blocks to progress).
    {
        cudaFuncAttributes fa;
        cudaDeviceProp prop;
        int dev = 0;
        const void* fn = dtype == kBF16 ? (const void*)fused_kernel<__nv_bfloat16, ShapeAny> : (const void*)fused_kernel<__half, ShapeAny>;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess &&
            cudaFuncGetAttributes(&fa, fn) == cudaSuccess) {
            const size_t smem_block = (size_t)kSmemBytes + fa.sharedSizeBytes + 1024;
            if (2 * smem_block <= prop.sharedMemPerMultiprocessor && 2 * fa.numRegs * NT <= prop.regsPerMultiprocessor &&
                2 * kTmemCols <= 512)
                occ = 2;
        } else {
            cudaGetLastError();
        }
    }
    if (getenv("AGENT_ATTN_LOG"))
        fprintf(stderr, "agent_attn: fused kernel spec=%d, %d blocks/SM, %d bytes of shared memory\n", pl.spec, occ, kSmemBytes);
    if (occ > 2) occ = 2;
    const long long total = (long long)slabs * (pl.g_tasks + pl.b_tasks);
    long long grid = (long long)occ * sm_count;
    if (grid > total) grid = total;
    pl.grid = (int)grid;
    if (pl.grid < pl.g_tasks) return pl;          // progress needs a resident block per G sibling
    // The aggregation runs ahead of the broadcast by `lag` slabs: far enough that B tasks rarely wait
    // for their slab's flag, close enough that the Q and V of the slabs in between stay in L2
    // (budget: half of a 126 MB L2 for those re-reads).
    const long long slab_qv_bytes = 2LL * H * W * d * 2;
    long long lag_l2 = (64LL << 20) / slab_qv_bytes;
    int lag = (5 * pl.grid / 2 + pl.g_tasks + pl.b_tasks - 1) / (pl.g_tasks + pl.b_tasks) + 2;
    if (lag_l2 > lag) lag = (int)(lag_l2 > 1000000 ? 1000000 : lag_l2);
    if (lag > slabs) lag = slabs;
    if (lag < 1) lag = 1;
    pl.lag = lag;
    pl.smem = kSmemBytes;
    pl.ok = true;
    return pl;
}

// Fills the tensor maps of `a` from its pointers and shape; false if one cannot be encoded.
bool fused_make_maps(FusedArgs* a) {
    const uint64_t N = (uint64_t)a->H * a->W, S = a->slabs;
    const int batch = a->slabs / a->heads;
    const TokLayout dl = dense_layout(a->heads, (long long)N, DK);
    a->dense_in = (a->lin.sb == dl.sb && a->lin.sh == dl.sh && a->lin.st == dl.st) ? 1 : 0;
    if (a->dense_in) {
        if (!make_map_2d_u16(&a->tm_k, a->k, S * N, DK, KT, DK)) return false;
        if (!make_map_2d_u16(&a->tm_v, a->v, S * N, DK, KT, DK)) return false;
        if (!make_map_2d_u16(&a->tm_q, a->q, S * N, DK, QT, DK)) return false;
    } else {
        if (!make_map_tok_u16(&a->tm_k, &a->hf_k, a->k, a->lin, batch, a->heads, (long long)N, DK, KT, true)) return false;
        if (!make_map_tok_u16(&a->tm_v, &a->hf_v, a->v, a->lin, batch, a->heads, (long long)N, DK, KT, true)) return false;
        if (!make_map_tok_u16(&a->tm_q, &a->hf_q, a->q, a->lin, batch, a->heads, (long long)N, DK, QT, true)) return false;
    }
    a->v_rows_contiguous = (a->lin.st == DK) ? 1 : 0;
    if (a->dwc_w && !a->v_rows_contiguous &&
        !make_map_tok_u16(&a->tm_vrow, &a->hf_vrow, a->v, a->lin, batch, a->heads, (long long)N, DK, (uint32_t)a->W, false))
        return false;
    if (!make_map_2d_u16(&a->tm_a, a->a_ws, S * a->n, DK, RP, DK)) return false;
    if (!make_map_2d_u16(&a->tm_va, a->va_ws, S * a->n, DK, (uint32_t)a->n, DK)) return false;    // box of n rows
    a->b1_tma = 0;
    if (a->b1 && N % 8 == 0 && ((uint64_t)a->plan.rows_per_g * a->W) % 8 == 0 && N >= KT)
        a->b1_tma = make_map_2d_u16(&a->tm_b1, a->b1, (uint64_t)a->heads * a->n, N, RP, KT) ? 1 : 0;
    return true;
}

cudaError_t launch_fused(int dtype, const FusedArgs& a, cudaStream_t st) {
    // the shape-specialised kernels assume both biases and the depthwise filter are present; each shape has
    // an instantiation for dense tensors and one for tensors with strides
    const TokLayout dl = dense_layout(a.heads, (long long)a.H * a.W, DK);
    const bool dense = a.dense_in && a.lout.sb == dl.sb && a.lout.sh == dl.sh && a.lout.st == dl.st;
    const bool full = a.b1 && a.b2 && a.dwc_w;
    if (full && a.plan.spec == 1) return dense ? launch_fused_s56(dtype, a, st) : launch_fused_s56s(dtype, a, st);
    if (full && a.plan.spec == 2) return dense ? launch_fused_s14(dtype, a, st) : launch_fused_s14s(dtype, a, st);
    return fused_launch_dt<ShapeAny>(dtype, a, st);
}

}  // namespace aa
