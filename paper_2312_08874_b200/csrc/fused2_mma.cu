// Host side of the role-specialised fused kernel (fused2_kernel.cuh): eligibility and task plan,
// tensor maps, and dispatch between the generic kernel and the kernels specialised for the paper's
// layer shapes (App. G: 56x56 grid with 7x7 agents, 14x14 grid with 7x7 agents).
#include "fused2_kernel.cuh"

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

namespace aa {

// defined in fused2_spec_56.cu / fused2_spec_14.cu
bool fused2_prepare_s56(int dtype);
bool fused2_prepare_s14(int dtype);
cudaError_t launch_fused2_s56(int dtype, const FusedArgs& a, cudaStream_t st);
cudaError_t launch_fused2_s14(int dtype, const FusedArgs& a, cudaStream_t st);

static int fused2_spec_of(int H, int W, int n_agents) {
#ifdef AA_FUSED2_TRACE
    return 0;                      // debug builds trace the generic kernel
#endif
    if (H == 56 && W == 56 && n_agents == 49) return 1;
    if (H == 14 && W == 14 && n_agents == 49) return 2;
    return 0;
}

FusedPlan plan_fused2(int dtype, int slabs, int H, int W, int d, int n_agents, int sm_count, bool has_b1) {
    using namespace f2;
    FusedPlan pl;
    memset(&pl, 0, sizeof(pl));
    if (getenv("AGENT_ATTN_NO_FUSED2")) return pl;
    if (dtype != kBF16 && dtype != kF16) return pl;
    if (d != DK) return pl;
    if (n_agents < 1 || n_agents > RP || W > MAXW || W < MINW || H < 1) return pl;
    int p = 1;
    while (p * p < n_agents) ++p;
    if (p * p != n_agents || H % p != 0 || W % p != 0) return pl;
    const int win_h = H / p;
    // about 448 tokens per G task, in whole agent rows
    int k = (448 + win_h * W / 2) / (win_h * W);
    if (k < 1) k = 1;
    if (k > p) k = p;
    pl.rows_per_g = k * win_h;
    pl.g_tasks = (p + k - 1) / k;
    if (pl.g_tasks > 32) return pl;
    pl.parts = pl.g_tasks;
    int R = QT / W;
    if (R > 16) R = 16;
    if (R > H) R = H;
    pl.rows_per_b = R;
    pl.b_tiles = (H + R - 1) / R;
    if ((2 * R + 2) * (W + 2) > kVTokens) return pl;
    // runs of about four tiles; a slab's runs are equally long where possible
    int tb = 4;
    const char* env_tb = getenv("AGENT_ATTN_FUSED2_TB");
    if (env_tb && atoi(env_tb) > 0) tb = atoi(env_tb);
    if (tb > pl.b_tiles) tb = pl.b_tiles;
    pl.tb = tb;
    pl.b_tasks = (pl.b_tiles + tb - 1) / tb;
    // B1 rows that TMA cannot fetch (row pitch not a multiple of 16 bytes, or ranges that do not start on
    // 8-token boundaries) are copied by plain loads before the loop, which needs the whole range in the ring
    const long long N = (long long)H * W;
    const bool b1_tma = N % 8 == 0 && ((long long)pl.rows_per_g * W) % 8 == 0 && N >= KT;
    const int tiles_per_g = (pl.rows_per_g * W + KT - 1) / KT;
    if (has_b1 && !b1_tma && tiles_per_g > RING) return pl;
    if (!encode_tiled_fn()) return pl;
    pl.spec = fused2_spec_of(H, W, n_agents);
    if (!fused2_prepare_dt<ShapeAny>(dtype)) return pl;
    if (pl.spec == 1 && !fused2_prepare_s56(dtype)) return pl;
    if (pl.spec == 2 && !fused2_prepare_s14(dtype)) return pl;
    const long long total = (long long)slabs * (2 * pl.g_tasks + 1 + pl.b_tasks);
    if (total > 0x3fffffffLL) return pl;
    long long grid = sm_count;                     // one block per SM: a block takes all of its tensor memory
    if (grid > total) grid = total;
    pl.grid = (int)grid;
    // Slabs are processed in groups: pooling, aggregation, merge and broadcast of consecutive groups
    // overlap in the queue, and a group is small enough that the Q and V of the groups in flight stay
    // in L2 between their first and second reads (budget: half of a 126 MB L2).
    const long long slab_qv_bytes = 2LL * H * W * d * 2;
    long long lag = (64LL << 20) / (3 * slab_qv_bytes);
    const char* env_lag = getenv("AGENT_ATTN_FUSED2_LAG");
    if (env_lag && atoi(env_lag) > 0) lag = atoi(env_lag);
    if (3 * lag >= slabs) lag = slabs;             // everything fits: one group, phase after phase
    if (lag < 1) lag = 1;
    pl.lag = (int)lag;
    pl.smem = kSmemBytes;
    pl.v2 = 1;
    pl.ok = true;
    if (getenv("AGENT_ATTN_LOG"))
        fprintf(stderr, "agent_attn: role-specialised fused kernel spec=%d grid=%d g_tasks=%d b_tasks=%d (tb=%d) lag=%d smem=%d\n",
                pl.spec, pl.grid, pl.g_tasks, pl.b_tasks, pl.tb, pl.lag, kSmemBytes);
    return pl;
}

bool fused2_make_maps(FusedArgs* a) {
    using namespace f2;
    const uint64_t N = (uint64_t)a->H * a->W, S = a->slabs;
    if (!make_map_2d_u16(&a->tm_k, a->k, S * N, DK, KT, DK)) return false;
    if (!make_map_2d_u16(&a->tm_v, a->v, S * N, DK, KT, DK)) return false;
    if (!make_map_2d_u16(&a->tm_q, a->q, S * N, DK, QT, DK)) return false;
    if (!make_map_2d_u16(&a->tm_ag, a->ag_ws, S * RP, DK, RP, DK)) return false;
    if (!make_map_2d_u16(&a->tm_ab, a->ab_ws, S * RP, DK, RP, DK)) return false;
    if (!make_map_2d_u16(&a->tm_va2, a->va2_ws, S * RP, DK, RP, DK)) return false;
    a->b1_tma = 0;
    if (a->b1 && N % 8 == 0 && ((uint64_t)a->plan.rows_per_g * a->W) % 8 == 0 && N >= KT)
        a->b1_tma = make_map_2d_u16(&a->tm_b1, a->b1, (uint64_t)a->heads * a->n, N, RP, KT) ? 1 : 0;
    if (a->b1 && !a->b1_tma && (a->plan.rows_per_g * a->W + KT - 1) / KT > RING) return false;
    return true;
}

cudaError_t launch_fused2(int dtype, const FusedArgs& a, cudaStream_t st) {
    using namespace f2;
    // the shape-specialised kernels assume both biases and the depthwise filter are present
    const bool full = a.b1 && a.b2 && a.dwc_w;
    if (full && a.plan.spec == 1) return launch_fused2_s56(dtype, a, st);
    if (full && a.plan.spec == 2) return launch_fused2_s14(dtype, a, st);
    return fused2_launch_dt<ShapeAny>(dtype, a, st);
}

}  // namespace aa

#ifdef AA_FUSED2_TRACE
extern "C" int aa_fused2_trace_buffer(void* device_buffer) {
    return (int)cudaMemcpyToSymbol(aa::f2::g_trace2, &device_buffer, sizeof(void*));
}
#endif
