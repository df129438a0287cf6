// Agent aggregation V_A = softmax(scale1 * A K^T + B1) V (Eq. 3, Eq. 5) for large agent counts
// (64 < n <= 256, d <= 64, 16-bit elements) on the 5th-generation tensor cores.
//
// Grid: (splits, slabs), one block of 19 warps per SM.  A block keeps the slab's agents resident (up to
// two 128-row operand blocks) and streams its share of the slab's 64-token tiles (K, V and the matching
// B1 columns) through a four-stage TMA ring.
//   warp 16 "producer":  one lane issues every TMA copy, ahead of the others through full/empty mbarriers.
//   warps 17, 18 "MMA issuers": one lane each, one per agent block ("chain"): S = A_block K^T (tcgen05.mma,
//                        accumulator in tensor memory) one tile ahead, and the products P V once the chain's
//                        probabilities of a tile are written.  The two chains (agents 0-127, agents 128-255)
//                        share the ring but have their own barriers, so that one computes while the other
//                        waits for its products.
//   warps 0-15 "row warps": thread (agent row, token half): reads its 32 logits of the tile from tensor
//                        memory, adds scale and bias, keeps its own running maximum / sum (no reduction
//                        crosses threads: each token half has its own accumulator in tensor memory),
//                        writes the probabilities back to shared memory as the A operand of P V, in place
//                        of the bias values it has just read (so P needs no buffer and the ring has a
//                        fourth stage).
//                        A row's reference maximum moves only when exceeded by a margin; then the thread
//                        rescales its accumulator row in tensor memory.
// At the end the two token halves of a row meet in shared memory and the block writes one partial state;
// a second small kernel merges the slab's partials in a fixed order, spread over many blocks (a merge by
// the slab's last block alone took longer than the streaming part).
// Every wait is bounded (pipe.cuh).  No TMA multicast, no clusters.
#include "common.cuh"
#include "kernels.h"
#include "merge.cuh"
#include "pipe.cuh"

#include <cstring>

namespace aa {

namespace {
constexpr int KT = 64;                 // tokens per tile
constexpr int NROW = 512;              // row-warp threads
constexpr int NT = NROW + 96;          // + producer warp + two MMA issuer warps (logits, products)
constexpr int STAGES = 4;
constexpr int kTile = 64 * 128;        // swizzled [64][64] tile of 16-bit elements
constexpr float kTau = 5.5f;           // margin (natural units) before a row's reference maximum moves
constexpr int kTimeoutTile = 3, kTimeoutLoads = 4, kTimeoutRole = 6;

// shared memory (bytes from a 1024-aligned base)
constexpr int OFF_BAR = 0;                               // mbarriers
constexpr int OFF_A = 1024;                              // agents [256][128 B]
constexpr int OFF_RING = OFF_A + 4 * kTile;              // STAGES x (K | V | B1 [256][128 B], later the probabilities)
constexpr int kStage = 2 * kTile + 4 * kTile;
constexpr int kSmemBytes = OFF_RING + STAGES * kStage + 1024;
static_assert(kSmemBytes <= 232448 && kSmemBytes > 116 * 1024, "one block per SM");

// mbarriers                                    count            waiter
constexpr int BAR_FULL = 0;       // [STAGES]        tx             each chain's MMA issuer
constexpr int BAR_EMPTY = 4;      // [STAGES]        one commit per chain     producer
constexpr int BAR_S_FULL = 8;     // [chain][2]      commit         the chain's row warps
constexpr int BAR_S_EMPTY = 12;   // [chain][2]      256 threads    the chain's MMA issuer
constexpr int BAR_P_FULL = 16;    // [chain]         256 threads    the chain's MMA issuer
constexpr int BAR_PV = 18;        // [chain]         commit         the chain's row warps
constexpr int BAR_AG = 20;        //                 tx             both MMA issuers
constexpr int kBars = 21;

// tensor memory: logits 2 buffers x (2 agent blocks x 64), accumulators (agent block, token half) x 64
constexpr uint32_t TM_S = 0, TM_O = 256;

struct UmmaAggArgs {
    AttnArgs a;
    int rows_pad, tps;                 // padded agent rows (128 or 256), tiles per split
    int hf_k, hf_v;                    // dimension order of the K and V maps (tma_load_tok)
    alignas(64) CUtensorMap tm_a, tm_k, tm_v, tm_b;
};
}  // namespace

template <typename T>
__global__ void __launch_bounds__(NT, 1) aggregate_umma_kernel(const __grid_constant__ UmmaAggArgs g) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_dead;
    __shared__ uint32_t s_tmem;
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const AttnArgs& p = g.a;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, slab = blockIdx.y;
    const int head = slab % p.heads;
    const int n = p.rows, N = p.cols;
    const int MB = g.rows_pad >> 7;                       // 128-row agent blocks
    const bool has_bias = p.bias != nullptr;
    const int tiles_all = (N + KT - 1) / KT;
    const int t0 = split * g.tps, t1 = min(tiles_all, t0 + g.tps);
    const int tiles = t1 - t0;                            // >= 1 by the plan

    Pipe pp;
    pp.status = p.status;
    pp.dead = &s_dead;
    pp.bars = smem_u32(smem + OFF_BAR);
    pp.ph = 0u;
    if (tid == 0) {
        s_dead = 0;
        for (int i = 0; i < kBars; ++i)
            mbar_init(pp.bars + 8 * i, (i >= BAR_S_EMPTY && i < BAR_PV) ? 256u : (i >= BAR_EMPTY && i < BAR_S_FULL) ? (uint32_t)MB : 1u);
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc<512>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem = s_tmem;

    const uint32_t sA = smem_u32(smem + OFF_A), ring = smem_u32(smem + OFF_RING);
    const size_t pf = partial_floats(g.rows_pad, 64);
    float* slab_parts = p.partials + (size_t)slab * gridDim.x * pf;

    if (warp == 16) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            mbar_arrive_expect_tx(pipe_bar(pp, BAR_AG), (uint32_t)MB * 2 * kTile);
            for (int mb = 0; mb < MB; ++mb) tma_load_2d(sA + mb * 2 * kTile, &g.tm_a, 0, slab * n + 128 * mb, pipe_bar(pp, BAR_AG));
            const uint32_t tx = 2 * kTile + (has_bias ? (uint32_t)MB * 2 * kTile : 0u);
            for (int t = 0; t < tiles; ++t) {
                const int s = t % STAGES, c0 = (t0 + t) * KT;
                if (t >= STAGES) pipe_wait_one(pp, BAR_EMPTY + s, kTimeoutRole);
                const uint32_t bar = pipe_bar(pp, BAR_FULL + s), dst = ring + s * kStage;
                mbar_arrive_expect_tx(bar, tx);
                tma_load_tok(dst, &g.tm_k, g.hf_k, c0, head, slab / p.heads, bar);
                tma_load_tok(dst + kTile, &g.tm_v, g.hf_v, c0, head, slab / p.heads, bar);
                if (has_bias)
                    for (int mb = 0; mb < MB; ++mb) tma_load_2d(dst + 2 * kTile + mb * 2 * kTile, &g.tm_b, c0, head * n + 128 * mb, bar);
            }
            for (int t = max(0, tiles - STAGES); t < tiles; ++t) pipe_wait_one(pp, BAR_EMPTY + t % STAGES, kTimeoutRole);
        }
        __syncwarp();
    } else if (warp == 17 || warp == 18) {
        // ------------------------------------------------------------------ MMA issuer of chain m = agent block m
        const int m = warp - 17;
        if (m < MB) {     // (the whole warp runs the loop; one elected lane issues)
            const uint32_t idK = umma_idesc(fmt, 128, 64, 0), idMN = umma_idesc(fmt, 128, 64, 1);
            const uint64_t dA = umma_desc_sw128(sA) + 1024 * m, dRing = umma_desc_sw128(ring);
            // descriptor start addresses count 16-byte units: + 2 per K-step of a K-major operand (32 bytes),
            // + 128 per K-step of an MN-major operand (16 rows of 128 bytes), + 1024 per 128-row block
            auto issue_S = [&](int t) {
                const int b = t & 1, s = t % STAGES;
                if (t >= 2) pipe_wait_one(pp, BAR_S_EMPTY + 2 * m + b, kTimeoutRole);
                pipe_wait_one(pp, BAR_FULL + s, kTimeoutTile);
                tc_fence_after_sync();
                const uint64_t dK = dRing + (uint64_t)(s * (kStage >> 4));
                const uint32_t dd = pp.tmem + TM_S + 128 * b + 64 * m;
                umma_ss_w(dd, dA, dK, idK, 0u);
                umma_ss_w(dd, dA + 2, dK + 2, idK, 1u);
                umma_ss_w(dd, dA + 4, dK + 4, idK, 1u);
                umma_ss_w(dd, dA + 6, dK + 6, idK, 1u);
                umma_commit_w(pipe_bar(pp, BAR_S_FULL + 2 * m + b));
            };
            pipe_wait_one(pp, BAR_AG, kTimeoutLoads);
            issue_S(0);
            for (int t = 0; t < tiles; ++t) {
                if (t + 1 < tiles) issue_S(t + 1);
                const int s = t % STAGES;
                pipe_wait_one(pp, BAR_P_FULL + m, kTimeoutRole);
                tc_fence_after_sync();
                const int ntok = min(KT, N - (t0 + t) * KT);
                const uint64_t dV = dRing + (uint64_t)(s * (kStage >> 4)) + (uint64_t)(kTile >> 4);
                const uint64_t dP = dV + (uint64_t)(kTile >> 4) + 1024 * m;      // the probabilities replaced the stage's bias tile
                for (int c = 0; c < 2; ++c) {
                    if (32 * c >= ntok) break;
                    const uint32_t dd = pp.tmem + TM_O + 64 * (2 * m + c);
                    const uint64_t da = dP + 4 * c, db = dV + 256 * c;
                    if (t > 0) umma_ss_w(dd, da, db, idMN, 1u); else umma_ss_w(dd, da, db, idMN, 0u);
                    umma_ss_w(dd, da + 2, db + 128, idMN, 1u);
                }
                umma_commit_w(pipe_bar(pp, BAR_EMPTY + s));
                umma_commit_w(pipe_bar(pp, BAR_PV + m));
            }
            for (int t = max(0, tiles - 2); t < tiles; ++t) pipe_wait_one(pp, BAR_S_EMPTY + 2 * m + (t & 1), kTimeoutRole);
        }
        __syncwarp();
    } else if ((warp >> 2 & 1) < MB) {
        // ------------------------------------------------------------------ row warps
        const int mb = (warp >> 2) & 1, c = warp >> 3;         // agent block, token half
        const int row = 128 * mb + 32 * (warp & 3) + lane;     // agent row (padded)
        const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
        const uint32_t tO = pp.tmem + TM_O + 64 * (2 * mb + c) + lane_base;
        float m_ref = -INFINITY, l = 0.f;
        bool started = false;
        for (int t = 0; t < tiles; ++t) {
            const int b = t & 1, s = t % STAGES;
            const int valid = min(32, N - ((t0 + t) * KT + 32 * c));      // tokens of this thread's half
            pipe_wait_one(pp, BAR_S_FULL + 2 * mb + b, kTimeoutTile);
            tc_fence_after_sync();
            float sv[32];
            {
                uint32_t ra[32];
                tmem_ld32(pp.tmem + TM_S + 128 * b + 64 * mb + 32 * c + lane_base, ra);
                tmem_ld_wait();
                tc_fence_before_sync();
                pipe_arrive(pp, BAR_S_EMPTY + 2 * mb + b);
                if (has_bias) {                              // logits in natural units: scale1 * a.k + b1
                    const unsigned char* sB = smem + OFF_RING + s * kStage + 2 * kTile + row * 128;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint4 raw = *reinterpret_cast<const uint4*>(sB + (((4 * c + j) ^ (row & 7)) << 4));
                        const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {            // packed pairs: one instruction per two logits
                            const float2 r2 = ffma2(make_float2(__uint_as_float(ra[8 * j + 2 * k]), __uint_as_float(ra[8 * j + 2 * k + 1])),
                                                    make_float2(p.scale, p.scale), unpack2<T>(w4[k]));
                            sv[8 * j + 2 * k] = r2.x; sv[8 * j + 2 * k + 1] = r2.y;
                        }
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 32; ++k) sv[k] = __uint_as_float(ra[k]) * p.scale;
                }
            }
            uint32_t pk[16];
            float corr = 1.f;
            bool resc = false;
            const bool tv = valid > 0;                         // uniform per warp
            if (tv) {
                if (valid < 32) {
#pragma unroll
                    for (int k = 0; k < 32; ++k) if (k >= valid) sv[k] = -INFINITY;
                }
                float mx0 = fmaxf(sv[0], sv[1]), mx1 = fmaxf(sv[2], sv[3]), mx2 = fmaxf(sv[4], sv[5]), mx3 = fmaxf(sv[6], sv[7]);
#pragma unroll
                for (int k = 8; k < 32; k += 8) {
                    mx0 = fmaxf(mx0, fmaxf(sv[k], sv[k + 1]));     mx1 = fmaxf(mx1, fmaxf(sv[k + 2], sv[k + 3]));
                    mx2 = fmaxf(mx2, fmaxf(sv[k + 4], sv[k + 5])); mx3 = fmaxf(mx3, fmaxf(sv[k + 6], sv[k + 7]));
                }
                const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                if (mx > m_ref + kTau) {                       // also the first tile (m_ref = -inf)
                    corr = fast_exp2((m_ref - mx) * kLog2e);
                    resc = started;
                    m_ref = mx;
                    l *= corr;
                }
                const float nb = -m_ref * kLog2e;
                float2 s01 = make_float2(0.f, 0.f), s23 = make_float2(0.f, 0.f);
                const float2 l2e = make_float2(kLog2e, kLog2e), nb2 = make_float2(nb, nb);
#pragma unroll
                for (int k = 0; k < 16; k += 2) {
                    const float2 a0 = ffma2(make_float2(sv[2 * k], sv[2 * k + 1]), l2e, nb2);
                    const float2 a1 = ffma2(make_float2(sv[2 * k + 2], sv[2 * k + 3]), l2e, nb2);
                    const float2 p01 = make_float2(fast_exp2(a0.x), fast_exp2(a0.y));     // exp2(-inf) = 0 past the range
                    const float2 p23 = make_float2(fast_exp2(a1.x), fast_exp2(a1.y));
                    s01 = fadd2(s01, p01); s23 = fadd2(s23, p23);
                    pk[k] = pack2<T>(p01.x, p01.y);
                    pk[k + 1] = pack2<T>(p23.x, p23.y);
                }
                l += (s01.x + s01.y) + (s23.x + s23.y);
                started = true;
            }
            // P of the previous tile has been consumed (and every product into this thread's accumulator is done)
            if (t > 0) { pipe_wait_one(pp, BAR_PV + mb, kTimeoutTile); tc_fence_after_sync(); }
            if (__any_sync(0xffffffffu, resc)) {               // rare: the reference maximum of some row moved
                uint32_t ra[32];
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    tmem_ld32(tO + 32 * hh, ra);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 32; ++k) ra[k] = __float_as_uint(__uint_as_float(ra[k]) * corr);
                    tmem_st32(tO + 32 * hh, ra);
                }
                tmem_st_wait();
            }
            if (tv) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    *reinterpret_cast<uint4*>(smem + OFF_RING + s * kStage + 2 * kTile + row * 128 + (((4 * c + j) ^ (row & 7)) << 4)) =
                        make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
            }
            fence_proxy_async();
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_P_FULL + mb);
        }
        pipe_wait_one(pp, BAR_PV + mb, kTimeoutTile);
        tc_fence_after_sync();
        // both chains are through with the ring before its memory is reused for the exchange below
        asm volatile("bar.sync 3, %0;\n" ::"r"(256 * MB) : "memory");
        // the two token halves of a row meet in shared memory (the ring is drained: every product is done)
        float o[64];
        {
            uint32_t ra[32], rb[32];
            tmem_ld32(tO, ra);
            tmem_ld32(tO + 32, rb);
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                o[k] = started ? __uint_as_float(ra[k]) : 0.f;
                o[32 + k] = started ? __uint_as_float(rb[k]) : 0.f;
            }
        }
        tc_fence_before_sync();
        float* sX = reinterpret_cast<float*>(smem + OFF_RING) + (size_t)row * 68;      // [256][68]: row, m, l
        if (c == 1) {
#pragma unroll
            for (int k = 0; k < 16; ++k) *reinterpret_cast<float4*>(sX + 4 * k) = make_float4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            sX[64] = m_ref; sX[65] = started ? l : 0.f;
        }
        asm volatile("bar.sync %0, 256;\n" ::"r"(1 + mb) : "memory");      // the chain's own barrier
        if (c == 0) {
            const float om = sX[64], ol = sX[65];
            const float mm = fmaxf(m_ref, om);
            const float bs = (mm == -INFINITY) ? 0.f : mm;
            const float wa = fast_exp2((m_ref - bs) * kLog2e), wb = fast_exp2((om - bs) * kLog2e);
            float* part = slab_parts + (size_t)split * pf;
            part[row] = mm * kLog2e;                       // the merge works in log2 units
            part[g.rows_pad + row] = (started ? l : 0.f) * wa + ol * wb;
            float* pacc = part + 2 * (size_t)g.rows_pad + (size_t)row * 64;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float4 xv = *reinterpret_cast<const float4*>(sX + 4 * k);
                *reinterpret_cast<float4*>(pacc + 4 * k) =
                    make_float4(o[4 * k] * wa + xv.x * wb, o[4 * k + 1] * wa + xv.y * wb,
                                o[4 * k + 2] * wa + xv.z * wb, o[4 * k + 3] * wa + xv.w * wb);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc<512>(pp.tmem);
}

// Merge of the slab's partial states into V_A, spread over many blocks: grid (row chunks, slabs), a
// thread per (agent row, four channels), the parts in their fixed order (bit-reproducible).
template <typename T>
__global__ void __launch_bounds__(256) merge_umma_kernel(const float* __restrict__ partials, int parts, int rows_pad,
                                                         int n, int d, T* __restrict__ out) {
    const int slab = blockIdx.y;
    const size_t pf = partial_floats(rows_pad, 64);
    const float* base = partials + (size_t)slab * parts * pf;
    const int groups = d >> 2;                             // d is a multiple of 8
    const int rows_per_block = 256 / 16;
    const int r = blockIdx.x * rows_per_block + (threadIdx.x >> 4), cg = threadIdx.x & 15;
    if (r >= n || cg >= groups) return;
    float mx = -INFINITY, den = 0.f;
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 16
    for (int q = 0; q < parts; ++q) {
        const float* pq = base + q * pf;
        const float mq = __ldcg(pq + r);
        const float lq = __ldcg(pq + rows_pad + r);
        const float4 a = __ldcg(reinterpret_cast<const float4*>(pq + 2 * (size_t)rows_pad + (size_t)r * 64 + 4 * cg));
        const float mn = fmaxf(mx, mq);
        const float bs = (mn == -INFINITY) ? 0.f : mn;
        const float c0 = exp2f(mx - bs), c1 = exp2f(mq - bs);
        den = den * c0 + lq * c1;
        num.x = num.x * c0 + a.x * c1; num.y = num.y * c0 + a.y * c1;
        num.z = num.z * c0 + a.z * c1; num.w = num.w * c0 + a.w * c1;
        mx = mn;
    }
    const float inv = 1.f / den;
    uint2 o;
    o.x = pack2<T>(num.x * inv, num.y * inv);
    o.y = pack2<T>(num.z * inv, num.w * inv);
    *reinterpret_cast<uint2*>(out + ((size_t)slab * n + r) * d + 4 * cg) = o;
}

// ------------------------------------------------------------------------------------- host
bool aggregate_umma_eligible(int dtype, int n_agents, int n_tokens, int d, bool has_bias) {
    if (dtype != kBF16 && dtype != kF16) return false;
    if (n_agents <= 64 || n_agents > 256 || d > 64 || d % 8 != 0 || n_tokens < KT) return false;
    if (has_bias && n_tokens % 8 != 0) return false;        // TMA needs 16-byte aligned bias rows
    return encode_tiled_fn() != nullptr;
}

AggPlan plan_aggregate_umma(int slabs, int n_agents, int n_tokens, int d, int sm_count) {
    (void)d;
    AggPlan pl;
    pl.rows_pad = n_agents <= 128 ? 128 : 256;
    pl.dpad = 64;
    pl.row_blocks = 1;
    const int tiles = (n_tokens + KT - 1) / KT;
    int splits = sm_count / slabs;                          // one block per SM, one wave
    if (splits < 1) splits = 1;
    if (splits > (tiles + 3) / 4) splits = (tiles + 3) / 4; // at least four tiles per block
    if (splits < 1) splits = 1;
    if (splits > 64) splits = 64;
    const int tps = (tiles + splits - 1) / splits;
    pl.splits = (tiles + tps - 1) / tps;
    pl.parts = pl.splits;
    return pl;
}

template <typename T>
static cudaError_t launch_umma_t(const UmmaAggArgs& g, cudaStream_t st) {
    auto kern = aggregate_umma_kernel<T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    dim3 grid(g.a.splits, g.a.slabs);
    kern<<<grid, NT, kSmemBytes, st>>>(g);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dim3 mgrid((g.a.rows + 15) / 16, g.a.slabs);
    merge_umma_kernel<T><<<mgrid, 256, 0, st>>>(g.a.partials, g.a.splits, g.rows_pad, g.a.rows, g.a.d, static_cast<T*>(g.a.out));
    return cudaGetLastError();
}

// cudaErrorNotSupported: a tensor map could not be encoded; the caller falls back to the mma.sync kernel.
cudaError_t launch_aggregate_umma(int dtype, const AttnArgs& p, const AggPlan& plan, cudaStream_t st) {
    UmmaAggArgs g;
    memset(&g, 0, sizeof(g));
    g.a = p;
    g.a.splits = plan.splits;
    g.rows_pad = plan.rows_pad;
    const int tiles = (p.cols + KT - 1) / KT;
    g.tps = (tiles + plan.splits - 1) / plan.splits;
    const uint64_t S = p.slabs, N = p.cols, n = p.rows;
    if (!make_map_2d_u16(&g.tm_a, p.qm, S * n, p.d, 128, 64)) return cudaErrorNotSupported;
    const int batch = p.slabs / p.heads;
    if (!make_map_tok_u16(&g.tm_k, &g.hf_k, p.km, p.lin, batch, p.heads, (long long)N, p.d, 64, true)) return cudaErrorNotSupported;
    if (!make_map_tok_u16(&g.tm_v, &g.hf_v, p.vm, p.lin, batch, p.heads, (long long)N, p.d, 64, true)) return cudaErrorNotSupported;
    if (p.bias && !make_map_2d_u16(&g.tm_b, p.bias, (uint64_t)p.heads * n, N, 128, 64)) return cudaErrorNotSupported;
    if (dtype == kBF16) return launch_umma_t<__nv_bfloat16>(g, st);
    if (dtype == kF16) return launch_umma_t<__half>(g, st);
    return cudaErrorInvalidValue;
}

}  // namespace aa
