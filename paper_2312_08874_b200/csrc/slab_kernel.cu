// The whole module of Eq. 6 for SMALL token counts (N <= 256 per slab, n <= 64 agents, d = 64, 16-bit):
// a slab's Q, K and V stay in shared memory, so every stage works on-chip and nothing but the inputs
// and O crosses HBM; there are no flags between blocks and no partial states.
//
// One block of 18 warps per SM walks a contiguous range of slabs (ordered head by head, so that the
// head's bias tables and filter taps stay in shared memory):
//   warp 16 "producer":   one lane reloads the Q, K and V buffers (TMA, 128-byte swizzle) as soon as their
//                         last reader of the previous slab is done.
//   warp 17 "MMA issuer": one lane issues every tcgen05.mma (accumulators in tensor memory).
//   warps 0-15:           pooling from the resident Q (text under Eq. 6); aggregation softmax: the agent
//                         operand is stacked twice, rows 0-63 take tokens 0-127 and rows 64-127 tokens
//                         128-255, thread = (row, 32 tokens), exact row maximum and sum through shared
//                         memory (Eq. 3, Eq. 5); V_A from the two accumulators; broadcast per 128-token
//                         tile: thread = (query row, 16 agents), softmax with B2, O = P V_A; depthwise 3x3
//                         term straight from the resident V (Eq. 6); one rounded store of O.
// Every mbarrier wait is bounded (pipe.cuh).  No TMA multicast, no clusters.
#include "common.cuh"
#include "kernels.h"
#include "pipe.cuh"

#include <cstring>

namespace aa {

namespace {
constexpr int NC = 512;                // compute threads
constexpr int NT = NC + 64;            // + producer warp + MMA issuer warp
constexpr int kTile = 64 * 128;        // swizzled [64][64] tile of 16-bit elements
constexpr int kTimeoutLoads = 4, kTimeoutRole = 6;

// shared memory (bytes from a 1024-aligned base)
constexpr int OFF_BAR = 0;
constexpr int OFF_RED = 1024;                            // exchange of row maxima and sums (8 KB)
constexpr int OFF_W = OFF_RED + 8192;                    // filter taps [9][64] fp32
constexpr int OFF_AS = 12288;                            // agents stacked twice [128][128 B]; later the broadcast's P
constexpr int OFF_AB = OFF_AS + 2 * kTile;               // agents [64][128 B]
constexpr int OFF_VA = OFF_AB + kTile;                   // agent features [64][128 B]
constexpr int OFF_Q = OFF_VA + kTile;                    // [256][128 B]
constexpr int OFF_K = OFF_Q + 4 * kTile;
constexpr int OFF_V = OFF_K + 4 * kTile;
constexpr int OFF_PG = OFF_V + 4 * kTile;                // aggregation P [128][2 x 128 B]; then V_A exchange; then the patch
constexpr int OFF_BIAS = OFF_PG + 4 * kTile;             // B1 [n][N] flat, then B2 [N][n] flat
static_assert(OFF_W + 9 * 64 * 4 <= OFF_AS, "small buffers");
constexpr int kSmemMax = 232448;

// mbarriers
constexpr int BAR_Q_FULL = 0, BAR_K_FULL = 1, BAR_V_FULL = 2;        // tx
constexpr int BAR_Q_EMPTY = 3, BAR_K_EMPTY = 4;                       // commit
constexpr int BAR_V_EMPTY = 5;                                        // NC arrivals
constexpr int BAR_A_READY = 6, BAR_VA_READY = 11, BAR_PB_FULL = 12;   // one arrival
constexpr int BAR_SG_FULL = 7, BAR_SB_FULL = 8, BAR_PVG = 10, BAR_PVB = 13;   // commit
constexpr int BAR_PG_FULL = 9;                                        // NC arrivals
constexpr int kBars = 14;

// tensor memory columns
constexpr uint32_t TM_SG = 0;          // aggregation logits [128 lanes][256]
constexpr uint32_t TM_OG = 256;        // aggregation accumulators: 2 x 64
constexpr uint32_t TM_SB = 384;        // broadcast logits: 2 tiles x 64
constexpr uint32_t TM_OB = 0;          // broadcast output (over the dead aggregation logits)

struct SlabArgs {
    const void *q, *k, *v, *b1, *b2, *dwc_w;
    void* out;
    int* status;
    int slabs, heads, H, W, n, p, items_per_block;
    float scale1, scale2;
    int bias_bytes;                    // bytes reserved for each of B1 and B2 in shared memory
    alignas(64) CUtensorMap tm_q, tm_k, tm_v;
};

__device__ __forceinline__ int swz(int row, int col) {
    return row * 128 + ((((col >> 3) ^ row) & 7) << 4) + (col & 7) * 2;
}
__device__ __forceinline__ void sync_compute() { asm volatile("bar.sync 1, %0;\n" ::"n"(NC) : "memory"); }
}  // namespace

template <typename T>
__global__ void __launch_bounds__(NT, 1) slab_kernel(const __grid_constant__ SlabArgs p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_dead;
    __shared__ uint32_t s_tmem;
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = p.H, W = p.W, N = H * W, n = p.n, P = p.p;
    const int ntile = (N + 127) >> 7;                      // 128-token broadcast tiles
    const bool has_b1 = p.b1 != nullptr, has_b2 = p.b2 != nullptr, has_dwc = p.dwc_w != nullptr;
    const int item0 = blockIdx.x * p.items_per_block;
    const int item1 = min(p.slabs, item0 + p.items_per_block);
    const int B = p.slabs / p.heads;                       // items are ordered head by head: item = head * B + b

    Pipe pp;
    pp.status = p.status;
    pp.dead = &s_dead;
    pp.bars = smem_u32(smem + OFF_BAR);
    pp.ph = 0u;
    if (tid == 0) {
        s_dead = 0;
        for (int i = 0; i < kBars; ++i)
            mbar_init(pp.bars + 8 * i, (i == BAR_V_EMPTY || i == BAR_PG_FULL) ? (uint32_t)NC : 1u);
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc<512>(smem_u32(&s_tmem));
    // operand buffers that are only ever written in part start as zeros (padded agent rows)
    for (int e = tid; e < (4 * kTile) / 16; e += NT) reinterpret_cast<uint4*>(smem + OFF_AS)[e] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem = s_tmem;

    const uint32_t sQ = smem_u32(smem + OFF_Q), sK = smem_u32(smem + OFF_K), sV = smem_u32(smem + OFF_V);

    if (warp == 16) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            for (int it = item0; it < item1; ++it) {
                const int slab = (it % B) * p.heads + it / B;
                const int row0 = slab * N;
                if (it > item0) pipe_wait_one(pp, BAR_K_EMPTY, kTimeoutRole);
                mbar_arrive_expect_tx(pipe_bar(pp, BAR_K_FULL), 4 * kTile);
                for (int t = 0; t < 4; ++t) tma_load_2d(sK + t * kTile, &p.tm_k, 0, row0 + 64 * t, pipe_bar(pp, BAR_K_FULL));
                if (it > item0) pipe_wait_one(pp, BAR_Q_EMPTY, kTimeoutRole);
                mbar_arrive_expect_tx(pipe_bar(pp, BAR_Q_FULL), 4 * kTile);
                for (int t = 0; t < 4; ++t) tma_load_2d(sQ + t * kTile, &p.tm_q, 0, row0 + 64 * t, pipe_bar(pp, BAR_Q_FULL));
                if (it > item0) pipe_wait_one(pp, BAR_V_EMPTY, kTimeoutRole);
                mbar_arrive_expect_tx(pipe_bar(pp, BAR_V_FULL), 4 * kTile);
                for (int t = 0; t < 4; ++t) tma_load_2d(sV + t * kTile, &p.tm_v, 0, row0 + 64 * t, pipe_bar(pp, BAR_V_FULL));
            }
        }
        __syncwarp();
    } else if (warp == 17) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t id128 = umma_idesc(fmt, 128, 128, 0), id64 = umma_idesc(fmt, 128, 64, 0), idMN = umma_idesc(fmt, 128, 64, 1);
            const uint64_t dAS = umma_desc_sw128(smem_u32(smem + OFF_AS)), dAB = umma_desc_sw128(smem_u32(smem + OFF_AB));
            const uint64_t dVA = umma_desc_sw128(smem_u32(smem + OFF_VA)), dPG = umma_desc_sw128(smem_u32(smem + OFF_PG));
            const uint64_t dQ = umma_desc_sw128(sQ), dK = umma_desc_sw128(sK), dV = umma_desc_sw128(sV);
            const int n16 = (n + 15) >> 4;
            // descriptor start addresses count 16-byte units: + 2 per K-step of a K-major operand, + 128 per K-step
            // of an MN-major operand (16 rows), + 512 per 64-row tile
            for (int it = item0; it < item1; ++it) {
                pipe_wait_one(pp, BAR_A_READY, kTimeoutRole);
                pipe_wait_one(pp, BAR_K_FULL, kTimeoutLoads);
                tc_fence_after_sync();
                for (int hh = 0; hh < 2; ++hh) {             // logits of tokens 128 hh .. 128 hh + 127 against the stacked agents
                    const uint32_t dd = pp.tmem + TM_SG + 128 * hh;
                    umma_f16_c<0>(dd, dAS, dK + 1024 * hh, id128);
                    umma_f16_c<1>(dd, dAS + 2, dK + 1024 * hh + 2, id128);
                    umma_f16_c<1>(dd, dAS + 4, dK + 1024 * hh + 4, id128);
                    umma_f16_c<1>(dd, dAS + 6, dK + 1024 * hh + 6, id128);
                }
                umma_commit(pipe_bar(pp, BAR_SG_FULL));
                umma_commit(pipe_bar(pp, BAR_K_EMPTY));
                pipe_wait_one(pp, BAR_Q_FULL, kTimeoutLoads);
                tc_fence_after_sync();
                for (int t = 0; t < ntile; ++t) {            // broadcast logits of both tiles
                    const uint32_t dd = pp.tmem + TM_SB + 64 * t;
                    umma_f16_c<0>(dd, dQ + 1024 * t, dAB, id64);
                    umma_f16_c<1>(dd, dQ + 1024 * t + 2, dAB + 2, id64);
                    umma_f16_c<1>(dd, dQ + 1024 * t + 4, dAB + 4, id64);
                    umma_f16_c<1>(dd, dQ + 1024 * t + 6, dAB + 6, id64);
                }
                umma_commit(pipe_bar(pp, BAR_SB_FULL));
                umma_commit(pipe_bar(pp, BAR_Q_EMPTY));
                pipe_wait_one(pp, BAR_PG_FULL, kTimeoutRole);
                pipe_wait_one(pp, BAR_V_FULL, kTimeoutLoads);
                tc_fence_after_sync();
                for (int hh = 0; hh < 2; ++hh) {             // rows 64 hh .. 64 hh + 63 of accumulator hh are the real ones
                    const uint32_t dd = pp.tmem + TM_OG + 64 * hh;
#pragma unroll
                    for (int a = 0; a < 2; ++a)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            const uint64_t da = dPG + 1024 * a + 2 * kk, db = dV + 128 * (8 * hh + 4 * a + kk);
                            if (a == 0 && kk == 0) umma_f16_c<0>(dd, da, db, idMN); else umma_f16_c<1>(dd, da, db, idMN);
                        }
                }
                umma_commit(pipe_bar(pp, BAR_PVG));
                pipe_wait_one(pp, BAR_VA_READY, kTimeoutRole);
                for (int t = 0; t < ntile; ++t) {
                    pipe_wait_one(pp, BAR_PB_FULL, kTimeoutRole);
                    tc_fence_after_sync();
                    for (int kk = 0; kk < n16; ++kk)
                        umma_f16(pp.tmem + TM_OB, dAS + 2 * kk, dVA + 128 * kk, idMN, kk > 0);      // P of the tile sits in the stack buffer
                    umma_commit(pipe_bar(pp, BAR_PVB));
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ compute warps
        const int lq = warp & 3, gq = warp >> 2;
        const int r = 32 * lq + lane;                          // tensor-memory lane
        const uint32_t lane_base = ((uint32_t)(32 * lq)) << 16;
        const int half = r >> 6, agent = r & 63;
        float* sRed = reinterpret_cast<float*>(smem + OFF_RED);            // [8][64] maxima | [8][64] sums, or [4][128] x 2
        float* sW = reinterpret_cast<float*>(smem + OFF_W);
        const T* sB1 = reinterpret_cast<const T*>(smem + OFF_BIAS);
        const T* sB2 = reinterpret_cast<const T*>(smem + OFF_BIAS + p.bias_bytes);
        const int win_h = H / P, win_w = W / P, cnt = win_h * win_w;
        const float inv_cnt = 1.f / (float)cnt;
        int cur_head = -1;
        for (int it = item0; it < item1; ++it) {
            const int head = it / B, slab = (it % B) * p.heads + head;
            if (head != cur_head) {                         // the head's bias tables and filter taps
                cur_head = head;
                sync_compute();
                if (has_b1) {
                    const T* g = static_cast<const T*>(p.b1) + (size_t)head * n * N;
                    T* d = reinterpret_cast<T*>(smem + OFF_BIAS);
                    for (int e = tid; e < n * N; e += NC) d[e] = g[e];
                }
                if (has_b2) {
                    const T* g = static_cast<const T*>(p.b2) + (size_t)head * N * n;
                    T* d = reinterpret_cast<T*>(smem + OFF_BIAS + p.bias_bytes);
                    for (int e = tid; e < n * N; e += NC) d[e] = g[e];
                }
                if (has_dwc) {
                    const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * 64 * 9;
                    for (int e = tid; e < 9 * 64; e += NC) sW[(e % 9) * 64 + e / 9] = Elem<T>::to_f32(w[e]);
                }
                sync_compute();
            }
            // ---- agents: window means of the resident Q, written as both operands
            pipe_wait(pp, BAR_Q_FULL, kTimeoutLoads);
            for (int e = tid; e < n * 8; e += NC) {
                const int wi = e >> 3, c = e & 7;
                const int y0 = (wi / P) * win_h, x0 = (wi % P) * win_w;
                float acc[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] = 0.f;
                for (int i = 0; i < cnt; ++i) {
                    const int tok = (y0 + i / win_w) * W + x0 + i % win_w;
                    float f[8];
                    unpack16<T>(*reinterpret_cast<const uint4*>(smem + OFF_Q + tok * 128 + ((c ^ (tok & 7)) << 4)), f);
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] += f[k];
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] *= inv_cnt;
                const uint4 v = pack16<T>(acc);
                const int off = wi * 128 + ((c ^ (wi & 7)) << 4);
                *reinterpret_cast<uint4*>(smem + OFF_AB + off) = v;
                *reinterpret_cast<uint4*>(smem + OFF_AS + off) = v;
                *reinterpret_cast<uint4*>(smem + OFF_AS + kTile + off) = v;        // rows 64 .. 127: the same agents
            }
            fence_proxy_async();
            sync_compute();
            if (tid == 0) pipe_arrive(pp, BAR_A_READY);

            // ---- aggregation: thread = (stacked agent row, 32 tokens); exact softmax over all N tokens
            pipe_wait(pp, BAR_SG_FULL, kTimeoutRole);
            tc_fence_after_sync();
            float sv[32];
            {
                uint32_t ra[32];
                tmem_ld32(pp.tmem + TM_SG + 128 * half + 32 * gq + lane_base, ra);
                tmem_ld_wait();
                const int tok0 = 128 * half + 32 * gq;
                if (has_b1 && agent < n) {
                    const uint32_t e0 = (uint32_t)agent * N + tok0;             // element index in the flat table
                    const uint32_t* w32 = reinterpret_cast<const uint32_t*>(sB1) + (e0 >> 1);
                    const int sh = (e0 & 1) * 16;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        float2 bb = make_float2(0.f, 0.f);
                        if (tok0 + 2 * j < N) bb = unpack2<T>(__funnelshift_r(w32[j], w32[j + 1], sh));
                        sv[2 * j] = fmaf(__uint_as_float(ra[2 * j]), p.scale1, bb.x);
                        sv[2 * j + 1] = fmaf(__uint_as_float(ra[2 * j + 1]), p.scale1, bb.y);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 32; ++k) sv[k] = __uint_as_float(ra[k]) * p.scale1;
                }
#pragma unroll
                for (int k = 0; k < 32; ++k) if (tok0 + k >= N) sv[k] = -INFINITY;
            }
            float mx = sv[0];
#pragma unroll
            for (int k = 1; k < 32; ++k) mx = fmaxf(mx, sv[k]);
            sRed[(4 * half + gq) * 64 + agent] = mx;
            sync_compute();
#pragma unroll
            for (int q = 0; q < 8; ++q) mx = fmaxf(mx, sRed[q * 64 + agent]);
            {
                const float nb = -mx * kLog2e;
                float sum = 0.f;
                uint32_t pk[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const float p0 = fast_exp2(fmaf(sv[2 * k], kLog2e, nb));          // exp2(-inf) = 0 past the last token
                    const float p1 = fast_exp2(fmaf(sv[2 * k + 1], kLog2e, nb));
                    sum += p0 + p1;
                    pk[k] = pack2<T>(p0, p1);
                }
                sRed[512 + (4 * half + gq) * 64 + agent] = sum;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    *reinterpret_cast<uint4*>(smem + OFF_PG + (gq >> 1) * 2 * kTile + r * 128 + (((4 * (gq & 1) + j) ^ (r & 7)) << 4)) =
                        make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
            }
            fence_proxy_async();
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_PG_FULL);

            // ---- V_A: rows of the two accumulators meet in shared memory, normalised, written as the B operand
            pipe_wait(pp, BAR_PVG, kTimeoutRole);
            tc_fence_after_sync();
            {
                uint32_t ro[16];
                tmem_ld16(pp.tmem + TM_OG + 64 * half + 16 * gq + lane_base, ro);
                tmem_ld_wait();
                float* sX = reinterpret_cast<float*>(smem + OFF_PG);           // [64][64]: the upper rows' share
                if (half == 1) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *reinterpret_cast<float4*>(sX + agent * 64 + 16 * gq + 4 * k) =
                            make_float4(__uint_as_float(ro[4 * k]), __uint_as_float(ro[4 * k + 1]), __uint_as_float(ro[4 * k + 2]), __uint_as_float(ro[4 * k + 3]));
                }
                sync_compute();
                if (half == 0 && agent < n) {
                    float l = 0.f;
#pragma unroll
                    for (int q = 0; q < 8; ++q) l += sRed[512 + q * 64 + agent];
                    const float inv = 1.f / l;
                    float o[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) o[k] = (__uint_as_float(ro[k]) + sX[agent * 64 + 16 * gq + k]) * inv;
                    *reinterpret_cast<uint4*>(smem + OFF_VA + agent * 128 + (((2 * gq) ^ (agent & 7)) << 4)) = pack16<T>(o);
                    *reinterpret_cast<uint4*>(smem + OFF_VA + agent * 128 + (((2 * gq + 1) ^ (agent & 7)) << 4)) = pack16<T>(o + 8);
                }
                tc_fence_before_sync();
                fence_proxy_async();
                sync_compute();
                if (tid == 0) pipe_arrive(pp, BAR_VA_READY);
            }

            // ---- broadcast, one 128-token tile at a time: thread = (query row, 16 agents)
            pipe_wait(pp, BAR_SB_FULL, kTimeoutRole);
            if (has_dwc) pipe_wait(pp, BAR_V_FULL, kTimeoutLoads);
            tc_fence_after_sync();
            T* gO = static_cast<T*>(p.out) + (size_t)slab * N * 64;
            float* sPatch = reinterpret_cast<float*>(smem + OFF_PG);          // [128][64] fp32, 16-byte chunks XORed with the row
            for (int t = 0; t < ntile; ++t) {
                const int tok = 128 * t + r;
                float s16[16];
                {
                    uint32_t ro[16];
                    tmem_ld16(pp.tmem + TM_SB + 64 * t + 16 * gq + lane_base, ro);
                    tmem_ld_wait();
                    if (has_b2 && tok < N) {
                        const uint32_t e0 = (uint32_t)tok * n + 16 * gq;
                        const uint32_t* w32 = reinterpret_cast<const uint32_t*>(sB2) + (e0 >> 1);
                        const int sh = (e0 & 1) * 16;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float2 bb = make_float2(0.f, 0.f);
                            if (16 * gq + 2 * j < n) bb = unpack2<T>(__funnelshift_r(w32[j], w32[j + 1], sh));
                            s16[2 * j] = fmaf(__uint_as_float(ro[2 * j]), p.scale2, bb.x);
                            s16[2 * j + 1] = fmaf(__uint_as_float(ro[2 * j + 1]), p.scale2, bb.y);
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 16; ++k) s16[k] = __uint_as_float(ro[k]) * p.scale2;
                    }
#pragma unroll
                    for (int k = 0; k < 16; ++k) if (16 * gq + k >= n) s16[k] = -INFINITY;
                }
                float mx2 = s16[0];
#pragma unroll
                for (int k = 1; k < 16; ++k) mx2 = fmaxf(mx2, s16[k]);
                sRed[gq * 128 + r] = mx2;
                sync_compute();
#pragma unroll
                for (int q = 0; q < 4; ++q) mx2 = fmaxf(mx2, sRed[q * 128 + r]);
                {
                    const float nb = -mx2 * kLog2e;
                    float sum = 0.f;
                    uint32_t pk[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float p0 = fast_exp2(fmaf(s16[2 * k], kLog2e, nb));     // exp2(-inf) = 0 past the last agent
                        const float p1 = fast_exp2(fmaf(s16[2 * k + 1], kLog2e, nb));
                        pk[k] = pack2<T>(p0, p1);
                        const float2 q = unpack2<T>(pk[k]);                            // the normaliser sums the rounded weights
                        sum += q.x + q.y;
                    }
                    sRed[512 + gq * 128 + r] = sum;
                    *reinterpret_cast<uint4*>(smem + OFF_AS + r * 128 + (((2 * gq) ^ (r & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    *reinterpret_cast<uint4*>(smem + OFF_AS + r * 128 + (((2 * gq + 1) ^ (r & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
                fence_proxy_async();
                tc_fence_before_sync();
                sync_compute();
                if (tid == 0) pipe_arrive(pp, BAR_PB_FULL);
                pipe_wait(pp, BAR_PVB, kTimeoutRole);
                tc_fence_after_sync();
                {
                    float l = 0.f;
#pragma unroll
                    for (int q = 0; q < 4; ++q) l += sRed[512 + q * 128 + r];
                    const float inv = 1.f / l;
                    uint32_t ro[16];
                    tmem_ld16(pp.tmem + TM_OB + 16 * gq + lane_base, ro);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *reinterpret_cast<float4*>(sPatch + r * 64 + (((4 * gq + k) ^ (r & 15)) << 2)) =
                            make_float4(__uint_as_float(ro[4 * k]) * inv, __uint_as_float(ro[4 * k + 1]) * inv,
                                        __uint_as_float(ro[4 * k + 2]) * inv, __uint_as_float(ro[4 * k + 3]) * inv);
                    tc_fence_before_sync();
                }
                sync_compute();
                // depthwise 3x3 term from the resident V + store: item = (token, 4 channels)
                for (int item = tid; item < 128 * 16; item += NC) {
                    const int i = item >> 4, cq = item & 15;
                    const int g = 128 * t + i;
                    if (g >= N) continue;
                    const float4 a4 = *reinterpret_cast<const float4*>(sPatch + i * 64 + ((cq ^ (i & 15)) << 2));
                    float2 o0 = make_float2(a4.x, a4.y), o1 = make_float2(a4.z, a4.w);
                    if (has_dwc) {
                        const int y = g / W, x = g - y * W;
#pragma unroll
                        for (int u = 0; u < 3; ++u) {
                            const int yy = y + u - 1;
                            if (yy < 0 || yy >= H) continue;
#pragma unroll
                            for (int v = 0; v < 3; ++v) {
                                const int xx = x + v - 1;
                                if (xx < 0 || xx >= W) continue;
                                const int tt = yy * W + xx;
                                const uint2 raw = *reinterpret_cast<const uint2*>(smem + OFF_V + tt * 128 + ((((cq >> 1) ^ tt) & 7) << 4) + (cq & 1) * 8);
                                const float4 w4 = *reinterpret_cast<const float4*>(sW + (u * 3 + v) * 64 + 4 * cq);
                                o0 = ffma2(make_float2(w4.x, w4.y), unpack2<T>(raw.x), o0);
                                o1 = ffma2(make_float2(w4.z, w4.w), unpack2<T>(raw.y), o1);
                            }
                        }
                    }
                    uint2 outw;
                    outw.x = pack2<T>(o0.x, o0.y);
                    outw.y = pack2<T>(o1.x, o1.y);
                    *reinterpret_cast<uint2*>(gO + (size_t)g * 64 + 4 * cq) = outw;
                }
                sync_compute();                              // the patch and the exchange arrays are free again
            }
            pipe_arrive(pp, BAR_V_EMPTY);                    // V (products and stencil) is consumed
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc<512>(pp.tmem);
}

// ------------------------------------------------------------------------------------- host
static int slab_bias_bytes(int n_tokens, int n_agents) { return (n_tokens * n_agents * 2 + 64 + 15) & ~15; }

bool slab_eligible(int dtype, int H, int W, int d, int n_agents) {
    if (dtype != kBF16 && dtype != kF16) return false;
    const int N = H * W;
    if (d != 64 || N < 1 || N > 256 || n_agents < 1 || n_agents > 64) return false;
    int p = 1;
    while (p * p < n_agents) ++p;
    if (p * p != n_agents || H % p != 0 || W % p != 0) return false;
    if (OFF_BIAS + 2 * slab_bias_bytes(N, n_agents) + 1024 > kSmemMax) return false;
    return encode_tiled_fn() != nullptr;
}

template <typename T>
static cudaError_t launch_slab_t(const SlabArgs& a, int grid, int smem, cudaStream_t st) {
    auto kern = slab_kernel<T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, NT, smem, st>>>(a);
    return cudaGetLastError();
}

// cudaErrorNotSupported: a tensor map could not be encoded.
cudaError_t launch_slab(int dtype, const void* q, const void* k, const void* v, const void* b1, const void* b2,
                        const void* dwc_w, void* out, int* status, int slabs, int heads, int H, int W, int n_agents,
                        int pool, float scale1, float scale2, int sm_count, cudaStream_t st) {
    SlabArgs a;
    memset(&a, 0, sizeof(a));
    a.q = q; a.k = k; a.v = v; a.b1 = b1; a.b2 = b2; a.dwc_w = dwc_w; a.out = out; a.status = status;
    a.slabs = slabs; a.heads = heads; a.H = H; a.W = W; a.n = n_agents; a.p = pool;
    a.scale1 = scale1; a.scale2 = scale2;
    const int N = H * W;
    a.bias_bytes = slab_bias_bytes(N, n_agents);
    int grid = sm_count < slabs ? sm_count : slabs;
    a.items_per_block = (slabs + grid - 1) / grid;
    grid = (slabs + a.items_per_block - 1) / a.items_per_block;
    const uint64_t rows = (uint64_t)slabs * N;
    if (!make_map_2d_u16(&a.tm_q, q, rows, 64, 64, 64)) return cudaErrorNotSupported;
    if (!make_map_2d_u16(&a.tm_k, k, rows, 64, 64, 64)) return cudaErrorNotSupported;
    if (!make_map_2d_u16(&a.tm_v, v, rows, 64, 64, 64)) return cudaErrorNotSupported;
    const int smem = OFF_BIAS + 2 * a.bias_bytes + 1024;
    if (dtype == kBF16) return launch_slab_t<__nv_bfloat16>(a, grid, smem, st);
    if (dtype == kF16) return launch_slab_t<__half>(a, grid, smem, st);
    return cudaErrorInvalidValue;
}

}  // namespace aa
