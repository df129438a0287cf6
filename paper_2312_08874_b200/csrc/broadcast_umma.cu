// Agent broadcast O = softmax(scale2 * Q A^T + B2) V_A + DWC(V) (Eq. 3, Eq. 5, Eq. 6) for large agent
// counts (64 < n <= 256, d <= 64, 16-bit elements) on the 5th-generation tensor cores.
//
// Grid: (splits, slabs), one block of 19 warps per SM.  The slab's agents A and agent features V_A stay
// resident in shared memory; a block walks its share of the slab's 128-token tiles.  Per tile the agents
// are taken in blocks of 128 ("steps"): S = Q A_block^T by tcgen05.mma into tensor memory, one step ahead.
//   warp 16 "producer":   one lane issues every TMA copy (Q tiles, B2 tiles) through full/empty mbarriers.
//   warp 17 "MMA issuer": one lane issues the logits; warp 18 issues the products P V_A once the
//                         probabilities of a step are written (two issuing threads, so that neither
//                         instruction stream delays the other).
//   warps 0-15 "row warps": thread (query row, agent group g of 32 columns per step): online softmax over
//                         the steps with its own running maximum, sum and accumulator O_g in tensor memory
//                         (no reduction crosses threads inside the loop).  At the end of a tile the four
//                         groups of a row exchange (max, sum), every thread combines 16 output channels from
//                         the four accumulators, adds the depthwise 3x3 term, rounds once and stores.
// The probabilities of a step overwrite, in place, the bias values that the same thread has just read (same
// rows, same columns of the B2 stage), so P needs no buffer of its own; the room holds the V tokens of the
// depthwise window instead: three runs of 130 consecutive tokens (the tile's own, and those one grid row above
// and below, each with one token more on either side), fetched by TMA with the 128-byte swizzle.
// Every wait is bounded (pipe.cuh).  No TMA multicast, no clusters.
#include "common.cuh"
#include "kernels.h"
#include "pipe.cuh"

#include <cstring>

namespace aa {

namespace {
constexpr int QT = 128;                // query rows per tile
constexpr int NROW = 512;              // row-warp threads
constexpr int NT = NROW + 96;          // + producer warp + two MMA issuer warps (logits, products)
constexpr int kTile = 64 * 128;        // swizzled [64][64] tile of 16-bit elements
constexpr float kTau = 5.5f;
constexpr int kTimeoutTile = 3, kTimeoutLoads = 4, kTimeoutRole = 6;

// shared memory (bytes from a 1024-aligned base)
constexpr int OFF_BAR = 0;
constexpr int OFF_ML = 1024;                             // [4 groups][128 rows] (max, sum)
constexpr int OFF_W = OFF_ML + 4 * 128 * 8;              // filter taps [9][64] fp32
constexpr int OFF_A = 8192;                              // agents [256][128 B]
constexpr int OFF_VA = OFF_A + 4 * kTile;                // agent features [256][128 B]
constexpr int OFF_Q = OFF_VA + 4 * kTile;                // 2 x query tile [128][128 B]
constexpr int OFF_B2 = OFF_Q + 4 * kTile;                // 2 stages x (2 column atoms x [128][128 B]): bias, then probabilities
constexpr int kHaloRows = 136;                           // 130 tokens of a run, rounded up to whole swizzle atoms
constexpr int kHaloSeg = kHaloRows * 128;
constexpr int OFF_H = OFF_B2 + 2 * 4 * kTile;            // 3 runs of V tokens [136][128 B]
constexpr int kSmemBytes = OFF_H + 3 * kHaloSeg + 1024;
static_assert(OFF_W + 9 * 64 * 4 <= OFF_A, "small buffers");
static_assert(kSmemBytes <= 232448 && kSmemBytes > 116 * 1024, "one block per SM");

// mbarriers                                   count          waiter
constexpr int BAR_AG = 0;          //          tx             row warps
constexpr int BAR_PREP = 1;        //          1              MMA issuer      V_A pad rows zeroed
constexpr int BAR_Q_FULL = 2;      // [2]      tx             MMA issuer
constexpr int BAR_Q_EMPTY = 4;     // [2]      commit         producer
constexpr int BAR_B_FULL = 6;      // [2]      tx             row warps
constexpr int BAR_B_EMPTY = 8;     // [2]      commit         producer        the product that read the stage is done
constexpr int BAR_S_FULL = 10;     // [2]      commit         row warps
constexpr int BAR_S_EMPTY = 12;    // [2]      row threads    MMA issuer
constexpr int BAR_P_FULL = 14;     //          row threads    MMA issuer
constexpr int BAR_PV = 15;         //          commit         row warps
constexpr int BAR_H_FULL = 16;     //          tx             row warps       V tokens of the tile's depthwise window
constexpr int BAR_H_EMPTY = 17;    //          row threads    producer
constexpr int kBars = 18;

// tensor memory: logits 2 buffers x 128 columns, accumulators 4 groups x 64 columns
constexpr uint32_t TM_S = 0, TM_O = 256;

struct UmmaBcArgs {
    AttnArgs a;
    int MB, tps;                       // 128-agent blocks (1 or 2), tiles per split
    int hf_q, hf_h;                    // dimension order of the Q and V maps (tma_load_tok)
    alignas(64) CUtensorMap tm_q, tm_a, tm_va, tm_b, tm_h;     // tm_h: V with 136-token boxes
};
}  // namespace

template <typename T>
__global__ void __launch_bounds__(NT, 1) broadcast_umma_kernel(const __grid_constant__ UmmaBcArgs g) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_dead;
    __shared__ uint32_t s_tmem;
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const AttnArgs& p = g.a;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, slab = blockIdx.y;
    const int head = slab % p.heads;
    const int N = p.rows, n = p.cols, d = p.d;
    const int MB = g.MB;
    const bool has_b2 = p.bias != nullptr, has_dwc = p.dwc_w != nullptr;
    const int tiles_all = (N + QT - 1) / QT;
    const int i0 = split * g.tps, i1 = min(tiles_all, i0 + g.tps);
    const int tiles = i1 - i0;                            // >= 1 by the plan
    const int steps = tiles * MB;

    Pipe pp;
    pp.status = p.status;
    pp.dead = &s_dead;
    pp.bars = smem_u32(smem + OFF_BAR);
    pp.ph = 0u;
    if (tid == 0) {
        s_dead = 0;
        for (int i = 0; i < kBars; ++i) {
            const bool many = i == BAR_S_EMPTY || i == BAR_S_EMPTY + 1 || i == BAR_P_FULL || i == BAR_H_EMPTY;
            mbar_init(pp.bars + 8 * i, many ? (uint32_t)NROW : 1u);
        }
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc<512>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem = s_tmem;

    const uint32_t sA = smem_u32(smem + OFF_A), sVA = smem_u32(smem + OFF_VA), sQ = smem_u32(smem + OFF_Q);
    const uint32_t sB2 = smem_u32(smem + OFF_B2), sH = smem_u32(smem + OFF_H);

    if (warp == 16) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            mbar_arrive_expect_tx(pipe_bar(pp, BAR_AG), (uint32_t)MB * 4 * kTile);
            for (int mb = 0; mb < MB; ++mb) {
                tma_load_2d(sA + mb * 2 * kTile, &g.tm_a, 0, slab * n + 128 * mb, pipe_bar(pp, BAR_AG));
                tma_load_2d(sVA + mb * 2 * kTile, &g.tm_va, 0, slab * n + 128 * mb, pipe_bar(pp, BAR_AG));
            }
            for (int i = 0; i < tiles; ++i) {
                const int tok0 = (i0 + i) * QT;
                if (i >= 2) pipe_wait_one(pp, BAR_Q_EMPTY + (i & 1), kTimeoutRole);
                mbar_arrive_expect_tx(pipe_bar(pp, BAR_Q_FULL + (i & 1)), 2 * kTile);
                tma_load_tok(sQ + (i & 1) * 2 * kTile, &g.tm_q, g.hf_q, tok0, head, slab / p.heads, pipe_bar(pp, BAR_Q_FULL + (i & 1)));
                if (has_dwc) {
                    // runs of tokens one grid row above, around and below the tile, each from one token before
                    // it (tokens outside the slab are zero-filled)
                    if (i >= 1) pipe_wait_one(pp, BAR_H_EMPTY, kTimeoutRole);
                    mbar_arrive_expect_tx(pipe_bar(pp, BAR_H_FULL), 3 * kHaloSeg);
                    for (int u = 0; u < 3; ++u)
                        tma_load_tok(sH + u * kHaloSeg, &g.tm_h, g.hf_h, tok0 + (u - 1) * p.W - 1, head, slab / p.heads, pipe_bar(pp, BAR_H_FULL));
                }
                if (has_b2)
                    for (int a = 0; a < MB; ++a) {
                        const int j = i * MB + a, b = j & 1;
                        if (j >= 2) pipe_wait_one(pp, BAR_B_EMPTY + b, kTimeoutRole);
                        const uint32_t bar = pipe_bar(pp, BAR_B_FULL + b);
                        mbar_arrive_expect_tx(bar, 4 * kTile);
                        tma_load_2d(sB2 + b * 4 * kTile, &g.tm_b, 128 * a, head * N + tok0, bar);
                        tma_load_2d(sB2 + b * 4 * kTile + 2 * kTile, &g.tm_b, 128 * a + 64, head * N + tok0, bar);
                    }
            }
            for (int i = max(0, tiles - 2); i < tiles; ++i) pipe_wait_one(pp, BAR_Q_EMPTY + (i & 1), kTimeoutRole);
            if (has_b2)
                for (int j = max(0, steps - 2); j < steps; ++j) pipe_wait_one(pp, BAR_B_EMPTY + (j & 1), kTimeoutRole);
            if (has_dwc) pipe_wait_one(pp, BAR_H_EMPTY, kTimeoutRole);
        }
        __syncwarp();
    } else if (warp == 17) {
        // ------------------------------------------------------------------ MMA issuer: logits, one step ahead
        {     // (the whole warp runs the loop; one elected lane issues)
            const uint32_t idS = umma_idesc(fmt, 128, 128, 0);
            const uint64_t dA = umma_desc_sw128(sA), dQ = umma_desc_sw128(sQ);
            // descriptor start addresses count 16-byte units: + 2 per K-step of a K-major operand (32 bytes),
            // + 1024 per 16 KB
            pipe_wait_one(pp, BAR_PREP, kTimeoutLoads);
            for (int j = 0; j < steps; ++j) {
                const int i = j / MB, a = j - i * MB, b = j & 1;
                if (j >= 2) pipe_wait_one(pp, BAR_S_EMPTY + b, kTimeoutRole);
                if (a == 0) pipe_wait_one(pp, BAR_Q_FULL + (i & 1), kTimeoutLoads);
                tc_fence_after_sync();
                const uint32_t dd = pp.tmem + TM_S + 128 * b;
                const uint64_t da = dQ + 1024 * (i & 1), db = dA + 1024 * a;
                umma_ss_w(dd, da, db, idS, 0u);
                umma_ss_w(dd, da + 2, db + 2, idS, 1u);
                umma_ss_w(dd, da + 4, db + 4, idS, 1u);
                umma_ss_w(dd, da + 6, db + 6, idS, 1u);
                if (a == MB - 1) umma_commit_w(pipe_bar(pp, BAR_Q_EMPTY + (i & 1)));
                umma_commit_w(pipe_bar(pp, BAR_S_FULL + b));
            }
            for (int j = max(0, steps - 2); j < steps; ++j) pipe_wait_one(pp, BAR_S_EMPTY + (j & 1), kTimeoutRole);
        }
        __syncwarp();
    } else if (warp == 18) {
        // ------------------------------------------------------------------ MMA issuer: products P V_A
        {     // (the whole warp runs the loop; one elected lane issues)
            const uint32_t idMN = umma_idesc(fmt, 128, 64, 1);
            const uint64_t dVA = umma_desc_sw128(sVA), dP0 = umma_desc_sw128(sB2);
            // + 128 per K-step of an MN-major operand (16 rows of 128 bytes)
            pipe_wait_one(pp, BAR_PREP, kTimeoutLoads);
            unsigned started = 0u;
            for (int j = 0; j < steps; ++j) {
                const int a = j % MB;
                if (a == 0) started = 0u;
                pipe_wait_one(pp, BAR_P_FULL, kTimeoutRole);
                tc_fence_after_sync();
                const uint64_t dP = dP0 + 2048 * (j & 1);             // the step's stage: 32 KB = 2048 units
                for (int gq = 0; gq < 4; ++gq) {
                    if (128 * a + 32 * gq >= n) break;
                    const uint32_t dd = pp.tmem + TM_O + 64 * gq;
                    const uint64_t da = dP + 1024 * (gq >> 1) + 4 * (gq & 1), db = dVA + 128 * (8 * a + 2 * gq);
                    if ((started >> gq) & 1u) umma_ss_w(dd, da, db, idMN, 1u); else umma_ss_w(dd, da, db, idMN, 0u);
                    umma_ss_w(dd, da + 2, db + 128, idMN, 1u);
                    started |= 1u << gq;
                }
                if (has_b2) umma_commit_w(pipe_bar(pp, BAR_B_EMPTY + (j & 1)));     // the stage may take the bias of step j + 2
                umma_commit_w(pipe_bar(pp, BAR_PV));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ row warps
        const int gq = (warp >> 2) & 3;                        // agent group: 32 columns of every step
        const int row = 32 * (warp & 3) + lane;                // query row of the tile = tensor-memory lane
        const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
        const uint32_t tO = pp.tmem + TM_O + 64 * gq + lane_base;
        float* sW = reinterpret_cast<float*>(smem + OFF_W);
        float2* sML = reinterpret_cast<float2*>(smem + OFF_ML);
        const int H = p.H, W = p.W;
        const int c0 = 16 * gq;                                // this thread's output channels
        const int nch = max(0, min(16, d - c0));               // 0, 8 or 16
        // set-up: filter taps, zero rows of V_A past the last agent (0 * NaN is not 0)
        if (has_dwc) {
            const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * d * 9;
            for (int e = tid; e < 9 * 64; e += NROW) {
                const int tap = e >> 6, ch = e & 63;
                sW[e] = ch < d ? Elem<T>::to_f32(w[ch * 9 + tap]) : 0.f;
            }
        }
        pipe_wait_one(pp, BAR_AG, kTimeoutLoads);
        for (int e = tid; e < (128 * MB - n) * 8; e += NROW)
            *(reinterpret_cast<uint4*>(smem + OFF_VA + (n + (e >> 3)) * 128) + (e & 7)) = make_uint4(0u, 0u, 0u, 0u);
        fence_proxy_async();
        asm volatile("bar.sync 1, %0;\n" ::"n"(NROW) : "memory");
        if (tid == 0) pipe_arrive(pp, BAR_PREP);

        T* gO = static_cast<T*>(p.out) + tok_offset(p.lout, slab, p.heads, 0);
        const size_t so = (size_t)p.lout.st;
        for (int i = 0; i < tiles; ++i) {
            const int tok = (i0 + i) * QT + row;
            float m_ref = -INFINITY, l = 0.f;
            bool started = false;
            for (int a = 0; a < MB; ++a) {
                const int j = i * MB + a, b = j & 1;
                const int valid = min(32, n - (128 * a + 32 * gq));     // agents of this thread in the step
                const bool tv = valid > 0;                              // uniform per warp
                pipe_wait_one(pp, BAR_S_FULL + b, kTimeoutTile);
                tc_fence_after_sync();
                float sv[32];
                {
                    uint32_t ra[32];
                    tmem_ld32(pp.tmem + TM_S + 128 * b + 32 * gq + lane_base, ra);
                    tmem_ld_wait();
                    tc_fence_before_sync();
                    pipe_arrive(pp, BAR_S_EMPTY + b);
                    if (has_b2) {                            // logits in natural units: scale2 * q.a + b2
                        pipe_wait_one(pp, BAR_B_FULL + b, kTimeoutLoads);
                        const unsigned char* sB = smem + OFF_B2 + b * 4 * kTile + (gq >> 1) * 2 * kTile + row * 128;
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {
                            const uint4 raw = *reinterpret_cast<const uint4*>(sB + (((4 * (gq & 1) + jj) ^ (row & 7)) << 4));
                            const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                            for (int k = 0; k < 4; ++k) {        // packed pairs: one instruction per two logits
                                const float2 r2 = ffma2(make_float2(__uint_as_float(ra[8 * jj + 2 * k]), __uint_as_float(ra[8 * jj + 2 * k + 1])),
                                                        make_float2(p.scale, p.scale), unpack2<T>(w4[k]));
                                sv[8 * jj + 2 * k] = r2.x; sv[8 * jj + 2 * k + 1] = r2.y;
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
                    if (mx > m_ref + kTau) {                   // also the first step (m_ref = -inf)
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
                        const float2 p01 = make_float2(fast_exp2(a0.x), fast_exp2(a0.y));     // exp2(-inf) = 0 past the last agent
                        const float2 p23 = make_float2(fast_exp2(a1.x), fast_exp2(a1.y));
                        s01 = fadd2(s01, p01); s23 = fadd2(s23, p23);
                        pk[k] = pack2<T>(p01.x, p01.y);
                        pk[k + 1] = pack2<T>(p23.x, p23.y);
                    }
                    l += (s01.x + s01.y) + (s23.x + s23.y);
                    started = true;
                }
                // the previous step's product is done: P may be overwritten, this thread's accumulator is at rest
                if (a > 0) { pipe_wait_one(pp, BAR_PV, kTimeoutTile); tc_fence_after_sync(); }
                if (__any_sync(0xffffffffu, resc)) {           // rare: the reference maximum of some row moved
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
                    for (int jj = 0; jj < 4; ++jj)
                        *reinterpret_cast<uint4*>(smem + OFF_B2 + b * 4 * kTile + (gq >> 1) * 2 * kTile + row * 128 + (((4 * (gq & 1) + jj) ^ (row & 7)) << 4)) =
                            make_uint4(pk[4 * jj], pk[4 * jj + 1], pk[4 * jj + 2], pk[4 * jj + 3]);
                }
                fence_proxy_async();
                tc_fence_before_sync();
                pipe_arrive(pp, BAR_P_FULL);
            }
            // depthwise 3x3 term for this thread's 16 channels of its token, while the last product is in flight
            float2 dw[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) dw[k] = make_float2(0.f, 0.f);
            if (has_dwc) {
                // tap (u, v) of this thread's token sits at row (row + v) of run u; taps outside the grid
                // (or in another slab, or past the head dim) contribute nothing
                pipe_wait_one(pp, BAR_H_FULL, kTimeoutLoads);
                const int tk = min(tok, N - 1);
                const int y = tk / W, x = tk - y * W;
                const bool live = tok < N && nch > 0;
#pragma unroll
                for (int u = 0; u < 3; ++u) {
                    const int yy = y + u - 1;
                    const bool rowok = live && yy >= 0 && yy < H;
#pragma unroll
                    for (int v = 0; v < 3; ++v) {
                        const int xx = x + v - 1;
                        const bool ok = rowok && xx >= 0 && xx < W;
                        const int r = row + v;
                        const unsigned char* src = smem + OFF_H + u * kHaloSeg + r * 128;
                        const float4* wt = reinterpret_cast<const float4*>(sW + (u * 3 + v) * 64 + c0);
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            uint4 rr = *reinterpret_cast<const uint4*>(src + ((((c0 >> 3) + hh) ^ (r & 7)) << 4));
                            if (!ok || (hh == 1 && nch <= 8)) rr = make_uint4(0u, 0u, 0u, 0u);
                            const float4 w0 = wt[2 * hh], w1 = wt[2 * hh + 1];
                            dw[4 * hh + 0] = ffma2(make_float2(w0.x, w0.y), unpack2<T>(rr.x), dw[4 * hh + 0]);
                            dw[4 * hh + 1] = ffma2(make_float2(w0.z, w0.w), unpack2<T>(rr.y), dw[4 * hh + 1]);
                            dw[4 * hh + 2] = ffma2(make_float2(w1.x, w1.y), unpack2<T>(rr.z), dw[4 * hh + 2]);
                            dw[4 * hh + 3] = ffma2(make_float2(w1.z, w1.w), unpack2<T>(rr.w), dw[4 * hh + 3]);
                        }
                    }
                }
                pipe_arrive(pp, BAR_H_EMPTY);
            }
            sML[gq * 128 + row] = make_float2(started ? m_ref : -INFINITY, started ? l : 0.f);
            pipe_wait_one(pp, BAR_PV, kTimeoutTile);
            tc_fence_after_sync();
            asm volatile("bar.sync 1, %0;\n" ::"n"(NROW) : "memory");
            {
                float2 ml[4];
                float mm = -INFINITY;
#pragma unroll
                for (int q = 0; q < 4; ++q) { ml[q] = sML[q * 128 + row]; mm = fmaxf(mm, ml[q].x); }
                float wgt[4], den = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    wgt[q] = fast_exp2((ml[q].x - mm) * kLog2e);        // exp2(-inf) = 0 for a group without agents
                    den += wgt[q] * ml[q].y;
                }
                float acc[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) acc[k] = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t ro[16];
                    tmem_ld16(pp.tmem + TM_O + 64 * q + c0 + lane_base, ro);
                    tmem_ld_wait();
                    if (ml[q].y > 0.f) {                               // uniform enough: skip accumulators never written
#pragma unroll
                        for (int k = 0; k < 16; ++k) acc[k] = fmaf(wgt[q], __uint_as_float(ro[k]), acc[k]);
                    }
                }
                tc_fence_before_sync();
                const float inv = 1.f / den;
                if (tok < N && nch > 0) {
                    float o8[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) o8[k] = fmaf(acc[k], inv, (k & 1) ? dw[k >> 1].y : dw[k >> 1].x);
                    *reinterpret_cast<uint4*>(gO + (size_t)tok * so + c0) = pack16<T>(o8);
                    if (nch > 8) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) o8[k] = fmaf(acc[8 + k], inv, (k & 1) ? dw[4 + (k >> 1)].y : dw[4 + (k >> 1)].x);
                        *(reinterpret_cast<uint4*>(gO + (size_t)tok * so + c0) + 1) = pack16<T>(o8);
                    }
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc<512>(pp.tmem);
}

// ------------------------------------------------------------------------------------- host
bool broadcast_umma_eligible(int dtype, int n_agents, int n_tokens, int d) {
    if (dtype != kBF16 && dtype != kF16) return false;
    if (n_agents <= 64 || n_agents > 256 || n_agents % 8 != 0 || d > 64 || d % 8 != 0 || n_tokens < QT) return false;
    return encode_tiled_fn() != nullptr;
}

template <typename T>
static cudaError_t launch_bc_umma_t(const UmmaBcArgs& g, int splits, cudaStream_t st) {
    auto kern = broadcast_umma_kernel<T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    dim3 grid(splits, g.a.slabs);
    kern<<<grid, NT, kSmemBytes, st>>>(g);
    return cudaGetLastError();
}

// cudaErrorNotSupported: a tensor map could not be encoded.
cudaError_t launch_broadcast_umma(int dtype, const AttnArgs& p, int sm_count, cudaStream_t st) {
    UmmaBcArgs g;
    memset(&g, 0, sizeof(g));
    g.a = p;
    g.MB = p.cols <= 128 ? 1 : 2;
    const int tiles = (p.rows + QT - 1) / QT;
    int splits = sm_count / p.slabs;                        // one block per SM, one wave
    if (splits < 1) splits = 1;
    if (splits > tiles) splits = tiles;
    g.tps = (tiles + splits - 1) / splits;
    splits = (tiles + g.tps - 1) / g.tps;
    const uint64_t S = p.slabs, N = p.rows, n = p.cols;
    const int batch = p.slabs / p.heads;
    if (!make_map_tok_u16(&g.tm_q, &g.hf_q, p.qm, p.lin, batch, p.heads, (long long)N, p.d, 128, true)) return cudaErrorNotSupported;
    if (!make_map_2d_u16(&g.tm_a, p.km, S * n, p.d, 128, 64)) return cudaErrorNotSupported;
    if (!make_map_2d_u16(&g.tm_va, p.vm, S * n, p.d, 128, 64)) return cudaErrorNotSupported;
    if (p.bias && !make_map_2d_u16(&g.tm_b, p.bias, (uint64_t)p.heads * N, n, 128, 64)) return cudaErrorNotSupported;
    if (p.dwc_w && !make_map_tok_u16(&g.tm_h, &g.hf_h, p.dwc_v, p.lin, batch, p.heads, (long long)N, p.d, kHaloRows, true)) return cudaErrorNotSupported;
    if (dtype == kBF16) return launch_bc_umma_t<__nv_bfloat16>(g, splits, st);
    if (dtype == kF16) return launch_bc_umma_t<__half>(g, splits, st);
    return cudaErrorInvalidValue;
}

}  // namespace aa
