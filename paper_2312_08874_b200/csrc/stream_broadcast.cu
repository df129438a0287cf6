// Agent broadcast with the depthwise term, O = softmax(scale2 * Q A^T + B2) V_A + DWC(V) (Eq. 3, Eq. 5, Eq. 6)
// for small agent counts (n <= 64, d = 64, 16-bit elements) as a streaming kernel on the 5th-generation
// tensor cores: both attention products AND the depthwise 3x3 term run on tcgen05.
//
// Persistent blocks, one per SM; block c walks a contiguous run of the (slab, row tile) sequence.  A tile is R
// whole grid rows in a padded token index: row i of every 128-row operand is (tile row r, padded column xp) with
// i = r (W + 2) + xp, xp = 0 and xp = W + 1 being pad positions whose results are dropped (R (W + 2) <= 128).
// The depthwise term on the tensor core: for tap (u, v) the V rows of the tile, with one grid row above and
// below and a zero column at either end (all filled in by one TMA box: coordinates outside the grid read zero),
// sit in shared memory as a K-major, 128-byte-swizzled tile; the swizzle is a function of the address, so an
// operand may start at any row: the tap's operand is the same tile started u (W + 2) + v - 1 rows later.  Times
// a diagonal weight slice (16 channels at a time) it accumulates w[c][u][v] V[y+u-1][x+v-1][c] over the nine
// taps into its own tensor-memory accumulator, in fp32: 36 small instructions per tile and no stencil code.
//   warp 8 "producer":  one lane issues every TMA copy: Q tile and padded-B2 tile (two stages), V rows (two
//       stages), and per slab the agents A (times scale2), V_A and the head's diagonal weight slices.
//   warp 9 "MMA issuer, attention": S = Q A^T + B2 I (the bias through four 16-column identity slices, its pad
//       columns removing the agents past n), one tile ahead; then O = P V_A with P read from tensor memory.
//   warps 10, 11 "MMA issuers, depthwise": the 36 tap instructions of a tile, taps 0-4 and taps 5-8, each into an
//       accumulator of its own (the order of two issuing threads is not defined), ahead of the attention part.
//   warps 0-3 "softmax warps": thread = operand row.  Logits from tensor memory, maximum, fp32 exponentials,
//       their sum (to the output warps through shared memory), probabilities rounded to the operand type back
//       to tensor memory.
//   warps 4-7 "output warps": thread = operand row.  O times 1 / row sum plus the depthwise accumulator,
//       rounded once, stored (pad positions skipped).
// Every wait is bounded.  No TMA multicast, no clusters.
#include "stream_common.cuh"

namespace aa {

namespace {
constexpr int NROW = 128;              // softmax threads, and output threads
constexpr int NT = 2 * NROW + 128;     // + producer warp + three MMA issuer warps
constexpr int kWtBytes = 9 * 2048;     // diagonal weight slices of one head: 9 taps x [16][128 B]
constexpr int kTimeoutTile = 3, kTimeoutLoads = 4, kTimeoutRole = 6;

// shared memory (bytes from a 1024-aligned base)
constexpr int OFF_BAR = 0;
constexpr int OFF_L = 256;             // [2][128] row sums of the probabilities (fp32)
constexpr int OFF_I16 = 2048;          // [16][128 B]: identity slice, K-major B operand of the bias steps
constexpr int OFF_A2 = 4096;           // 2 x agents [64][128 B]
constexpr int OFF_VA = OFF_A2 + 2 * 8192;   // 2 x agent features [64][128 B]
constexpr int OFF_WT = OFF_VA + 2 * 8192;   // 2 x diagonal weight slices
constexpr int OFF_QB = OFF_WT + 2 * kWtBytes;   // 2 stages x (Q tile | B2 tile), then 2 stages of V rows with guards
static_assert(OFF_QB % 1024 == 0, "swizzled tiles need 1024-byte alignment");

struct BcLayout {
    int wp, tq, qsz, hsz, off_h, total;
};
__host__ __device__ inline BcLayout bc_layout(int R, int W) {
    BcLayout l;
    l.wp = W + 2;
    l.tq = R * l.wp;                                         // operand rows that hold (padded) tokens
    l.qsz = (l.tq * 128 + 1023) / 1024 * 1024;
    // V rows: (R + 2) (W + 2) rows, one guard KB before (tap (0,0) starts one row early) and room after for
    // the 128-row operand of the last tap (read, never used)
    l.hsz = 1024 + ((2 * l.wp + 1 + 128) * 128 + 1023) / 1024 * 1024;
    if (l.hsz < 1024 + ((R + 2) * l.wp * 128 + 1023) / 1024 * 1024) l.hsz = 1024 + ((R + 2) * l.wp * 128 + 1023) / 1024 * 1024;
    l.off_h = OFF_QB + 4 * l.qsz + 2048;                     // (the last Q-sized operand read runs up to 2 KB past its tile)
    l.total = l.off_h + 2 * l.hsz;
    return l;
}

// mbarriers                                  count           waiter
constexpr int BAR_OPS = 0;        // [2]       tx              both MMA issuers    agents, agent features, weight slices of a slab
constexpr int BAR_QB_FULL = 2;    // [2]       tx              attention issuer
constexpr int BAR_QB_EMPTY = 4;   // [2]       commit          producer
constexpr int BAR_H_FULL = 6;     // [2]       tx              depthwise issuer
constexpr int BAR_H_EMPTY = 8;    // [2]       2 commits       producer
constexpr int BAR_S_FULL = 10;    // [2]       commit          softmax warps
constexpr int BAR_P_FULL = 12;    // [2]       softmax threads attention issuer
constexpr int BAR_O_FULL = 14;    // [2]       commit          output warps
constexpr int BAR_D_FULL = 16;    // [2]       2 commits       output warps
constexpr int BAR_O_EMPTY = 18;   // [2]       output threads  both MMA issuers, softmax warps (the row sums' buffer)
constexpr int BAR_DRAIN = 20;     // [3]       commit          each MMA issuer, once, at its end
constexpr int kBars = 23;

// tensor memory columns: logits 2 x 64 (the probabilities overwrite the first 32), output 2 x 64,
// depthwise 2 issuers x 2 x 64
constexpr uint32_t TM_S = 0, TM_O = 128, TM_D = 256;

__device__ __forceinline__ int swz16(int row, int col) {
    return row * 128 + ((((col >> 3) ^ row) & 7) << 4) + (col & 7) * 2;
}
// The (slab, tile) pair of a block's i-th tile, advanced without divisions.
struct TileIter {
    int slab, tb, TB;
    __device__ __forceinline__ void next() { if (++tb == TB) { tb = 0; ++slab; } }
};
}  // namespace

template <typename T>
__global__ void __launch_bounds__(NT, 1) stream_broadcast_kernel(const __grid_constant__ StreamArgs p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_dead;
    __shared__ uint32_t s_tmem;
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = p.H, W = p.W, N = H * W, n = p.n;
    const int R = p.plan.rows_b, TB = p.plan.tiles_b;
    const BcLayout L = bc_layout(R, W);
    const bool has_dwc = p.dwc_w != nullptr;
    // this block's run of the (slab, tile) sequence
    const int total = p.slabs * TB;
    const int g0 = (int)((long long)total * blockIdx.x / gridDim.x), g1 = (int)((long long)total * (blockIdx.x + 1) / gridDim.x);
    const int T_ = g1 - g0;
    TileIter it;
    it.slab = g0 / TB; it.tb = g0 - it.slab * TB; it.TB = TB;

    Pipe pp;
    pp.status = p.status;
    pp.dead = &s_dead;
    pp.bars = smem_u32(smem + OFF_BAR);
    pp.ph = 0u;
    if (tid == 0) {
        s_dead = 0;
        for (int i = 0; i < kBars; ++i)
            mbar_init(pp.bars + 8 * i, ((i >= BAR_P_FULL && i < BAR_O_FULL) || (i >= BAR_O_EMPTY && i < BAR_DRAIN)) ? (uint32_t)NROW
                                       : ((i >= BAR_H_EMPTY && i < BAR_S_FULL) || (i >= BAR_D_FULL && i < BAR_O_EMPTY)) ? 2u : 1u);
        mbar_fence_init();
    }
    // constant operand; rows n..63 of the agent tiles never receive data (their copies bring n rows): zero
    for (int e = tid; e < 16 * 64; e += NT) {
        const int r = e >> 6, c = e & 63;
        *reinterpret_cast<uint16_t*>(smem + OFF_I16 + swz16(r, c)) = (r == c) ? (uint16_t)Pair<T>::kOne : (uint16_t)0;
    }
    for (int e = tid; e < 4 * (64 - n) * 8; e += NT) {
        const int buf = e / ((64 - n) * 8), rest = e - buf * ((64 - n) * 8);
        *(reinterpret_cast<uint4*>(smem + OFF_A2 + buf * 8192 + (n + (rest >> 3)) * 128) + (rest & 7)) = make_uint4(0u, 0u, 0u, 0u);
    }
    // (operand rows past the tile's tokens and the guard rows of the V stages are read but never used; they are
    // cleared once so that no NaN pattern of stale shared memory enters a product with a zero weight)
    for (int e = tid; e < (L.total - OFF_QB) / 16; e += NT) *(reinterpret_cast<uint4*>(smem + OFF_QB) + e) = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
    if (warp == 0) tmem_alloc<512>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem = s_tmem;

    const uint32_t sQB = smem_u32(smem + OFF_QB), sH = smem_u32(smem + L.off_h);
    const uint32_t sA2 = smem_u32(smem + OFF_A2), sVA = smem_u32(smem + OFF_VA), sWT = smem_u32(smem + OFF_WT);
    float* sL = reinterpret_cast<float*>(smem + OFF_L);

    if (warp == 8) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            // V is an input of the call: its first two stages are requested before the wait for the preceding kernels
            const uint32_t h_tx = (uint32_t)(R + 2) * L.wp * 128u;
            TileIter ih = it;
            if (has_dwc)
                for (int i = 0; i < min(T_, 2); ++i, ih.next()) {
                    const uint32_t bar = pipe_bar(pp, BAR_H_FULL + i);
                    mbar_arrive_expect_tx(bar, h_tx);
                    tma_load_4d(sH + i * L.hsz + 1024, &p.tm_h, 0, -1, ih.tb * R - 1, ih.slab, bar);
                }
            pdl_wait();      // A, V_A, the padded B2 and the weight slices come from the preceding kernels
            int cur = -1, ord = -1;
            const uint32_t qb_tx = 2u * (uint32_t)L.tq * 128u;
            for (int i = 0; i < T_ && !pipe_dead(pp); ++i, it.next()) {
                if (it.slab != cur) {
                    // (a buffer is reused two slabs later: every product that read it is long done, since the
                    // stage waits below already cover the tiles of the slab in between)
                    cur = it.slab; ++ord;
                    const uint32_t bar = pipe_bar(pp, BAR_OPS + (ord & 1));
                    mbar_arrive_expect_tx(bar, 2u * (uint32_t)n * 128u + (has_dwc ? (uint32_t)kWtBytes : 0u));
                    tma_load_2d(sA2 + (ord & 1) * 8192, &p.tm_a2, 0, it.slab * n, bar);
                    tma_load_2d(sVA + (ord & 1) * 8192, &p.tm_va, 0, it.slab * n, bar);
                    if (has_dwc)
                        bulk_load_1d(sWT + (ord & 1) * kWtBytes, static_cast<const unsigned char*>(p.wt) + (size_t)(it.slab % p.heads) * kWtBytes,
                                     (uint32_t)kWtBytes, bar);
                }
                const int s2 = i & 1;
                if (i >= 2) wait_spin(pp, BAR_QB_EMPTY + s2, (i >> 1) - 1, kTimeoutRole);
                const uint32_t bar = pipe_bar(pp, BAR_QB_FULL + s2), dst = sQB + s2 * 2 * L.qsz;
                mbar_arrive_expect_tx(bar, qb_tx);
                tma_load_4d(dst, &p.tm_q, 0, -1, it.tb * R, it.slab, bar);
                tma_load_4d(dst + L.qsz, &p.tm_b2, 0, -1, it.tb * R, p.b2 ? it.slab % p.heads : 0, bar);
                if (has_dwc && i >= 2) {
                    wait_spin(pp, BAR_H_EMPTY + s2, (i >> 1) - 1, kTimeoutRole);
                    const uint32_t hb = pipe_bar(pp, BAR_H_FULL + s2);
                    mbar_arrive_expect_tx(hb, h_tx);
                    tma_load_4d(sH + s2 * L.hsz + 1024, &p.tm_h, 0, -1, it.tb * R - 1, it.slab, hb);
                }
            }
        }
        __syncwarp();
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer: attention
        {   // (the whole warp runs the loop; one elected lane issues)
            const uint32_t idS = umma_idesc(fmt, 128, 64, 0), idI = umma_idesc(fmt, 128, 16, 0);
            const uint32_t idPV = umma_idesc(fmt, 128, 64, 1);
            const uint64_t dI = umma_desc_sw128(smem_u32(smem + OFF_I16));
            const uint64_t dA2 = umma_desc_sw128(sA2), dVA = umma_desc_sw128(sVA);
            const uint64_t dQ0 = umma_desc_sw128(sQB), dQ1 = dQ0 + (uint64_t)(2 * L.qsz >> 4);
            const uint64_t dB0 = dQ0 + (uint64_t)(L.qsz >> 4), dB1 = dQ1 + (uint64_t)(L.qsz >> 4);
            const uint32_t tS = pp.tmem + TM_S, tO = pp.tmem + TM_O;
            TileIter is = it;                    // slab bookkeeping of the logits (one tile ahead) ...
            int cur_s = -1, ord_s = -1;
            int cur_o = -1, ord_o = -1;          // ... and of the products
            // descriptor start addresses count 16-byte units: + 2 per K-step of a K-major operand (32 bytes),
            // + 128 per K-step of an MN-major operand (16 rows of 128 bytes), + 512 per 8 KB buffer.  `b` is a
            // compile-time constant at every call (the tile loop is unrolled by two).
            auto issue_S = [&](int i, int b) {
                if (is.slab != cur_s) {
                    cur_s = is.slab; ++ord_s;
                    wait_spin(pp, BAR_OPS + (ord_s & 1), ord_s >> 1, kTimeoutLoads);
                }
                is.next();
                wait_spin(pp, BAR_QB_FULL + b, i >> 1, kTimeoutTile);
                tc_fence_after_sync();
                const uint64_t dQ = b ? dQ1 : dQ0, dB = b ? dB1 : dB0;
                const uint64_t da = dA2 + 512 * (ord_s & 1);
                const uint32_t dd = tS + 64 * b;
                umma_ss_w(dd, dQ, da, idS, 0u);
#pragma unroll
                for (int k = 1; k < 4; ++k) umma_ss_w(dd, dQ + 2 * k, da + 2 * k, idS, 1u);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_ss_w(dd + 16 * k, dB + 2 * k, dI, idI, 1u);
                umma_commit_w(pipe_bar(pp, BAR_QB_EMPTY + b));
                umma_commit_w(pipe_bar(pp, BAR_S_FULL + b));
            };
            if (T_ > 0) issue_S(0, 0);
            for (int i0 = 0; i0 < T_ && !pipe_dead(pp); i0 += 2) {
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int i = i0 + b;
                    if (i < T_) {
                        if (i + 1 < T_) issue_S(i + 1, b ^ 1);
                        if (it.slab != cur_o) { cur_o = it.slab; ++ord_o; }
                        it.next();
                        wait_spin(pp, BAR_P_FULL + b, i >> 1, kTimeoutRole);
                        if (i >= 2) wait_spin(pp, BAR_O_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
                        tc_fence_after_sync();
                        const uint32_t tP = tS + 64 * b, dd = tO + 64 * b;
                        const uint64_t dv = dVA + 512 * (ord_o & 1);
                        umma_ts_w(dd, tP, dv, idPV, 0u);
#pragma unroll
                        for (int k = 1; k < 4; ++k) umma_ts_w(dd, tP + 8 * k, dv + 128 * k, idPV, 1u);
                        umma_commit_w(pipe_bar(pp, BAR_O_FULL + b));
                    }
                }
            }
            umma_drain_w(pp, BAR_DRAIN);
        }
        __syncwarp();
    } else if (warp == 10 || warp == 11) {
        // ------------------------------------------------------------------ MMA issuers: depthwise term (taps 0-4 | taps 5-8)
        const int half = warp - 10;
        if (has_dwc) {   // (the whole warp runs the loop; one elected lane issues)
            const uint32_t idW = umma_idesc(fmt, 128, 16, 0);
            const uint64_t dWT = umma_desc_sw128(sWT);
            const uint64_t dH0 = umma_desc_sw128(sH + 1024), dH1 = umma_desc_sw128(sH + L.hsz + 1024);
            const uint32_t tD = pp.tmem + TM_D + 128 * half;
            const int wp8 = L.wp * 8;                        // one grid row of the V tile, in 16-byte descriptor units
            int cur = -1, ord = -1;
            for (int i0 = 0; i0 < T_ && !pipe_dead(pp); i0 += 2) {
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int i = i0 + b;
                    if (i < T_) {
                        if (it.slab != cur) {
                            cur = it.slab; ++ord;
                            wait_spin(pp, BAR_OPS + (ord & 1), ord >> 1, kTimeoutLoads);
                        }
                        it.next();
                        wait_spin(pp, BAR_H_FULL + b, i >> 1, kTimeoutTile);
                        if (i >= 2) wait_spin(pp, BAR_O_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
                        tc_fence_after_sync();
                        const uint64_t dh = (b ? dH1 : dH0) - 8;         // tap (0, 0) starts one row before the tile
                        const uint64_t dw = dWT + (uint64_t)((ord & 1) * (kWtBytes >> 4));
                        const uint32_t dd = tD + 64 * b;
                        // tap (u, v): the V tile started u (W + 2) + v - 1 rows later, times the tap's diagonal slices
#pragma unroll
                        for (int t = 0; t < 5; ++t) {
                            const int tap = t + 5 * half;        // (the second issuer's fifth slot is empty)
                            if (tap < 9) {
                                const int u = tap / 3, v = tap - 3 * u;
                                const uint64_t da = dh + (uint64_t)(u * wp8 + v * 8), db = dw + (uint64_t)(tap * 128);
#pragma unroll
                                for (int g = 0; g < 4; ++g)
                                    umma_ss_w(dd + 16 * g, da + 2 * g, db + 2 * g, idW, t ? 1u : 0u);
                            }
                        }
                        umma_commit_w(pipe_bar(pp, BAR_H_EMPTY + b));
                        umma_commit_w(pipe_bar(pp, BAR_D_FULL + b));
                    }
                }
            }
            umma_drain_w(pp, BAR_DRAIN + 1 + half);
        }
        __syncwarp();
    } else if (warp < 4) {
        // ------------------------------------------------------------------ softmax warps
        const int row = tid;
        const uint32_t lane_base = ((uint32_t)(32 * warp)) << 16;
        const float2 l2e = make_float2(kLog2e, kLog2e);
        for (int i = 0; i < T_; ++i) {
            const int b = i & 1;
            const uint32_t tS = pp.tmem + TM_S + 64 * b + lane_base;
            wait_par(pp, BAR_S_FULL + b, i >> 1, kTimeoutTile);
            tc_fence_after_sync();
            uint32_t sa[32], sb[32];
            tmem_ld32(tS, sa);
            tmem_ld32(tS + 32, sb);
            tmem_ld_wait();
            float m0 = __uint_as_float(sa[0]), m1 = __uint_as_float(sb[0]);
#pragma unroll
            for (int j = 1; j < 31; j += 2) {
                m0 = max3(m0, __uint_as_float(sa[j]), __uint_as_float(sa[j + 1]));
                m1 = max3(m1, __uint_as_float(sb[j]), __uint_as_float(sb[j + 1]));
            }
            const float mx = max3(m0, m1, fmaxf(__uint_as_float(sa[31]), __uint_as_float(sb[31])));
            const float nb = -mx * kLog2e;
            const float2 nb2 = make_float2(nb, nb);
            float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
            uint32_t pk[32];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float2 x0 = ffma2(make_float2(__uint_as_float(sa[2 * j]), __uint_as_float(sa[2 * j + 1])), l2e, nb2);
                const float2 x1 = ffma2(make_float2(__uint_as_float(sb[2 * j]), __uint_as_float(sb[2 * j + 1])), l2e, nb2);
                const float2 e0 = make_float2(fast_exp2(x0.x), fast_exp2(x0.y)), e1 = make_float2(fast_exp2(x1.x), fast_exp2(x1.y));
                s0 = fadd2(s0, e0);
                s1 = fadd2(s1, e1);
                pk[j] = Pair<T>::cvt(e0.x, e0.y);
                pk[16 + j] = Pair<T>::cvt(e1.x, e1.y);
            }
            tmem_st32(tS, pk);
            // (the buffer of row sums is free once the output warps have taken tile i - 2)
            if (i >= 2) wait_par(pp, BAR_O_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
            sL[b * 128 + row] = (s0.x + s0.y) + (s1.x + s1.y);
            tmem_st_wait();
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_P_FULL + b);
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------------ output warps
        const int row = tid - NROW;                        // operand row = tensor-memory lane
        const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
        const int r = row / L.wp, xp = row - r * L.wp;     // tile row, padded column
        for (int i = 0; i < T_; ++i, it.next()) {
            const int b = i & 1;
            const int rows = min(R, H - it.tb * R);
            const bool live = r < rows && xp >= 1 && xp <= W;
            const uint32_t tO = pp.tmem + TM_O + 64 * b + lane_base, tD = pp.tmem + TM_D + 64 * b + lane_base;
            uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(p.out) + ((size_t)it.slab * N + (size_t)(it.tb * R + r) * W + (xp - 1)) * 64);
            wait_par(pp, BAR_O_FULL + b, i >> 1, kTimeoutTile);
            if (has_dwc) wait_par(pp, BAR_D_FULL + b, i >> 1, kTimeoutTile);
            tc_fence_after_sync();
            // The buffers are handed back BEFORE the global stores (an mbarrier arrival is a release: it would
            // otherwise wait for the stores): both halves are combined in registers first.
            const float inv = 1.f / sL[b * 128 + row];
            const float2 inv2 = make_float2(inv, inv);
            uint32_t w[32];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t acc[32], da[32], db[32];
                tmem_ld32(tO + 32 * q, acc);
                if (has_dwc) { tmem_ld32(tD + 32 * q, da); tmem_ld32(tD + 128 + 32 * q, db); }
                tmem_ld_wait();
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    float2 d2 = make_float2(0.f, 0.f);
                    if (has_dwc) d2 = fadd2(make_float2(__uint_as_float(da[2 * k]), __uint_as_float(da[2 * k + 1])),
                                            make_float2(__uint_as_float(db[2 * k]), __uint_as_float(db[2 * k + 1])));
                    const float2 v = ffma2(make_float2(__uint_as_float(acc[2 * k]), __uint_as_float(acc[2 * k + 1])), inv2, d2);
                    w[16 * q + k] = Pair<T>::cvt(v.x, v.y);
                }
            }
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_O_EMPTY + b);
            if (live) {
#pragma unroll
                for (int k = 0; k < 8; ++k) dst[k] = make_uint4(w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc<512>(pp.tmem);
}

// ------------------------------------------------------------------------------------- host
StreamPlan plan_stream(int dtype, int slabs, int H, int W, int d, int n_agents, bool pooled, int sm_count) {
    StreamPlan pl;
    memset(&pl, 0, sizeof(pl));
    if (dtype != kBF16 && dtype != kF16) return pl;
    const long long N = (long long)H * W;
    if (d != 64 || n_agents < 1 || n_agents > 64 || W < 8 || W > 64 || N < 1024 || N % 8 != 0 || N > (1 << 24)) return pl;
    if (pooled) {
        int pw = 1;
        while (pw * pw < n_agents) ++pw;
        if (pw * pw != n_agents || H % pw != 0 || W % pw != 0) return pl;
    }
    if (!encode_tiled_fn()) return pl;
    // aggregation: about one block per SM, ranges of whole 128-token tiles
    const int tiles = (int)((N + 127) / 128);
    int splits = sm_count / slabs;
    if (splits < 1) splits = 1;
    if (splits > 8) splits = 8;
    if (splits > tiles / 4) splits = tiles / 4 > 0 ? tiles / 4 : 1;
    pl.tiles_per_split = (tiles + splits - 1) / splits;
    pl.splits = (tiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
    // broadcast: tiles of whole grid rows
    int R = 128 / (W + 2);                                   // operand rows are padded token positions
    if (R > 16) R = 16;
    if (R > H) R = H;
    if (R < 1) return pl;
    pl.rows_b = R;
    pl.tiles_b = (H + R - 1) / R;
    pl.halo_stages = 2;
    pl.smem_b = bc_layout(R, W).total + 1024;
    if (pl.smem_b > 232448 - 1024) return pl;
    const long long total = (long long)slabs * pl.tiles_b;
    pl.grid_b = (int)(total < sm_count ? total : sm_count);
    pl.ok = true;
    return pl;
}

size_t stream_extra_bytes(int slabs, int heads, int N, int n_agents) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t av = up((size_t)slabs * n_agents * 64 * 2);
    return 2 * av + 2 * up((size_t)heads * N * 64 * 2) + up((size_t)heads * 9 * 2048);
}

bool stream_make_maps(StreamArgs* a) {
    const uint64_t N = (uint64_t)a->H * a->W, S = a->slabs;
    if (!make_map_rows3d_u16(&a->tm_k, a->k, S, N, 128, true)) return false;
    if (!make_map_rows3d_u16(&a->tm_v, a->v, S, N, 128, true)) return false;
    if (!make_map_grid4d_u16(&a->tm_q, a->q, S, (uint64_t)a->H, (uint64_t)a->W, (uint32_t)a->plan.rows_b, (uint32_t)(a->W + 2), true)) return false;
    if (!make_map_grid4d_u16(&a->tm_b2, a->b2p, a->b2 ? (uint64_t)a->heads : 1u, (uint64_t)a->H, (uint64_t)a->W, (uint32_t)a->plan.rows_b, (uint32_t)(a->W + 2), true)) return false;
    if (a->dwc_w && !make_map_grid4d_u16(&a->tm_h, a->v, S, (uint64_t)a->H, (uint64_t)a->W, (uint32_t)(a->plan.rows_b + 2), (uint32_t)(a->W + 2), true)) return false;
    if (a->b1 && !make_map_rows3d_u16(&a->tm_b1, a->b1c, (uint64_t)a->heads, N, 128, true)) return false;
    if (!make_map_2d_u16(&a->tm_a2, a->a2s, S * a->n, 64, (uint32_t)a->n, 64)) return false;
    if (!make_map_2d_u16(&a->tm_va, a->va_ws, S * a->n, 64, (uint32_t)a->n, 64)) return false;
    return true;
}

cudaError_t launch_stream_broadcast(int dtype, const StreamArgs& a, cudaStream_t st) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)a.plan.grid_b);
    cfg.blockDim = dim3(NT);
    cfg.dynamicSmemBytes = (size_t)a.plan.smem_b;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (dtype == kBF16) {
        auto kern = stream_broadcast_kernel<__nv_bfloat16>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, a.plan.smem_b);
        if (e != cudaSuccess) return e;
        return cudaLaunchKernelEx(&cfg, kern, a);
    }
    if (dtype == kF16) {
        auto kern = stream_broadcast_kernel<__half>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, a.plan.smem_b);
        if (e != cudaSuccess) return e;
        return cudaLaunchKernelEx(&cfg, kern, a);
    }
    return cudaErrorInvalidValue;
}

}  // namespace aa
