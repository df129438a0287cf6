// Agent broadcast with the depthwise term, O = softmax(scale2 * Q A^T + B2) V_A + DWC(V) (Eq. 3, Eq. 5, Eq. 6)
// for small agent counts (n <= 64, d = 64, 16-bit elements) as a streaming kernel on the 5th-generation
// tensor cores.
//
// Persistent blocks, one per SM; block c walks a contiguous run of the (slab, row tile) sequence, a tile being
// R whole grid rows (R * W <= 128 tokens).  Nothing is carried from tile to tile, so the run is one
// continuous pipeline across slab boundaries (the agents of the next slab arrive in a second buffer).
//   warp 16 "producer":  one lane issues every TMA copy: the Q tile and the matching rows of the padded B2
//       (two stages), the V rows of the tile with one grid row above and below (two stages of their own; rows
//       outside the grid are zero-filled by the copy), and the slab's agents A (times scale2) and V_A.
//   warp 17 "MMA issuer": one lane.  S = Q A^T + B2 I: the bias enters through four 16-column identity
//       slices, and its pad columns (a large negative value) remove the agents past n; one tile ahead.
//       Then O = P [V_A | 1] with the probabilities read from tensor memory and a ones block for the row sums.
//   warps 0-3 "softmax warps": thread = token.  Logits from tensor memory -> maximum, probabilities (two per
//       packed exponential, rounded to the operand type) -> back to tensor memory.
//   warps 4-7 "output warps": thread = token.  Row of O from tensor memory times 1 / row sum, plus the
//       depthwise term from the patch, rounded once, stored.
//   warps 8-15 "stencil warps": thread = (tile row, 4 channels, x-segment): a 3x3 window slides along x over
//       the V rows in shared memory (packed fp32 FMAs, taps in registers) and leaves the depthwise term in an
//       fp32 patch (two buffers, so that the stencil runs ahead of the attention part).
// Every wait is bounded.  No TMA multicast, no clusters.
#include "stream_common.cuh"

namespace aa {

namespace {
constexpr int NROW = 128;              // softmax threads, and output threads
constexpr int NDWC = 256;              // stencil threads
constexpr int NT = 2 * NROW + NDWC + 64;   // + producer warp + MMA issuer warp
constexpr int kPatchPitch = 68;        // floats per patch row: 16-byte row reads by consecutive lanes spread over all banks
constexpr int kTimeoutTile = 3, kTimeoutLoads = 4, kTimeoutRole = 6;

// shared memory (bytes from a 1024-aligned base)
constexpr int OFF_BAR = 0;
constexpr int OFF_I16 = 1024;          // [16][128 B]: identity slice, K-major B operand of the bias steps
constexpr int OFF_ONES = 3072;         // [16][128 B] of ones: B operand of the row sums
constexpr int OFF_A2 = 5120;           // 2 x agents [64][128 B]
constexpr int OFF_VA = OFF_A2 + 2 * 8192;   // 2 x agent features [64][128 B]
constexpr int OFF_QB = OFF_VA + 2 * 8192;   // 2 stages x (Q tile | B2 tile), then the V-row stages, then the patches
static_assert(OFF_QB % 1024 == 0, "swizzled tiles need 1024-byte alignment");

struct BcLayout {
    int tq, qsz, hsz, psz, off_h, off_patch, total;
};
__host__ __device__ inline BcLayout bc_layout(int R, int W) {
    BcLayout l;
    l.tq = R * W;
    l.qsz = (l.tq * 128 + 1023) / 1024 * 1024;
    l.hsz = ((R + 2) * W * 128 + 1023) / 1024 * 1024;
    l.psz = (l.tq * kPatchPitch * 4 + 1023) / 1024 * 1024;
    l.off_h = OFF_QB + 4 * l.qsz;
    l.off_patch = l.off_h + 2 * l.hsz;
    l.total = l.off_patch + 2 * l.psz;
    if (l.total < l.off_h + 2048) l.total = l.off_h + 2048;      // the last Q-sized operand read runs up to 2 KB past its tile
    return l;
}

// mbarriers                                  count           waiter
constexpr int BAR_OPS = 0;        // [2]       tx              MMA issuer      agents and agent features of a slab
constexpr int BAR_QB_FULL = 2;    // [2]       tx              MMA issuer
constexpr int BAR_QB_EMPTY = 4;   // [2]       commit          producer
constexpr int BAR_H_FULL = 6;     // [2]       tx              stencil warps
constexpr int BAR_H_EMPTY = 8;    // [2]       stencil threads producer
constexpr int BAR_S_FULL = 10;    // [2]       commit          softmax warps
constexpr int BAR_P_FULL = 12;    // [2]       softmax threads MMA issuer
constexpr int BAR_O_FULL = 14;    // [2]       commit          output warps
constexpr int BAR_O_EMPTY = 16;   // [2]       output threads  MMA issuer
constexpr int BAR_PATCH_FULL = 18;  // [2]     stencil threads output warps
constexpr int BAR_PATCH_EMPTY = 20; // [2]     output threads  stencil warps
constexpr int kBars = 22;

// tensor memory columns: logits 2 x 64 (the probabilities overwrite the first 32), output 2 x (64 + 16 row sums)
constexpr uint32_t TM_S = 0, TM_O = 128, kOStride = 96;

__device__ __forceinline__ int swz16(int row, int col) {
    return row * 128 + ((((col >> 3) ^ row) & 7) << 4) + (col & 7) * 2;
}
// packed pairs of fp32 kept in 64-bit registers
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
template <typename T> __device__ __forceinline__ f32x2 widen2(uint32_t w) {      // one packed 16-bit pair -> two fp32
    const float2 f = unpack2<T>(w);
    return pk2(f.x, f.y);
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, f32x2 a, f32x2 b) {
    asm volatile("st.shared.v2.b64 [%0], {%1, %2};" ::"r"(addr), "l"(a), "l"(b) : "memory");
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
        for (int i = 0; i < kBars; ++i) {
            uint32_t cnt = 1u;
            if ((i >= BAR_H_EMPTY && i < BAR_S_FULL) || (i >= BAR_PATCH_FULL && i < BAR_PATCH_EMPTY)) cnt = NDWC;
            if ((i >= BAR_P_FULL && i < BAR_O_FULL) || (i >= BAR_O_EMPTY && i < BAR_PATCH_FULL) || i >= BAR_PATCH_EMPTY) cnt = NROW;
            mbar_init(pp.bars + 8 * i, cnt);
        }
        mbar_fence_init();
    }
    // constant operands; rows n..63 of the agent tiles never receive data (their copies bring n rows): zero
    for (int e = tid; e < 16 * 64; e += NT) {
        const int r = e >> 6, c = e & 63;
        *reinterpret_cast<uint16_t*>(smem + OFF_I16 + swz16(r, c)) = (r == c) ? (uint16_t)Pair<T>::kOne : (uint16_t)0;
        *reinterpret_cast<uint16_t*>(smem + OFF_ONES + swz16(r, c)) = (uint16_t)Pair<T>::kOne;
    }
    for (int e = tid; e < 4 * (64 - n) * 8; e += NT) {
        const int buf = e / ((64 - n) * 8), rest = e - buf * ((64 - n) * 8);
        *(reinterpret_cast<uint4*>(smem + OFF_A2 + buf * 8192 + (n + (rest >> 3)) * 128) + (rest & 7)) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async();
    if (warp == 0) tmem_alloc<512>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem = s_tmem;
    pdl_wait();              // V_A comes from the aggregation kernel (and, before it, A and the padded B2)

    const uint32_t sQB = smem_u32(smem + OFF_QB), sH = smem_u32(smem + L.off_h), sPatch = smem_u32(smem + L.off_patch);
    const uint32_t sA2 = smem_u32(smem + OFF_A2), sVA = smem_u32(smem + OFF_VA);

    if (warp == 16) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            int cur = -1, ord = -1;
            const uint32_t qb_tx = 2u * (uint32_t)L.tq * 128u, h_tx = (uint32_t)(R + 2) * W * 128u;
            for (int i = 0; i < T_; ++i, it.next()) {
                if (it.slab != cur) {
                    // (a buffer is reused two slabs later: every product that read it is long done, since the
                    // stage waits below already cover the tiles of the slab in between)
                    cur = it.slab; ++ord;
                    const uint32_t bar = pipe_bar(pp, BAR_OPS + (ord & 1));
                    mbar_arrive_expect_tx(bar, 2u * (uint32_t)n * 128u);
                    tma_load_2d(sA2 + (ord & 1) * 8192, &p.tm_a2, 0, it.slab * n, bar);
                    tma_load_2d(sVA + (ord & 1) * 8192, &p.tm_va, 0, it.slab * n, bar);
                }
                const int s2 = i & 1;
                if (i >= 2) wait_par(pp, BAR_QB_EMPTY + s2, (i >> 1) - 1, kTimeoutRole);
                {
                    const uint32_t bar = pipe_bar(pp, BAR_QB_FULL + s2), dst = sQB + s2 * 2 * L.qsz;
                    mbar_arrive_expect_tx(bar, qb_tx);
                    tma_load_3d(dst, &p.tm_q, 0, it.tb * L.tq, it.slab, bar);
                    tma_load_3d(dst + L.qsz, &p.tm_b2, 0, it.tb * L.tq, p.b2 ? it.slab % p.heads : 0, bar);
                }
                if (has_dwc) {
                    if (i >= 2) wait_par(pp, BAR_H_EMPTY + s2, (i >> 1) - 1, kTimeoutRole);
                    const uint32_t bar = pipe_bar(pp, BAR_H_FULL + s2);
                    mbar_arrive_expect_tx(bar, h_tx);
                    tma_load_3d(sH + s2 * L.hsz, &p.tm_h, 0, (it.tb * R - 1) * W, it.slab, bar);
                }
            }
        }
        __syncwarp();
    } else if (warp == 17) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idS = umma_idesc(fmt, 128, 64, 0), idI = umma_idesc(fmt, 128, 16, 0);
            const uint32_t idPV = umma_idesc(fmt, 128, 64, 1), idL = umma_idesc(fmt, 128, 16, 1);
            const uint64_t dI = umma_desc_sw128(smem_u32(smem + OFF_I16)), dOnes = umma_desc_sw128(smem_u32(smem + OFF_ONES));
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
                    wait_par(pp, BAR_OPS + (ord_s & 1), ord_s >> 1, kTimeoutLoads);
                }
                is.next();
                wait_par(pp, BAR_QB_FULL + b, i >> 1, kTimeoutTile);
                tc_fence_after_sync();
                const uint64_t dQ = b ? dQ1 : dQ0, dB = b ? dB1 : dB0;
                const uint64_t da = dA2 + 512 * (ord_s & 1);
                const uint32_t dd = tS + 64 * b;
                umma_f16(dd, dQ, da, idS, 0u);
#pragma unroll
                for (int k = 1; k < 4; ++k) umma_f16(dd, dQ + 2 * k, da + 2 * k, idS, 1u);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_f16(dd + 16 * k, dB + 2 * k, dI, idI, 1u);
                umma_commit(pipe_bar(pp, BAR_QB_EMPTY + b));
                umma_commit(pipe_bar(pp, BAR_S_FULL + b));
            };
            if (T_ > 0) issue_S(0, 0);
            for (int i0 = 0; i0 < T_; i0 += 2) {
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int i = i0 + b;
                    if (i < T_) {
                        if (i + 1 < T_) issue_S(i + 1, b ^ 1);
                        if (it.slab != cur_o) { cur_o = it.slab; ++ord_o; }
                        it.next();
                        wait_par(pp, BAR_P_FULL + b, i >> 1, kTimeoutRole);
                        if (i >= 2) wait_par(pp, BAR_O_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
                        tc_fence_after_sync();
                        const uint32_t tP = tS + 64 * b, dd = tO + kOStride * b;
                        const uint64_t dv = dVA + 512 * (ord_o & 1);
                        umma_ts(dd, tP, dv, idPV, 0u);
#pragma unroll
                        for (int k = 1; k < 4; ++k) umma_ts(dd, tP + 8 * k, dv + 128 * k, idPV, 1u);
                        umma_ts(dd + 64, tP, dOnes, idL, 0u);
#pragma unroll
                        for (int k = 1; k < 4; ++k) umma_ts(dd + 64, tP + 8 * k, dOnes, idL, 1u);
                        umma_commit(pipe_bar(pp, BAR_O_FULL + b));
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp < 4) {
        // ------------------------------------------------------------------ softmax warps
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
            uint32_t pk[32];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float2 x0 = ffma2(make_float2(__uint_as_float(sa[2 * j]), __uint_as_float(sa[2 * j + 1])), l2e, nb2);
                const float2 x1 = ffma2(make_float2(__uint_as_float(sb[2 * j]), __uint_as_float(sb[2 * j + 1])), l2e, nb2);
                pk[j] = Pair<T>::ex2(Pair<T>::cvt(x0.x, x0.y));
                pk[16 + j] = Pair<T>::ex2(Pair<T>::cvt(x1.x, x1.y));
            }
            tmem_st32(tS, pk);
            tmem_st_wait();
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_P_FULL + b);
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------------ output warps
        const int row = tid - NROW;                        // token of the tile = tensor-memory lane
        const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
        for (int i = 0; i < T_; ++i, it.next()) {
            const int b = i & 1;
            const int rows = min(R, H - it.tb * R);
            const bool live = row < rows * W;
            const uint32_t tO = pp.tmem + TM_O + kOStride * b + lane_base;
            const uint32_t prow = sPatch + b * L.psz + (uint32_t)min(row, L.tq - 1) * (kPatchPitch * 4);
            uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(p.out) + ((size_t)it.slab * N + (size_t)it.tb * L.tq + row) * 64);
            wait_par(pp, BAR_O_FULL + b, i >> 1, kTimeoutTile);
            tc_fence_after_sync();
            const uint32_t rl = tmem_ld1(tO + 64);
            tmem_ld_wait();
            const float inv = 1.f / __uint_as_float(rl);
            const f32x2 inv2 = pk2(inv, inv);
            if (has_dwc) wait_par(pp, BAR_PATCH_FULL + b, i >> 1, kTimeoutRole);
            // four quarters of 16 channels: row of O times 1 / row sum, plus the depthwise term, rounded once
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t acc[16];
                tmem_ld16(tO + 16 * q, acc);
                tmem_ld_wait();
                uint32_t w[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    f32x2 d0 = 0ull, d1 = 0ull;
                    if (has_dwc) asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(d0), "=l"(d1) : "r"(prow + 64 * q + 16 * k));
                    const f32x2 v0 = fma2(pk2(__uint_as_float(acc[4 * k]), __uint_as_float(acc[4 * k + 1])), inv2, d0);
                    const f32x2 v1 = fma2(pk2(__uint_as_float(acc[4 * k + 2]), __uint_as_float(acc[4 * k + 3])), inv2, d1);
                    float a0, a1, a2, a3;
                    asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(v0));
                    asm("mov.b64 {%0, %1}, %2;" : "=f"(a2), "=f"(a3) : "l"(v1));
                    w[2 * k] = Pair<T>::cvt(a0, a1);
                    w[2 * k + 1] = Pair<T>::cvt(a2, a3);
                }
                if (live) {
                    dst[2 * q] = make_uint4(w[0], w[1], w[2], w[3]);
                    dst[2 * q + 1] = make_uint4(w[4], w[5], w[6], w[7]);
                }
            }
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_O_EMPTY + b);
            if (has_dwc) pipe_arrive(pp, BAR_PATCH_EMPTY + b);
        }
    } else if (warp < 16 && has_dwc) {
        // ------------------------------------------------------------------ stencil warps
        const int dt = tid - 2 * NROW;                     // 0 .. 255
        const int npairs = R * 16;
        int nseg = NDWC / npairs;
        if (nseg > W) nseg = W;
        const int seg_len = (W + nseg - 1) / nseg;        // <= 8 for every eligible shape
        const int pair = dt % npairs, seg = dt / npairs;
        const int r = pair >> 4, cq = pair & 15;
        const int x0 = seg * seg_len, x1 = min(W, x0 + seg_len), len = x1 - x0;
        const bool active = seg < nseg && len > 0;
        const uint32_t rp = (uint32_t)W * 128u;           // bytes between grid rows of the V-row buffer
        const uint32_t hoff = (uint32_t)(r * W + x0) * 128u + cq * 8;        // this thread's first window column (centre), row y-1
        const uint32_t poff = (uint32_t)(r * W + x0) * (kPatchPitch * 4) + cq * 16;
        f32x2 w[9][2];
        int cur_head = -1;
        for (int i = 0; i < T_; ++i, it.next()) {
            const int b = i & 1;
            const int head = it.slab % p.heads;
            const int rows = min(R, H - it.tb * R);
            if (head != cur_head) {                        // filter taps of this thread's four channels
                cur_head = head;
                const T* gw = static_cast<const T*>(p.dwc_w) + ((size_t)head * 64 + cq * 4) * 9;
#pragma unroll
                for (int tap = 0; tap < 9; ++tap) {
                    w[tap][0] = pk2(Elem<T>::to_f32(gw[tap]), Elem<T>::to_f32(gw[9 + tap]));
                    w[tap][1] = pk2(Elem<T>::to_f32(gw[18 + tap]), Elem<T>::to_f32(gw[27 + tap]));
                }
            }
            wait_par(pp, BAR_H_FULL + b, i >> 1, kTimeoutLoads);
            if (i >= 2) wait_par(pp, BAR_PATCH_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
            if (active && r < rows) {
                // buffer rows r, r+1, r+2 are grid rows y-1, y, y+1 of this thread's tile row; columns outside the grid are zero
                const uint32_t hb = sH + b * L.hsz + hoff, pb = sPatch + b * L.psz + poff;
                f32x2 col[3][3][2];
                auto load_col = [&](int j, f32x2 (&c)[3][2]) {     // window column at x0 + j
                    const int hx = x0 + j;
                    if (hx < 0 || hx >= W) {
#pragma unroll
                        for (int u = 0; u < 3; ++u) c[u][0] = c[u][1] = 0ull;
                    } else {
#pragma unroll
                        for (int u = 0; u < 3; ++u) {
                            const uint2 raw = lds64(hb + u * rp + j * 128);
                            c[u][0] = widen2<T>(raw.x);
                            c[u][1] = widen2<T>(raw.y);
                        }
                    }
                };
                load_col(-1, col[0]);
                load_col(0, col[1]);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (j < len) {
                        f32x2 (&cl)[3][2] = col[j % 3];
                        f32x2 (&cc)[3][2] = col[(j + 1) % 3];
                        f32x2 (&cr)[3][2] = col[(j + 2) % 3];
                        load_col(j + 1, cr);
                        f32x2 o0 = mul2(w[0][0], cl[0][0]), o1 = mul2(w[0][1], cl[0][1]);
                        o0 = fma2(w[1][0], cc[0][0], o0); o1 = fma2(w[1][1], cc[0][1], o1);
                        o0 = fma2(w[2][0], cr[0][0], o0); o1 = fma2(w[2][1], cr[0][1], o1);
#pragma unroll
                        for (int u = 1; u < 3; ++u) {
                            o0 = fma2(w[u * 3 + 0][0], cl[u][0], o0); o1 = fma2(w[u * 3 + 0][1], cl[u][1], o1);
                            o0 = fma2(w[u * 3 + 1][0], cc[u][0], o0); o1 = fma2(w[u * 3 + 1][1], cc[u][1], o1);
                            o0 = fma2(w[u * 3 + 2][0], cr[u][0], o0); o1 = fma2(w[u * 3 + 2][1], cr[u][1], o1);
                        }
                        sts128(pb + j * (kPatchPitch * 4), o0, o1);
                    }
                }
            }
            pipe_arrive(pp, BAR_H_EMPTY + b);
            pipe_arrive(pp, BAR_PATCH_FULL + b);
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
    int R = 128 / W;
    if (R > 16) R = 16;
    if (R > H) R = H;
    pl.rows_b = R;
    pl.tiles_b = (H + R - 1) / R;
    if ((R + 2) * W > 256) return pl;
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
    return 2 * av + 2 * up((size_t)heads * N * 64 * 2);
}

bool stream_make_maps(StreamArgs* a) {
    const uint64_t N = (uint64_t)a->H * a->W, S = a->slabs;
    const BcLayout L = bc_layout(a->plan.rows_b, a->W);
    if (!make_map_rows3d_u16(&a->tm_k, a->k, S, N, 128, true)) return false;
    if (!make_map_rows3d_u16(&a->tm_v, a->v, S, N, 128, true)) return false;
    if (!make_map_rows3d_u16(&a->tm_q, a->q, S, N, (uint32_t)L.tq, true)) return false;
    if (!make_map_rows3d_u16(&a->tm_b2, a->b2p, a->b2 ? (uint64_t)a->heads : 1u, N, (uint32_t)L.tq, true)) return false;
    if (a->dwc_w && !make_map_rows3d_u16(&a->tm_h, a->v, S, N, (uint32_t)((a->plan.rows_b + 2) * a->W), false)) return false;
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

cudaError_t launch_stream(int dtype, const StreamArgs& a, cudaStream_t st) {
    cudaError_t e = launch_stream_prep(dtype, a, st);
    if (e != cudaSuccess) return e;
    e = launch_stream_aggregate(dtype, a, st);
    if (e != cudaSuccess) return e;
    return launch_stream_broadcast(dtype, a, st);
}

}  // namespace aa
