// Agent broadcast with the depthwise term, O = softmax(scale2 * Q A^T + B2) V_A + DWC(V) (Eq. 3, Eq. 5, Eq. 6)
// for small agent counts (n <= 64, d = 64, 16-bit elements) as a streaming kernel on the 5th-generation
// tensor cores.
//
// Persistent blocks, one per SM; block c walks a contiguous run of the (slab, row tile) sequence, a tile being
// R whole grid rows (R * W <= 128 tokens).  Nothing is carried from tile to tile, so the run is one
// continuous pipeline across slab boundaries (the agents of the next slab arrive in a second buffer).
// 27 warps, each role with a small register footprint so that all of them are resident together:
//   warp 24 "tile producer": one lane issues the TMA copies of the Q tile and of the matching rows of the padded
//       B2 (two stages), and of the slab's agents A (times scale2) and V_A.
//   warp 25 "row producer": one lane keeps a ring of four chunks of R grid rows of V (each row with a zero column
//       at either end; rows outside the grid zero-filled by the copy) filled two tiles ahead.  A tile's 3x3
//       windows read the chunk before it, its own and the one after it, so every V row enters shared memory once.
//   warp 26 "MMA issuer": one lane.  S = Q A^T + B2 I: the bias enters through four 16-column identity
//       slices, and its pad columns (a large negative value) remove the agents past n; one tile ahead.
//       Then O = P V_A with the probabilities read from tensor memory.
//   warps 0-3 "softmax warps": thread = token.  Two passes over the logits in tensor memory, 16 columns at a
//       time: maximum; then fp32 exponentials, their sum (handed to the output warps through shared memory)
//       and the probabilities, rounded to the operand type, back to tensor memory over the logits.
//   warps 4-7 "output warps": thread = token.  Row of O from tensor memory times 1 / row sum, plus the
//       depthwise term from the patch, rounded once, stored.
//   warps 8-23 "stencil warps": thread = (tile row, 2 channels, x-segment): a 3x3 window slides along x over
//       the V rows in shared memory (packed fp32 FMAs, taps in registers) and leaves the depthwise term in an
//       fp32 patch (two buffers, so that the stencil runs ahead of the attention part).
// Every wait is bounded.  No TMA multicast, no clusters.
#include "stream_common.cuh"

namespace aa {

namespace {
constexpr int NROW = 128;              // softmax threads, and output threads
constexpr int NDWC = 512;              // stencil threads
constexpr int NT = 2 * NROW + NDWC + 96;   // + two producer warps + MMA issuer warp
constexpr int kPatchPitch = 68;        // floats per patch row: 16-byte row reads by consecutive lanes spread over all banks
constexpr int kChunks = 4;             // ring of V-row chunks
constexpr int kTimeoutTile = 3, kTimeoutLoads = 4, kTimeoutRole = 6;

// shared memory (bytes from a 1024-aligned base)
constexpr int OFF_BAR = 0;
constexpr int OFF_L = 256;             // [2][128] row sums of the probabilities (fp32)
constexpr int OFF_I16 = 2048;          // [16][128 B]: identity slice, K-major B operand of the bias steps
constexpr int OFF_A2 = 4096;           // 2 x agents [64][128 B]
constexpr int OFF_VA = OFF_A2 + 2 * 8192;   // 2 x agent features [64][128 B]
constexpr int OFF_QB = OFF_VA + 2 * 8192;   // 2 stages x (Q tile | B2 tile), then the V-row ring, then the patches
static_assert(OFF_QB % 1024 == 0, "swizzled tiles need 1024-byte alignment");

struct BcLayout {
    int tq, qsz, rowb, chunkb, psz, off_h, off_patch, total;
};
__host__ __device__ inline BcLayout bc_layout(int R, int W) {
    BcLayout l;
    l.tq = R * W;
    l.qsz = (l.tq * 128 + 1023) / 1024 * 1024;
    l.rowb = (W + 2) * 128;                                 // one grid row of V with a zero column at either end
    l.chunkb = R * l.rowb;
    l.psz = (l.tq * kPatchPitch * 4 + 1023) / 1024 * 1024;
    l.off_h = OFF_QB + 4 * l.qsz;
    l.off_patch = l.off_h + (kChunks * l.chunkb + 1023) / 1024 * 1024;
    l.total = l.off_patch + 2 * l.psz;
    if (l.total < l.off_h + 2048) l.total = l.off_h + 2048;      // the last Q-sized operand read runs up to 2 KB past its tile
    return l;
}

// mbarriers                                  count           waiter
constexpr int BAR_OPS = 0;        // [2]       tx              MMA issuer      agents and agent features of a slab
constexpr int BAR_QB_FULL = 2;    // [2]       tx              MMA issuer
constexpr int BAR_QB_EMPTY = 4;   // [2]       commit          tile producer
constexpr int BAR_H_FULL = 6;     // [4]       tx              stencil warps
constexpr int BAR_H_EMPTY = 10;   // [4]       stencil threads row producer
constexpr int BAR_S_FULL = 14;    // [2]       commit          softmax warps
constexpr int BAR_P_FULL = 16;    // [2]       softmax threads MMA issuer
constexpr int BAR_O_FULL = 18;    // [2]       commit          output warps
constexpr int BAR_O_EMPTY = 20;   // [2]       output threads  MMA issuer, softmax warps (the row sums' buffer)
constexpr int BAR_PATCH_FULL = 22;  // [2]     stencil threads output warps
constexpr int BAR_PATCH_EMPTY = 24; // [2]     output threads  stencil warps
constexpr int kBars = 26;

// tensor memory columns: logits 2 x 64 (the probabilities overwrite the first 32), output 2 x 64
constexpr uint32_t TM_S = 0, TM_O = 128;

__device__ __forceinline__ int swz16(int row, int col) {
    return row * 128 + ((((col >> 3) ^ row) & 7) << 4) + (col & 7) * 2;
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};\n"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
// Spinning wait of a single-lane role on the critical path (no back-off: a hand-off costs tens of cycles);
// bounded like every other wait.
__device__ __forceinline__ void wait_spin(Pipe& pp, int i, uint32_t parity, int code) {
    const uint32_t bar = pipe_bar(pp, i);
    for (unsigned tries = 0; tries < (1u << 24); ++tries) {
        if (mbar_try_wait(bar, parity & 1u)) return;
        if ((tries & 1023u) == 1023u && pipe_dead(pp)) return;
    }
    *reinterpret_cast<volatile int*>(pp.dead) = 1;
    if (pp.status) atomicCAS(pp.status, 0, code);
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
    // constant operand; rows n..63 of the agent tiles never receive data (their copies bring n rows): zero
    for (int e = tid; e < 16 * 64; e += NT) {
        const int r = e >> 6, c = e & 63;
        *reinterpret_cast<uint16_t*>(smem + OFF_I16 + swz16(r, c)) = (r == c) ? (uint16_t)Pair<T>::kOne : (uint16_t)0;
    }
    for (int e = tid; e < 4 * (64 - n) * 8; e += NT) {
        const int buf = e / ((64 - n) * 8), rest = e - buf * ((64 - n) * 8);
        *(reinterpret_cast<uint4*>(smem + OFF_A2 + buf * 8192 + (n + (rest >> 3)) * 128) + (rest & 7)) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async();
    if (warp == 0) tmem_alloc<256>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem = s_tmem;

    const uint32_t sQB = smem_u32(smem + OFF_QB), sH = smem_u32(smem + L.off_h);
    const uint32_t sA2 = smem_u32(smem + OFF_A2), sVA = smem_u32(smem + OFF_VA);
    float* sL = reinterpret_cast<float*>(smem + OFF_L);

    if (warp == 24) {
        // ------------------------------------------------------------------ tile producer
        if (lane == 0) {
            pdl_wait();      // A, V_A and the padded B2 come from the preceding kernels
            int cur = -1, ord = -1;
            const uint32_t qb_tx = 2u * (uint32_t)L.tq * 128u;
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
                if (i >= 2) wait_spin(pp, BAR_QB_EMPTY + s2, (i >> 1) - 1, kTimeoutRole);
                const uint32_t bar = pipe_bar(pp, BAR_QB_FULL + s2), dst = sQB + s2 * 2 * L.qsz;
                mbar_arrive_expect_tx(bar, qb_tx);
                tma_load_3d(dst, &p.tm_q, 0, it.tb * L.tq, it.slab, bar);
                tma_load_3d(dst + L.qsz, &p.tm_b2, 0, it.tb * L.tq, p.b2 ? it.slab % p.heads : 0, bar);
            }
        }
        __syncwarp();
    } else if (warp == 25) {
        // ------------------------------------------------------------------ row producer (V is an input of the call: no wait)
        if (lane == 0 && has_dwc) {
            int c = 0;
            auto emit = [&](int slab, int tbc) {                 // chunk = grid rows tbc * R .. tbc * R + R - 1 of the slab
                const int slot = c & (kChunks - 1);
                if (c >= kChunks) wait_spin(pp, BAR_H_EMPTY + slot, (c >> 2) - 1, kTimeoutRole);
                const uint32_t bar = pipe_bar(pp, BAR_H_FULL + slot);
                mbar_arrive_expect_tx(bar, (uint32_t)L.chunkb);
                tma_load_4d(sH + slot * L.chunkb, &p.tm_h, 0, -1, tbc * R, slab, bar);
                ++c;
            };
            if (T_ > 0) emit(it.slab, it.tb - 1);
            for (int i = 0; i < T_; ++i, it.next()) {
                emit(it.slab, it.tb);
                // past a slab's last tile comes a chunk of zero rows, which also serves as the chunk before the
                // next slab's first tile; the run's last tile needs the chunk after it too
                if (it.tb == TB - 1 || i == T_ - 1) emit(it.slab, it.tb + 1);
            }
        }
        __syncwarp();
    } else if (warp == 26) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
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
                        wait_spin(pp, BAR_P_FULL + b, i >> 1, kTimeoutRole);
                        if (i >= 2) wait_spin(pp, BAR_O_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
                        tc_fence_after_sync();
                        const uint32_t tP = tS + 64 * b, dd = tO + 64 * b;
                        const uint64_t dv = dVA + 512 * (ord_o & 1);
                        umma_ts(dd, tP, dv, idPV, 0u);
#pragma unroll
                        for (int k = 1; k < 4; ++k) umma_ts(dd, tP + 8 * k, dv + 128 * k, idPV, 1u);
                        umma_commit(pipe_bar(pp, BAR_O_FULL + b));
                    }
                }
            }
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
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t s[16];
                tmem_ld16(tS + 16 * c, s);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; j += 2) mx = max3(mx, __uint_as_float(s[j]), __uint_as_float(s[j + 1]));
            }
            const float nb = -mx * kLog2e;
            const float2 nb2 = make_float2(nb, nb);
            float2 sum = make_float2(0.f, 0.f);
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t s[16], pk[8];
                tmem_ld16(tS + 16 * c, s);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float2 x = ffma2(make_float2(__uint_as_float(s[2 * j]), __uint_as_float(s[2 * j + 1])), l2e, nb2);
                    const float2 e = make_float2(fast_exp2(x.x), fast_exp2(x.y));
                    sum = fadd2(sum, e);
                    pk[j] = Pair<T>::cvt(e.x, e.y);
                }
                tmem_st8(tS + 8 * c, pk);      // over logit columns that both passes have already read
            }
            // (the buffer of row sums is free once the output warps have taken tile i - 2)
            if (i >= 2) wait_par(pp, BAR_O_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
            sL[b * 128 + row] = sum.x + sum.y;
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
            const uint32_t tO = pp.tmem + TM_O + 64 * b + lane_base;
            const float* prow = reinterpret_cast<const float*>(smem + L.off_patch + b * L.psz) + (size_t)min(row, L.tq - 1) * kPatchPitch;
            uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(p.out) + ((size_t)it.slab * N + (size_t)it.tb * L.tq + row) * 64);
            wait_par(pp, BAR_O_FULL + b, i >> 1, kTimeoutTile);
            tc_fence_after_sync();
            const float inv = 1.f / sL[b * 128 + row];
            const float2 inv2 = make_float2(inv, inv);
            if (has_dwc) wait_par(pp, BAR_PATCH_FULL + b, i >> 1, kTimeoutRole);
            // four quarters of 16 channels: row of O times 1 / row sum, plus the depthwise term, rounded once
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                uint32_t acc[16];
                tmem_ld16(tO + 16 * q, acc);
                float4 dw[4];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    dw[k] = has_dwc ? *reinterpret_cast<const float4*>(prow + 16 * q + 4 * k) : make_float4(0.f, 0.f, 0.f, 0.f);
                tmem_ld_wait();
                uint32_t w[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float2 v0 = ffma2(make_float2(__uint_as_float(acc[4 * k]), __uint_as_float(acc[4 * k + 1])), inv2, make_float2(dw[k].x, dw[k].y));
                    const float2 v1 = ffma2(make_float2(__uint_as_float(acc[4 * k + 2]), __uint_as_float(acc[4 * k + 3])), inv2, make_float2(dw[k].z, dw[k].w));
                    w[2 * k] = Pair<T>::cvt(v0.x, v0.y);
                    w[2 * k + 1] = Pair<T>::cvt(v1.x, v1.y);
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
    } else if (warp < 24 && has_dwc) {
        // ------------------------------------------------------------------ stencil warps
        const int dt = tid - 2 * NROW;                     // 0 .. 511
        const int npairs = R * 32;
        int nseg = NDWC / npairs;
        if (nseg > W) nseg = W;
        const int seg_len = (W + nseg - 1) / nseg;        // <= 8 for every eligible shape
        const int pair = dt % npairs, seg = dt / npairs;
        const int r = pair >> 5, cq = pair & 31;          // tile row, channel pair
        const int x0 = seg * seg_len, x1 = min(W, x0 + seg_len), len = x1 - x0;
        const bool active = seg < nseg && len > 0;
        // the window's three grid rows (tile rows r - 1, r, r + 1): chunk relative to the tile's own, and row inside it
        int rel[3], rin[3];
#pragma unroll
        for (int u = 0; u < 3; ++u) {
            const int q = r - 1 + u;
            rel[u] = q < 0 ? -1 : (q >= R ? 1 : 0);
            rin[u] = q < 0 ? R - 1 : (q >= R ? 0 : q);
        }
        const uint32_t col0 = (uint32_t)x0 * 128u + cq * 4;          // buffer column x0 is grid column x0 - 1
        float* pb0 = reinterpret_cast<float*>(smem + L.off_patch) + (size_t)(r * W + x0) * kPatchPitch + cq * 2;
        float2 w[9];
        int cur_head = -1;
        int ci = 1, waited = 0, released = 0;              // this tile's chunk; chunks known to be loaded; chunks given back
        for (int i = 0; i < T_; ++i) {
            const int b = i & 1;
            const int head = it.slab % p.heads;
            const int rows = min(R, H - it.tb * R);
            const int ci_next = ci + (it.tb == TB - 1 ? 2 : 1);
            it.next();
            if (head != cur_head) {                        // filter taps of this thread's two channels
                cur_head = head;
                const T* gw = static_cast<const T*>(p.dwc_w) + ((size_t)head * 64 + cq * 2) * 9;
#pragma unroll
                for (int tap = 0; tap < 9; ++tap) w[tap] = make_float2(Elem<T>::to_f32(gw[tap]), Elem<T>::to_f32(gw[9 + tap]));
            }
            while (waited <= ci + 1) {
                wait_par(pp, BAR_H_FULL + (waited & (kChunks - 1)), waited >> 2, kTimeoutLoads);
                ++waited;
            }
            if (i >= 2) wait_par(pp, BAR_PATCH_EMPTY + b, (i >> 1) - 1, kTimeoutRole);
            if (active && r < rows) {
                const unsigned char* rowp[3];
#pragma unroll
                for (int u = 0; u < 3; ++u)
                    rowp[u] = smem + L.off_h + ((ci + rel[u]) & (kChunks - 1)) * L.chunkb + rin[u] * L.rowb + col0;
                float* pb = pb0 + b * (L.psz >> 2);
                float2 col[3][3];
                auto load_col = [&](int j, float2 (&c)[3]) {       // buffer column x0 + j
#pragma unroll
                    for (int u = 0; u < 3; ++u) c[u] = unpack2<T>(*reinterpret_cast<const uint32_t*>(rowp[u] + j * 128));
                };
                load_col(0, col[0]);
                load_col(1, col[1]);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (j < len) {
                        float2 (&cl)[3] = col[j % 3];
                        float2 (&cc)[3] = col[(j + 1) % 3];
                        float2 (&cr)[3] = col[(j + 2) % 3];
                        load_col(j + 2, cr);
                        float2 o = fmul2(w[0], cl[0]);
                        o = ffma2(w[1], cc[0], o); o = ffma2(w[2], cr[0], o);
                        o = ffma2(w[3], cl[1], o); o = ffma2(w[4], cc[1], o); o = ffma2(w[5], cr[1], o);
                        o = ffma2(w[6], cl[2], o); o = ffma2(w[7], cc[2], o); o = ffma2(w[8], cr[2], o);
                        *reinterpret_cast<float2*>(pb + j * kPatchPitch) = o;
                    }
                }
            }
            pipe_arrive(pp, BAR_PATCH_FULL + b);
            // chunks before the next tile's window are not read again
            while (released < ci_next - 1) {
                pipe_arrive(pp, BAR_H_EMPTY + (released & (kChunks - 1)));
                ++released;
            }
            ci = ci_next;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc<256>(pp.tmem);
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
    if (a->dwc_w && !make_map_grid4d_u16(&a->tm_h, a->v, S, (uint64_t)a->H, (uint64_t)a->W, (uint32_t)a->plan.rows_b, (uint32_t)(a->W + 2))) return false;
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
