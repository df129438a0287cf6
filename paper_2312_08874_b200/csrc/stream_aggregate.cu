// Agent aggregation V_A = softmax(scale1 * A K^T + B1) V (Eq. 3, Eq. 5) for small agent counts
// (n <= 64, d = 64, 16-bit elements) as a streaming kernel on the 5th-generation tensor cores.
//
// Grid (splits, slabs), one block per SM; a block streams its range of the slab's tokens in tiles of 128
// (K, V and the matching rows of the transposed, padded B1) through a four-stage TMA ring.  The 64 (padded)
// agent rows are stacked twice so that all 128 tensor-memory lanes carry a row: lane r + 64 h owns agent r
// and the token half h of every tile, with its own reference maximum, row sum and accumulator row.
//   warp 4 "producer":  one lane issues every TMA copy, ahead of the others through full/empty mbarriers.
//   warps 5, 6 "MMA issuers": one lane each, one for the logits and one for the products, so that neither
//       instruction stream waits behind the other's barriers.  S = [A | I] [K | B1^T]^T: the agents (times scale1) and an identity block
//       sit in tensor memory as the A operand, so the bias is added inside the contraction and the logits
//       arrive complete, in natural units; eight instructions of 128 columns per tile, one tile ahead.  Then
//       D += P V with the probabilities read from tensor memory too.  (An instruction of this kind takes about
//       48 cycles whatever its width up to 64 columns, 66 at 128: few wide instructions, and the ring stage
//       a compile-time constant so that the issuing thread spends no time on descriptor arithmetic.)
//   warps 0-3 "row warps": read 64 logits from tensor memory, turn them into probabilities relative to the
//       row's reference (fp32 exponentials: the reference sits a margin above the maximum, where a 16-bit
//       exponent argument would be too coarse), add them to the row sum, round them to the operand type and
//       store them back over the logits.  No maximum is taken on this path: a probability >= 2 shows in the
//       top exponent bit of the packed pairs (one OR per pair); only then the reference moves up (true
//       maximum of the tile plus a margin) and the thread rescales its accumulator row.
// The blocks of a slab form a thread-block cluster.  At the end the two token halves of a row meet in shared
// memory, and after a cluster barrier every block merges its share of the agent rows from the partial states
// in its siblings' shared memory (plain distributed-shared-memory loads, fixed order of the blocks:
// bit-reproducible) and writes those rows of V_A.  No partial state goes through global memory.
// Every mbarrier wait is bounded; every block reaches both cluster barriers whatever happened before.
// No TMA multicast.
#include "stream_common.cuh"

namespace aa {

namespace {
constexpr int TK = 128;                // tokens per tile
constexpr int STAGES = 4;
constexpr int NROW = 128;              // row-warp threads
constexpr int NT = NROW + 96;          // + producer warp + two MMA issuer warps (logits; products)
constexpr int kTile = TK * 128;        // swizzled [128][64] tile of 16-bit elements
constexpr int kStage = 3 * kTile;      // K | V | B1^T
constexpr float kMargin = 4.f;         // a new reference sits this far (log2 units) above the tile's maximum
constexpr int kTimeoutTile = 3, kTimeoutLoads = 4, kTimeoutRole = 6;

// shared memory (bytes from a 1024-aligned base)
constexpr int OFF_BAR = 0;
constexpr int OFF_RING = 1024;
constexpr int kSmemBytes = OFF_RING + STAGES * kStage + 1024;
static_assert(kSmemBytes <= 232448 && kSmemBytes > 116 * 1024, "one block per SM");

// mbarriers                                  count          waiter
constexpr int BAR_FULL = 0;       // [STAGES]  tx             MMA issuer
constexpr int BAR_EMPTY = 4;      // [STAGES]  commit         producer
constexpr int BAR_S_FULL = 8;     // [2]       commit         row warps
constexpr int BAR_P_FULL = 10;    // [2]       row threads    MMA issuer
constexpr int BAR_PV = 12;        // [2]       commit         row warps (only when a reference moves, and at the end)
constexpr int BAR_A = 14;         //           row threads    MMA issuer      the agent operand is in tensor memory
constexpr int BAR_S_EMPTY = 15;   // [2]       row threads    MMA issuer      the logits have been read
constexpr int BAR_DRAIN = 17;     // [2]       commit         each MMA issuer, once, at its end
constexpr int kBars = 19;

// tensor memory columns: logits 2 x 128, probabilities 2 x 64 (16-bit pairs), accumulator 64,
// agent operand 32 (64 channels) + 32 (identity, 64 agents)
constexpr uint32_t TM_S = 0, TM_P = 256, TM_D = 384, TM_A = 448;

// Probabilities of one thread's 64 logits relative to the reference (nb = minus the reference, log2 units):
// packed pairs in pk, their fp32 sum in `sum`; returns the OR of the pairs.  Columns >= valid weigh nothing.
template <typename T, bool kRagged>
__device__ __forceinline__ uint32_t row_probs(const uint32_t (&sa)[32], const uint32_t (&sb)[32], float nb, int valid,
                                              uint32_t (&pk)[32], float& sum) {
    const float2 l2e = make_float2(kLog2e, kLog2e), nb2 = make_float2(nb, nb);
    float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
    uint32_t orr = 0u;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float2 x0 = ffma2(make_float2(__uint_as_float(sa[2 * j]), __uint_as_float(sa[2 * j + 1])), l2e, nb2);
        const float2 x1 = ffma2(make_float2(__uint_as_float(sb[2 * j]), __uint_as_float(sb[2 * j + 1])), l2e, nb2);
        float2 e0 = make_float2(fast_exp2(x0.x), fast_exp2(x0.y)), e1 = make_float2(fast_exp2(x1.x), fast_exp2(x1.y));
        if (kRagged) {
            if (2 * j >= valid) e0.x = 0.f;
            if (2 * j + 1 >= valid) e0.y = 0.f;
            if (32 + 2 * j >= valid) e1.x = 0.f;
            if (33 + 2 * j >= valid) e1.y = 0.f;
        }
        pk[j] = Pair<T>::cvt(e0.x, e0.y);
        pk[16 + j] = Pair<T>::cvt(e1.x, e1.y);
        orr |= pk[j] | pk[16 + j];
        s0 = fadd2(s0, e0);
        s1 = fadd2(s1, e1);
    }
    sum = (s0.x + s0.y) + (s1.x + s1.y);
    return orr;
}

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
// shared-memory address of the same variable in block `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}
}  // namespace

template <typename T>
__global__ void __launch_bounds__(NT, 1) stream_aggregate_kernel(const __grid_constant__ StreamArgs p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_dead;
    __shared__ uint32_t s_tmem;
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, slab = blockIdx.y;
    const int head = slab % p.heads;
    const int N = p.H * p.W, n = p.n;
    const bool has_bias = p.b1 != nullptr;
    const int tiles_all = (N + TK - 1) / TK;
    const int t0 = split * p.plan.tiles_per_split, t1 = min(tiles_all, t0 + p.plan.tiles_per_split);
    const int tiles = t1 - t0;                            // >= 1 by the plan

    Pipe pp;
    pp.status = p.status;
    pp.dead = &s_dead;
    pp.bars = smem_u32(smem + OFF_BAR);
    pp.ph = 0u;
    if (tid == 0) {
        s_dead = 0;
        for (int i = 0; i < kBars; ++i)
            mbar_init(pp.bars + 8 * i, ((i >= BAR_P_FULL && i < BAR_PV) || (i >= BAR_A && i < BAR_DRAIN)) ? (uint32_t)NROW : 1u);
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc<512>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem = s_tmem;
    const uint32_t ring = smem_u32(smem + OFF_RING);
    pdl_launch_dependents();     // the broadcast kernel may set itself up on idle SMs; it waits for this grid to finish

    if (warp == 4) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const uint32_t tx = (has_bias ? 3u : 2u) * kTile;
            // K and V are inputs of the call: the first ring stages are requested before the wait for the
            // preceding kernel, whose results (scaled agents, prepared bias) are only needed after it
            const int first = min(tiles, STAGES);
            for (int i = 0; i < first; ++i) {
                const uint32_t bar = pipe_bar(pp, BAR_FULL + i), dst = ring + i * kStage;
                mbar_arrive_expect_tx(bar, tx);
                tma_load_3d(dst, &p.tm_k, 0, (t0 + i) * TK, slab, bar);
                tma_load_3d(dst + kTile, &p.tm_v, 0, (t0 + i) * TK, slab, bar);
            }
            pdl_wait();
            if (has_bias)
                for (int i = 0; i < first; ++i)
                    tma_load_3d(ring + i * kStage + 2 * kTile, &p.tm_b1, 0, (t0 + i) * TK, head, pipe_bar(pp, BAR_FULL + i));
            for (int i = first; i < tiles && !pipe_dead(pp); ++i) {
                const int s = i % STAGES, c0 = (t0 + i) * TK;
                wait_spin(pp, BAR_EMPTY + s, (i / STAGES) - 1, kTimeoutRole);
                const uint32_t bar = pipe_bar(pp, BAR_FULL + s), dst = ring + s * kStage;
                mbar_arrive_expect_tx(bar, tx);
                tma_load_3d(dst, &p.tm_k, 0, c0, slab, bar);
                tma_load_3d(dst + kTile, &p.tm_v, 0, c0, slab, bar);
                if (has_bias) tma_load_3d(dst + 2 * kTile, &p.tm_b1, 0, c0, head, bar);
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer: logits, up to two tiles ahead
        // (the whole warp runs the loop; one elected lane issues)
        {
            const uint32_t idS = umma_idesc(fmt, 128, 128, 0);
            const uint64_t dRing = umma_desc_sw128(ring);
            const uint32_t tA = pp.tmem + TM_A, tS = pp.tmem + TM_S;
            // descriptor start addresses count 16-byte units: + 2 per K-step of a K-major operand (32 bytes).
            // `u` is a compile-time constant (the tile loop is unrolled over the ring).
            wait_spin(pp, BAR_A, 0, kTimeoutLoads);
            for (int i0 = 0; i0 < tiles && !pipe_dead(pp); i0 += STAGES) {
#pragma unroll
                for (int u = 0; u < STAGES; ++u) {
                    const int i = i0 + u;
                    if (i < tiles) {
                        // the logits buffer is free once the row warps have read tile i - 2 out of it
                        if (i >= 2) wait_spin(pp, BAR_S_EMPTY + (u & 1), (i >> 1) - 1, kTimeoutRole);
                        wait_spin(pp, BAR_FULL + u, i / STAGES, kTimeoutTile);
                        tc_fence_after_sync();
                        const uint64_t dK = dRing + (uint64_t)(u * (kStage >> 4));
                        const uint32_t dd = tS + 128 * (u & 1);
                        umma_ts_w(dd, tA, dK, idS, 0u);
#pragma unroll
                        for (int k = 1; k < 4; ++k) umma_ts_w(dd, tA + 8 * k, dK + 2 * k, idS, 1u);
                        if (has_bias) {
                            const uint64_t dB = dK + (uint64_t)(2 * kTile >> 4);
#pragma unroll
                            for (int k = 0; k < 4; ++k) umma_ts_w(dd, tA + 32 + 8 * k, dB + 2 * k, idS, 1u);
                        }
                        umma_commit_w(pipe_bar(pp, BAR_S_FULL + (u & 1)));
                    }
                }
            }
            umma_drain_w(pp, BAR_DRAIN);
        }
        __syncwarp();
    } else if (warp == 6) {
        // ------------------------------------------------------------------ MMA issuer: products
        {
            const uint32_t idPV = umma_idesc(fmt, 128, 64, 1);
            const uint64_t dRing = umma_desc_sw128(ring);
            const uint32_t tD = pp.tmem + TM_D, tPb = pp.tmem + TM_P;
            // + 128 per K-step of an MN-major operand (16 rows of 128 bytes)
            for (int i0 = 0; i0 < tiles && !pipe_dead(pp); i0 += STAGES) {
#pragma unroll
                for (int u = 0; u < STAGES; ++u) {
                    const int i = i0 + u;
                    if (i < tiles) {
                        wait_spin(pp, BAR_P_FULL + (u & 1), i >> 1, kTimeoutRole);
                        tc_fence_after_sync();
                        const uint64_t dV = dRing + (uint64_t)(u * (kStage >> 4) + (kTile >> 4));
                        const uint32_t tP = tPb + 64 * (u & 1);
                        umma_ts_w(tD, tP, dV, idPV, i > 0 ? 1u : 0u);
#pragma unroll
                        for (int k = 1; k < 8; ++k) umma_ts_w(tD, tP + 8 * k, dV + 128 * k, idPV, 1u);
                        umma_commit_w(pipe_bar(pp, BAR_EMPTY + u));
                        umma_commit_w(pipe_bar(pp, BAR_PV + (u & 1)));
                    }
                }
            }
            umma_drain_w(pp, BAR_DRAIN + 1);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ row warps
        const int r = tid & 63, h = tid >> 6;              // agent row (padded), token half
        const uint32_t lane_base = ((uint32_t)(32 * warp)) << 16;
        pdl_wait();          // the scaled agents come from the preceding kernel
        {
            // this lane's row of the A operand: 64 channels of scale1 * A, then the identity row that picks
            // the agent's own bias (rows past n stay zero: their logits are 0 and their results unused)
            uint32_t ra[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) ra[j] = 0u;
            if (r < n) {
                const uint4* src = reinterpret_cast<const uint4*>(static_cast<const T*>(p.a1s) + ((size_t)slab * n + r) * 64);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 v = __ldg(src + j);
                    ra[4 * j] = v.x; ra[4 * j + 1] = v.y; ra[4 * j + 2] = v.z; ra[4 * j + 3] = v.w;
                }
            }
            tmem_st32(pp.tmem + TM_A + lane_base, ra);
            const uint32_t one = (r < n) ? (Pair<T>::kOne << (16 * (r & 1))) : 0u;
#pragma unroll
            for (int j = 0; j < 32; ++j) ra[j] = (j == (r >> 1)) ? one : 0u;
            tmem_st32(pp.tmem + TM_A + 32 + lane_base, ra);
            // the other token half's share of both probability operands stays zero for the whole kernel
#pragma unroll
            for (int j = 0; j < 32; ++j) ra[j] = 0u;
            tmem_st32(pp.tmem + TM_P + 32 * (1 - h) + lane_base, ra);
            tmem_st32(pp.tmem + TM_P + 64 + 32 * (1 - h) + lane_base, ra);
            tmem_st_wait();
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_A);
        }
        const uint32_t tD = pp.tmem + TM_D + lane_base;
        float nb = 0.f;                                    // minus the row's reference, log2 units
        float l = 0.f;                                     // row sum of the probabilities, relative to the reference
        bool started = false;                              // the accumulator row holds something
        for (int i = 0; i < tiles; ++i) {
            const int b = i & 1;
            const int valid = max(0, min(64, N - ((t0 + i) * TK + 64 * h)));      // tokens of this half: uniform per warp
            const uint32_t tS = pp.tmem + TM_S + 128 * b + lane_base;
            wait_par(pp, BAR_S_FULL + b, i >> 1, kTimeoutTile);
            tc_fence_after_sync();
            uint32_t pk[32];
            if (valid > 0) {
                uint32_t sa[32], sb[32];
                tmem_ld32(tS + 64 * h, sa);
                tmem_ld32(tS + 64 * h + 32, sb);
                tmem_ld_wait();
                tc_fence_before_sync();
                pipe_arrive(pp, BAR_S_EMPTY + b);          // the next logits may land in this buffer
                float sum = 0.f;
                uint32_t orr = kPairGe2;
                if (started)
                    orr = valid == 64 ? row_probs<T, false>(sa, sb, nb, valid, pk, sum) : row_probs<T, true>(sa, sb, nb, valid, pk, sum);
                const bool trig = (orr & kPairGe2) != 0u;
                if (__any_sync(0xffffffffu, trig)) {       // first tile, or rare: some row's logits outgrew its reference
                    float mx = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < valid) mx = fmaxf(mx, __uint_as_float(sa[j]));
                        if (32 + j < valid) mx = fmaxf(mx, __uint_as_float(sb[j]));
                    }
                    float nb_new = nb;
                    if (trig) {
                        float ref = fmaf(mx, kLog2e, kMargin);
                        if (started) ref = fmaxf(ref, -nb);
                        nb_new = -ref;
                    }
                    const float corr = started ? exp2f(nb_new - nb) : 1.f;
                    if (i > 0) {
                        // every product into this thread's accumulator row is done before the row is rescaled
                        wait_par(pp, BAR_PV + ((i - 1) & 1), (i - 1) >> 1, kTimeoutTile);
                        tc_fence_after_sync();
                        uint32_t ra[32];
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            tmem_ld32(tD + 32 * hh, ra);
                            tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 32; ++k) ra[k] = __float_as_uint(__uint_as_float(ra[k]) * corr);
                            tmem_st32(tD + 32 * hh, ra);
                        }
                        tmem_st_wait();
                    }
                    l *= corr;
                    nb = nb_new;
                    if (valid == 64) row_probs<T, false>(sa, sb, nb, valid, pk, sum);
                    else row_probs<T, true>(sa, sb, nb, valid, pk, sum);
                }
                l += sum;
                started = true;
            } else {
                tc_fence_before_sync();
                pipe_arrive(pp, BAR_S_EMPTY + b);
#pragma unroll
                for (int j = 0; j < 32; ++j) pk[j] = 0u;
            }
            // the probability operand of this buffer is free once the product of tile i - 2 has read it
            if (i >= 2) { wait_par(pp, BAR_PV + b, (i >> 1) - 1, kTimeoutTile); tc_fence_after_sync(); }
            tmem_st32(pp.tmem + TM_P + 64 * b + 32 * h + lane_base, pk);
            tmem_st_wait();
            tc_fence_before_sync();
            pipe_arrive(pp, BAR_P_FULL + b);
        }
        wait_par(pp, BAR_PV + ((tiles - 1) & 1), (tiles - 1) >> 1, kTimeoutTile);
        tc_fence_after_sync();
        // the two token halves of a row meet in shared memory (the ring is drained: every product is done)
        float o[64];
        {
            uint32_t ra[32], rb[32];
            tmem_ld32(tD, ra);
            tmem_ld32(tD + 32, rb);
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                o[k] = started ? __uint_as_float(ra[k]) : 0.f;
                o[32 + k] = started ? __uint_as_float(rb[k]) : 0.f;
            }
        }
        tc_fence_before_sync();
        const float m_ref = started ? -nb : -INFINITY;     // log2 units
        float* sX = reinterpret_cast<float*>(smem + OFF_RING) + (size_t)r * 68;      // [64][68]: row, reference, sum
        if (h == 1) {
#pragma unroll
            for (int k = 0; k < 16; ++k) *reinterpret_cast<float4*>(sX + 4 * k) = make_float4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            sX[64] = m_ref; sX[65] = l;
        }
        asm volatile("bar.sync 1, %0;\n" ::"n"(NROW) : "memory");
        if (h == 0) {
            // this block's partial state of row r stays in shared memory: row, reference (log2 units), sum
            const float om = sX[64], ol = sX[65];
            const float mm = fmaxf(m_ref, om);
            const float bs = (mm == -INFINITY) ? 0.f : mm;
            const float wa = fast_exp2(m_ref - bs), wb = fast_exp2(om - bs);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float4 xv = *reinterpret_cast<const float4*>(sX + 4 * k);
                *reinterpret_cast<float4*>(sX + 4 * k) =
                    make_float4(o[4 * k] * wa + xv.x * wb, o[4 * k + 1] * wa + xv.y * wb,
                                o[4 * k + 2] * wa + xv.z * wb, o[4 * k + 3] * wa + xv.w * wb);
            }
            sX[64] = mm; sX[65] = l * wa + ol * wb;
        }
    }
    // every block of the slab has its partial state in shared memory; each merges its share of the agent rows
    tc_fence_before_sync();
    cluster_sync_all();
    {
        const int splits = p.plan.splits;
        const int rows_per = (n + splits - 1) / splits;
        const int rb = split * rows_per, re = min(n, rb + rows_per);
        const uint32_t sx0 = ring;                          // [64][68] floats at the start of the ring, in every block
        T* va = static_cast<T*>(p.va_ws) + (size_t)slab * n * 64;
        for (int e = tid; e < (re - rb) * 16; e += NT) {
            const int r = rb + (e >> 4), c4 = e & 15;
            float m[8], l[8];
            float4 a[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                m[q] = -INFINITY; l[q] = 0.f; a[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (q < splits) {
                    const uint32_t row = cluster_map(sx0 + (uint32_t)r * 272u, (uint32_t)q);
                    const float2 ml = ld_cluster_f2(row + 256u);
                    m[q] = ml.x; l[q] = ml.y;
                    a[q] = ld_cluster_f4(row + 16u * c4);
                }
            }
            float mm = m[0];
#pragma unroll
            for (int q = 1; q < 8; ++q) mm = fmaxf(mm, m[q]);
            const float bs = (mm == -INFINITY) ? 0.f : mm;
            float den = 0.f;
            float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float wq = exp2f(m[q] - bs);           // 0 for a block without tokens
                den = fmaf(l[q], wq, den);
                num.x = fmaf(a[q].x, wq, num.x); num.y = fmaf(a[q].y, wq, num.y);
                num.z = fmaf(a[q].z, wq, num.z); num.w = fmaf(a[q].w, wq, num.w);
            }
            const float inv = 1.f / den;
            uint2 o2;
            o2.x = pack2<T>(num.x * inv, num.y * inv);
            o2.y = pack2<T>(num.z * inv, num.w * inv);
            *(reinterpret_cast<uint2*>(va + (size_t)r * 64) + c4) = o2;
        }
    }
    cluster_sync_all();            // no block leaves while a sibling may still read its shared memory
    if (warp == 0) tmem_dealloc<512>(pp.tmem);
}

cudaError_t launch_stream_aggregate(int dtype, const StreamArgs& a, cudaStream_t st) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)a.plan.splits, (unsigned)a.slabs);
    cfg.blockDim = dim3(NT);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;       // the blocks of a slab exchange their partial states
    at[1].val.clusterDim.x = (unsigned)a.plan.splits;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    cudaError_t e;
    if (dtype == kBF16) {
        auto kern = stream_aggregate_kernel<__nv_bfloat16>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        return cudaLaunchKernelEx(&cfg, kern, a);
    }
    if (dtype == kF16) {
        auto kern = stream_aggregate_kernel<__half>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        return cudaLaunchKernelEx(&cfg, kern, a);
    }
    return cudaErrorInvalidValue;
}

}  // namespace aa
