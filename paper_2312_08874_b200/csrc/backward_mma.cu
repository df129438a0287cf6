// Backward pass of the agent-attention module (Eq. 6): the two gradient stages on the tensor cores
// (mma.sync m16n8k16, 16-bit operands, fp32 accumulation) for n <= 64 agents and d = 64.
//
// Same mathematics and the same tiling over tokens as the fp32 kernels of backward.cu (modes kBcast2 and
// kAgg1 there); here A, V_A / dV_A, the probabilities P and the logit gradients dS are rounded to the
// storage type to serve as tensor-core operands, as in the forward pass.  A block of four warps walks
// tiles of 64 tokens of one slab:
//   rows phase   warp w owns tokens 16w..16w+15: S = X A^T and dP = Y M^T (X = Q or K, Y = dO or V,
//                M = V_A or dV_A), softmax and its Jacobian in the accumulator layout, bias-gradient atomics,
//                then the per-token products dS A (dQ or dK) and P dV_A (dV) with P, dS re-used as A operands;
//   sums phase   warp w owns agents 16w..16w+15: P^T Y (dV_A) and dS^T X (dA) with P and dS read back
//                transposed from shared memory, accumulated in registers across the block's tiles and added
//                to global memory once per block with atomics.
#include "common.cuh"
#include "kernels.h"

namespace aa {

namespace {

constexpr int kThreads = 128;
constexpr int kNP = 64;          // agents, padded
constexpr int kD = 64;           // channels
constexpr int kTT = 64;          // tokens per tile
constexpr int kPA = 72;          // row pitch of the shared-memory matrices in elements (144 bytes)
constexpr int kMat = 64 * kPA;   // elements per matrix

template <typename T, bool BCAST>
__global__ void __launch_bounds__(kThreads, 3) bwd_mma_kernel(BwdArgs p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* sA = reinterpret_cast<T*>(smem_raw);      // [agent][c]   A
    T* sM = sA + kMat;                           // [agent][c]   V_A (broadcast stage) or dV_A (aggregation stage)
    T* sX = sM + kMat;                           // [token][c]   Q or K
    T* sY = sX + kMat;                           // [token][c]   dO or V
    T* sP = sY + kMat;                           // [token][agent] probabilities
    T* sG = sP + kMat;                           // [token][agent] logit gradients
    T* sM2 = sG + kMat;                          // [agent][c]   rounding residual of M: dP uses M = sM + sM2
    float* sStat = reinterpret_cast<float*>(sM2 + kMat);  // [2][64]: lse, dot (aggregation stage)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int slab = blockIdx.x / p.chunks, chunk = blockIdx.x - slab * p.chunks;
    const int head = slab % p.heads;
    const int n = p.n, N = p.N;

    for (int i = tid; i < kNP * kD; i += kThreads) {
        const int r = i >> 6, c = i & 63;
        const bool in = r < n;
        sA[r * kPA + c] = Elem<T>::from_f32(in ? p.m0[((size_t)slab * n + r) * kD + c] : 0.f);
        // dP = Y M^T feeds the difference dP - rowsum(P o dP), which cancels the part the agents have in common
        // (rows of V_A are close to the mean of V): M is carried as two 16-bit terms so that its rounding error
        // (2^-9 of the common part) does not dominate that difference
        const float mv = in ? p.m1[((size_t)slab * n + r) * kD + c] : 0.f;
        const T hi = Elem<T>::from_f32(mv);
        sM[r * kPA + c] = hi;
        sM2[r * kPA + c] = Elem<T>::from_f32(mv - Elem<T>::to_f32(hi));
    }
    if (!BCAST && tid < kNP) {
        sStat[tid] = tid < n ? p.lse[(size_t)slab * n + tid] * kLog2e : 0.f;
        sStat[kNP + tid] = tid < n ? p.dot[(size_t)slab * n + tid] : 0.f;
    }

    float accV[8][4], accA[8][4];                // sums over tokens for agents 16 warp .. + 15, all channels
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) accV[j][e] = accA[j][e] = 0.f;

    const T* xg = static_cast<const T*>(p.x) + (size_t)slab * N * kD;
    const T* yg = static_cast<const T*>(p.y) + (size_t)slab * N * kD;
    const T* bias = static_cast<const T*>(p.bias);
    const float scale_log2 = p.scale * kLog2e;
    const int tile_end = min((chunk + 1) * p.tiles_per_chunk, p.tiles);

    for (int tile = chunk * p.tiles_per_chunk; tile < tile_end; ++tile) {
        const int tok0 = tile * kTT;
        __syncthreads();                                   // the previous tile's readers are done
        for (int e = tid; e < kTT * (kD / 8); e += kThreads) {
            const int r = e >> 3, ch = e & 7;
            const bool ok = tok0 + r < N;
            const size_t off = ok ? ((size_t)(tok0 + r) * kD + ch * 8) : 0;
            cp_async16(sX + r * kPA + ch * 8, xg + off, ok ? 16 : 0);
            cp_async16(sY + r * kPA + ch * 8, yg + off, ok ? 16 : 0);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();

        // ---------------------------------------------------------------- rows phase: tokens 16 warp ..
        const int r0 = warp * 16;
        const int tok_a = tok0 + r0 + g, tok_b = tok_a + 8;
        const bool va = tok_a < N, vb = tok_b < N;
        float sc[8][4], dp[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[j][e] = dp[j][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t xf[4], yf[4];
            const int arow = r0 + (lane & 7) + ((lane >> 3) & 1) * 8, acol = ks * 16 + (lane >> 4) * 8;
            ldmatrix_x4(xf[0], xf[1], xf[2], xf[3], sX + arow * kPA + acol);
            ldmatrix_x4(yf[0], yf[1], yf[2], yf[3], sY + arow * kPA + acol);
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                const int brow = np * 16 + (lane & 7) + (lane >> 4) * 8, bcol = ks * 16 + ((lane >> 3) & 1) * 8;
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, sA + brow * kPA + bcol);
                mma16816<T>(sc[2 * np], xf, b0, b1);
                mma16816<T>(sc[2 * np + 1], xf, b2, b3);
                ldmatrix_x4(b0, b1, b2, b3, sM + brow * kPA + bcol);
                mma16816<T>(dp[2 * np], yf, b0, b1);
                mma16816<T>(dp[2 * np + 1], yf, b2, b3);
                ldmatrix_x4(b0, b1, b2, b3, sM2 + brow * kPA + bcol);
                mma16816<T>(dp[2 * np], yf, b0, b1);
                mma16816<T>(dp[2 * np + 1], yf, b2, b3);
            }
        }
        // logits in the log2 domain: scale * log2e * (x . a) + log2e * bias; columns past n are masked
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int col = 8 * j + 2 * t4 + (e & 1);
                const int tok = (e & 2) ? tok_b : tok_a;
                const bool ok = col < n && tok < N;
                float b = 0.f;
                if (bias && ok)
                    b = BCAST ? Elem<T>::to_f32(bias[((size_t)head * N + tok) * n + col])
                              : Elem<T>::to_f32(bias[((size_t)head * n + col) * N + tok]);
                sc[j][e] = ok ? fmaf(sc[j][e], scale_log2, b * kLog2e) : -INFINITY;
            }
        if (BCAST) {
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                m0 = fmaxf(m0, fmaxf(sc[j][0], sc[j][1]));
                m1 = fmaxf(m1, fmaxf(sc[j][2], sc[j][3]));
            }
            m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
            m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
            m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
            m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                sc[j][0] = va ? fast_exp2(sc[j][0] - m0) : 0.f;
                sc[j][1] = va ? fast_exp2(sc[j][1] - m0) : 0.f;
                sc[j][2] = vb ? fast_exp2(sc[j][2] - m1) : 0.f;
                sc[j][3] = vb ? fast_exp2(sc[j][3] - m1) : 0.f;
                l0 += sc[j][0] + sc[j][1];
                l1 += sc[j][2] + sc[j][3];
            }
            l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
            l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
            const float i0 = va ? 1.f / l0 : 0.f, i1 = vb ? 1.f / l1 : 0.f;
            float d0 = 0.f, d1 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                sc[j][0] *= i0; sc[j][1] *= i0; sc[j][2] *= i1; sc[j][3] *= i1;
                d0 += sc[j][0] * dp[j][0] + sc[j][1] * dp[j][1];
                d1 += sc[j][2] * dp[j][2] + sc[j][3] * dp[j][3];
            }
            d0 += __shfl_xor_sync(0xffffffffu, d0, 1);
            d0 += __shfl_xor_sync(0xffffffffu, d0, 2);
            d1 += __shfl_xor_sync(0xffffffffu, d1, 1);
            d1 += __shfl_xor_sync(0xffffffffu, d1, 2);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                dp[j][0] = sc[j][0] * (dp[j][0] - d0); dp[j][1] = sc[j][1] * (dp[j][1] - d0);
                dp[j][2] = sc[j][2] * (dp[j][2] - d1); dp[j][3] = sc[j][3] * (dp[j][3] - d1);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = 8 * j + 2 * t4 + (e & 1);
                    const float pr = fast_exp2(sc[j][e] - sStat[col]);     // exp2(-inf) = 0 for masked entries
                    sc[j][e] = pr;
                    dp[j][e] = pr * (dp[j][e] - sStat[kNP + col]);
                }
        }
        // sc = P, dp = dS (fp32).  Bias gradient, then both as 16-bit operands (registers and shared memory).
        if (p.dbias) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = 8 * j + 2 * t4 + (e & 1);
                    const int tok = (e & 2) ? tok_b : tok_a;
                    if (col < n && tok < N)
                        atomicAdd(BCAST ? p.dbias + ((size_t)head * N + tok) * n + col
                                        : p.dbias + ((size_t)head * n + col) * N + tok, dp[j][e]);
                }
        }
        uint32_t pk[8][2], gk[8][2];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            pk[j][0] = pack2<T>(sc[j][0], sc[j][1]); pk[j][1] = pack2<T>(sc[j][2], sc[j][3]);
            gk[j][0] = pack2<T>(dp[j][0], dp[j][1]); gk[j][1] = pack2<T>(dp[j][2], dp[j][3]);
            const int col = 8 * j + 2 * t4;
            *reinterpret_cast<uint32_t*>(sP + (r0 + g) * kPA + col) = pk[j][0];
            *reinterpret_cast<uint32_t*>(sP + (r0 + g + 8) * kPA + col) = pk[j][1];
            *reinterpret_cast<uint32_t*>(sG + (r0 + g) * kPA + col) = gk[j][0];
            *reinterpret_cast<uint32_t*>(sG + (r0 + g + 8) * kPA + col) = gk[j][1];
        }
        // per-token products: row0 = scale * dS A  (dQ or dK);  aggregation stage also row1 = P dV_A  (dV)
#pragma unroll
        for (int which = 0; which < (BCAST ? 1 : 2); ++which) {
            float o[8][4];
#pragma unroll
            for (int j = 0; j < 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
            const T* sB = which == 0 ? sA : sM;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t af[4];
                if (which == 0) { af[0] = gk[2 * kk][0]; af[1] = gk[2 * kk][1]; af[2] = gk[2 * kk + 1][0]; af[3] = gk[2 * kk + 1][1]; }
                else            { af[0] = pk[2 * kk][0]; af[1] = pk[2 * kk][1]; af[2] = pk[2 * kk + 1][0]; af[3] = pk[2 * kk + 1][1]; }
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(b0, b1, b2, b3,
                                      sB + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * kPA + np * 16 + (lane >> 4) * 8);
                    mma16816<T>(o[2 * np], af, b0, b1);
                    mma16816<T>(o[2 * np + 1], af, b2, b3);
                }
            }
            float* dst = which == 0 ? p.row0 : p.row1;
            const float f = which == 0 ? p.scale : 1.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int col = 8 * j + 2 * t4;
                if (va) *reinterpret_cast<float2*>(dst + ((size_t)slab * N + tok_a) * kD + col) = make_float2(f * o[j][0], f * o[j][1]);
                if (vb) *reinterpret_cast<float2*>(dst + ((size_t)slab * N + tok_b) * kD + col) = make_float2(f * o[j][2], f * o[j][3]);
            }
        }
        __syncthreads();                                   // P and dS of all 64 tokens are in shared memory

        // ---------------------------------------------------------------- sums phase: agents 16 warp ..
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {                   // 16 tokens per step
            const int trow = ks * 16 + (lane & 7) + (lane >> 4) * 8, mcol = r0 + ((lane >> 3) & 1) * 8;
            uint32_t pf[4], gf[4];
            if (BCAST) ldmatrix_x4_trans(pf[0], pf[1], pf[2], pf[3], sP + trow * kPA + mcol);
            ldmatrix_x4_trans(gf[0], gf[1], gf[2], gf[3], sG + trow * kPA + mcol);
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                const int brow = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, bcol = np * 16 + (lane >> 4) * 8;
                uint32_t b0, b1, b2, b3;
                if (BCAST) {
                    ldmatrix_x4_trans(b0, b1, b2, b3, sY + brow * kPA + bcol);
                    mma16816<T>(accV[2 * np], pf, b0, b1);
                    mma16816<T>(accV[2 * np + 1], pf, b2, b3);
                }
                ldmatrix_x4_trans(b0, b1, b2, b3, sX + brow * kPA + bcol);
                mma16816<T>(accA[2 * np], gf, b0, b1);
                mma16816<T>(accA[2 * np + 1], gf, b2, b3);
            }
        }
    }

    const int ra = warp * 16 + g, rb = ra + 8;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int col = 8 * j + 2 * t4;
        float* va0 = p.outer0 + ((size_t)slab * n + ra) * kD + col;
        float* va1 = p.outer0 + ((size_t)slab * n + rb) * kD + col;
        float* da0 = p.outer1 + ((size_t)slab * n + ra) * kD + col;
        float* da1 = p.outer1 + ((size_t)slab * n + rb) * kD + col;
        if (ra < n) {
            if (BCAST) { atomicAdd(va0, accV[j][0]); atomicAdd(va0 + 1, accV[j][1]); }
            atomicAdd(da0, p.scale * accA[j][0]); atomicAdd(da0 + 1, p.scale * accA[j][1]);
        }
        if (rb < n) {
            if (BCAST) { atomicAdd(va1, accV[j][2]); atomicAdd(va1 + 1, accV[j][3]); }
            atomicAdd(da1, p.scale * accA[j][2]); atomicAdd(da1 + 1, p.scale * accA[j][3]);
        }
    }
}

// Floats per agent row of a stage-1 partial: running max (log2 domain), running sum, 64 accumulators.
constexpr int kPartRow = 2 + kD;

// Aggregation stage recomputed (flash-attention style, agents as rows): per block, the running max and sum of
// the logits of each agent over the block's tokens and the unnormalised sum of exp(S - max) V.  Warp w owns
// agents 16w..16w+15; P enters the product with V as two 16-bit terms, so that V_A keeps fp32-level accuracy
// (its small differences between agents are what the broadcast stage's gradient is made of).
template <typename T>
__global__ void __launch_bounds__(kThreads, 3) bwd_fwd1_mma_kernel(BwdArgs p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* sA = reinterpret_cast<T*>(smem_raw);      // [agent][c]
    T* sX = sA + kMat;                           // [token][c]  K
    T* sY = sX + kMat;                           // [token][c]  V
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int slab = blockIdx.x / p.chunks, chunk = blockIdx.x - slab * p.chunks;
    const int head = slab % p.heads;
    const int n = p.n, N = p.N;
    for (int i = tid; i < kNP * kD; i += kThreads) {
        const int r = i >> 6, c = i & 63;
        sA[r * kPA + c] = Elem<T>::from_f32(r < n ? p.m0[((size_t)slab * n + r) * kD + c] : 0.f);
    }
    __syncthreads();
    const int r0 = warp * 16;
    uint32_t af[4][4];
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
        ldmatrix_x4(af[ks][0], af[ks][1], af[ks][2], af[ks][3],
                    sA + (r0 + (lane & 7) + ((lane >> 3) & 1) * 8) * kPA + ks * 16 + (lane >> 4) * 8);
    const int ag_a = r0 + g, ag_b = ag_a + 8;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

    const T* xg = static_cast<const T*>(p.x) + (size_t)slab * N * kD;
    const T* yg = static_cast<const T*>(p.y) + (size_t)slab * N * kD;
    const T* bias = static_cast<const T*>(p.bias);
    const float scale_log2 = p.scale * kLog2e;
    const int tile_end = min((chunk + 1) * p.tiles_per_chunk, p.tiles);
    for (int tile = chunk * p.tiles_per_chunk; tile < tile_end; ++tile) {
        const int tok0 = tile * kTT;
        __syncthreads();
        for (int e = tid; e < kTT * (kD / 8); e += kThreads) {
            const int r = e >> 3, ch = e & 7;
            const bool ok = tok0 + r < N;
            const size_t off = ok ? ((size_t)(tok0 + r) * kD + ch * 8) : 0;
            cp_async16(sX + r * kPA + ch * 8, xg + off, ok ? 16 : 0);
            cp_async16(sY + r * kPA + ch * 8, yg + off, ok ? 16 : 0);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
        float sc[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3,
                            sX + (np * 16 + (lane & 7) + (lane >> 4) * 8) * kPA + ks * 16 + ((lane >> 3) & 1) * 8);
                mma16816<T>(sc[2 * np], af[ks], b0, b1);
                mma16816<T>(sc[2 * np + 1], af[ks], b2, b3);
            }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int tok = tok0 + 8 * j + 2 * t4 + (e & 1);
                const int ag = (e & 2) ? ag_b : ag_a;
                const bool ok = ag < n && tok < N;
                float b = 0.f;
                if (bias && ok) b = Elem<T>::to_f32(bias[((size_t)head * n + ag) * N + tok]);
                sc[j][e] = ok ? fmaf(sc[j][e], scale_log2, b * kLog2e) : -INFINITY;
                if (e & 2) mx1 = fmaxf(mx1, sc[j][e]); else mx0 = fmaxf(mx0, sc[j][e]);
            }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const bool live0 = mn0 > -INFINITY, live1 = mn1 > -INFINITY;     // rows past n never come alive
        const float c0 = live0 ? fast_exp2(m0 - mn0) : 1.f, c1 = live1 ? fast_exp2(m1 - mn1) : 1.f;
        m0 = mn0; m1 = mn1;
        l0 *= c0; l1 *= c1;
        uint32_t hi[8][2], lo[8][2];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            acc[j][0] *= c0; acc[j][1] *= c0; acc[j][2] *= c1; acc[j][3] *= c1;
            const float p0 = live0 ? fast_exp2(sc[j][0] - mn0) : 0.f, p1 = live0 ? fast_exp2(sc[j][1] - mn0) : 0.f;
            const float p2 = live1 ? fast_exp2(sc[j][2] - mn1) : 0.f, p3 = live1 ? fast_exp2(sc[j][3] - mn1) : 0.f;
            l0 += p0 + p1;
            l1 += p2 + p3;
            hi[j][0] = pack2<T>(p0, p1);
            hi[j][1] = pack2<T>(p2, p3);
            const float2 h0 = unpack2<T>(hi[j][0]), h1 = unpack2<T>(hi[j][1]);
            lo[j][0] = pack2<T>(p0 - h0.x, p1 - h0.y);
            lo[j][1] = pack2<T>(p2 - h1.x, p3 - h1.y);
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const uint32_t ah[4] = {hi[2 * kk][0], hi[2 * kk][1], hi[2 * kk + 1][0], hi[2 * kk + 1][1]};
            const uint32_t al[4] = {lo[2 * kk][0], lo[2 * kk][1], lo[2 * kk + 1][0], lo[2 * kk + 1][1]};
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(b0, b1, b2, b3,
                                  sY + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * kPA + np * 16 + (lane >> 4) * 8);
                mma16816<T>(acc[2 * np], ah, b0, b1);
                mma16816<T>(acc[2 * np + 1], ah, b2, b3);
                mma16816<T>(acc[2 * np], al, b0, b1);
                mma16816<T>(acc[2 * np + 1], al, b2, b3);
            }
        }
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    float* pa = p.part + (((size_t)slab * p.chunks + chunk) * kNP + ag_a) * kPartRow;
    float* pb = p.part + (((size_t)slab * p.chunks + chunk) * kNP + ag_b) * kPartRow;
    if (t4 == 0) { pa[0] = m0; pa[1] = l0; pb[0] = m1; pb[1] = l1; }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int col = 2 + 8 * j + 2 * t4;
        *reinterpret_cast<float2*>(pa + col) = make_float2(acc[j][0], acc[j][1]);
        *reinterpret_cast<float2*>(pb + col) = make_float2(acc[j][2], acc[j][3]);
    }
}

// Merge of the stage-1 partials in chunk order: V_A (fp32) and the natural-log sum-exp of each agent's logits.
__global__ void bwd_fwd1_merge_kernel(BwdArgs p, float* va, float* lse) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;       // (slab * n + r) * 64 + c
    if (i >= (size_t)p.slabs * p.n * kD) return;
    const int c = (int)(i & 63);
    const size_t sr = i >> 6;
    const int r = (int)(sr % p.n), slab = (int)(sr / p.n);
    const float* base = p.part + ((size_t)slab * p.chunks * kNP + r) * kPartRow;
    const size_t stride = (size_t)kNP * kPartRow;
    float M = -INFINITY;
    for (int ch = 0; ch < p.chunks; ++ch) M = fmaxf(M, base[ch * stride]);
    float L = 0.f, v = 0.f;
    for (int ch = 0; ch < p.chunks; ++ch) {
        const float w = exp2f(base[ch * stride] - M);
        L = fmaf(base[ch * stride + 1], w, L);
        v = fmaf(base[ch * stride + 2 + c], w, v);
    }
    va[i] = v / L;
    if (c == 0) lse[sr] = (M + log2f(L)) * 0.6931471805599453f;
}

constexpr size_t kSmemBytes = 7 * (size_t)kMat * 2 + 2 * kNP * sizeof(float);

template <typename T, bool BCAST>
cudaError_t launch(const BwdArgs& a, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(bwd_mma_kernel<T, BCAST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    bwd_mma_kernel<T, BCAST><<<a.slabs * a.chunks, kThreads, kSmemBytes, st>>>(a);
    return cudaGetLastError();
}

}  // namespace

size_t backward_mma_part_floats(int slabs, const BwdPlan& pl) { return (size_t)slabs * pl.chunks * kNP * kPartRow; }

cudaError_t launch_backward_fwd1_mma(int dtype, const BwdArgs& a, float* va, float* lse, cudaStream_t st) {
    const size_t smem = 3 * (size_t)kMat * 2;
    if (dtype == kBF16) {
        cudaError_t e = cudaFuncSetAttribute(bwd_fwd1_mma_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        bwd_fwd1_mma_kernel<__nv_bfloat16><<<a.slabs * a.chunks, kThreads, smem, st>>>(a);
    } else if (dtype == kF16) {
        cudaError_t e = cudaFuncSetAttribute(bwd_fwd1_mma_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        bwd_fwd1_mma_kernel<__half><<<a.slabs * a.chunks, kThreads, smem, st>>>(a);
    } else {
        return cudaErrorInvalidValue;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t total = (size_t)a.slabs * a.n * kD;
    bwd_fwd1_merge_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(a, va, lse);
    return cudaGetLastError();
}

bool backward_mma_eligible(int dtype, int n, int d) { return (dtype == kBF16 || dtype == kF16) && n <= kNP && d == kD; }

BwdPlan plan_backward_mma(int slabs, int N, int sm_count) {
    BwdPlan pl;
    pl.tile = kTT;
    pl.np = kNP;
    pl.tiles = (N + kTT - 1) / kTT;
    const int slots = 3 * sm_count;                     // three blocks per SM
    int chunks = slots >= slabs ? slots / slabs : 1;
    chunks = max(1, min(chunks, pl.tiles));
    pl.tiles_per_chunk = (pl.tiles + chunks - 1) / chunks;
    pl.chunks = (pl.tiles + pl.tiles_per_chunk - 1) / pl.tiles_per_chunk;
    return pl;
}

cudaError_t launch_backward_mma(int dtype, bool broadcast_stage, const BwdArgs& a, cudaStream_t st) {
    if (dtype == kBF16) return broadcast_stage ? launch<__nv_bfloat16, true>(a, st) : launch<__nv_bfloat16, false>(a, st);
    if (dtype == kF16) return broadcast_stage ? launch<__half, true>(a, st) : launch<__half, false>(a, st);
    return cudaErrorInvalidValue;
}

}  // namespace aa
