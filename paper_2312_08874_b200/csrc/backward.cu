// Backward pass of the agent-attention module (Eq. 6), fp32 arithmetic on CUDA cores.
//
// With A = Pooling(Q), P1 = softmax(scale1 A K^T + B1), V_A = P1 V, P2 = softmax(scale2 Q A^T + B2)
// and O = P2 V_A + DWC(V), the chain rule gives, for an upstream gradient dO,
//     dV_A = P2^T dO                      dS2 = P2 o (dO V_A^T - rowsum(P2 o dO V_A^T))
//     dQ   = scale2 dS2 A + Pooling^T(dA) dA  = scale2 dS2^T Q + scale1 dS1 K
//     dS1  = P1 o (dV_A V^T - rowsum(P1 o dV_A V^T)),  rowsum(...)[r] = dV_A[r] . V_A[r]
//     dK   = scale1 dS1^T A               dV  = P1^T dV_A + DWC^T(dO)
//     dB1  = sum over the batch of dS1    dB2 = sum over the batch of dS2      dWd = corr(dO, V)
// No N x n matrix is stored: each one is recomputed tile by tile from Q, K, V and the agents.
//
// One kernel template walks tiles of kTile tokens of a slab; a warp owns a token, its lanes own the
// agents (agent r = lane + 32 t).  The agents' matrices sit transposed in shared memory ([d][np], np odd),
// so both "lane = agent" and "lane = channel" reads are conflict-free.  Sums over tokens (V_A, dV_A,
// dA) are kept per thread in registers across the tiles of a block and added to global memory once
// per block with atomics; the bias gradients are added with atomics per element.  The order of those
// additions is not fixed, so the last bits of the results can differ from run to run.
#include "common.cuh"
#include "kernels.h"

#include <cstring>

namespace aa {

namespace {

constexpr int kBwdThreads = 256;
constexpr int kBwdWarps = kBwdThreads / 32;
constexpr int kMaxLaneAgents = 8;                 // 256 agents / 32 lanes
constexpr int kMaxOuter = 16;                     // float4 accumulators per thread: n * d / 4 <= 16 * 256

// 0: n <= 64 and n d <= 4096;  1: n <= 128 and n d <= 8192;  2: n <= 256 and n d <= 16384
__host__ __device__ inline int backward_variant(int n, int d) {
    if (n <= 64 && n * d <= 4096) return 0;
    if (n <= 128 && n * d <= 8192) return 1;
    return 2;
}

enum BwdMode {
    kStats1 = 0,   // running (max, sum) of the aggregation logits over the block's tokens
    kVa1 = 1,      // V_A += P1 V
    kBcast2 = 2,   // dQ = scale2 dS2 A; dV_A += P2^T dO; dA += scale2 dS2^T Q; dB2 += dS2
    kAgg1 = 3      // dK = scale1 dS1^T A; dV = P1^T dV_A; dA += scale1 dS1 K; dB1 += dS1
};

template <typename T>
__device__ __forceinline__ float ld_f32(const T* p, size_t i) { return Elem<T>::to_f32(p[i]); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float f4c(const float4& v, int i) { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }

// NT = agents per lane (n <= 32 NT), KOUT = float4 sums over tokens per thread (n d / 4 <= 256 KOUT),
// TOK = tokens a warp works on at once (they share every load of the agents' matrices).
template <typename T, int MODE, int NT, int KOUT, int TOK>
__global__ void __launch_bounds__(kBwdThreads, KOUT <= 4 ? 2 : 1) bwd_tile_kernel(BwdArgs p) {
    constexpr bool kHasM1 = MODE == kBcast2 || MODE == kAgg1;
    constexpr bool kRowSoftmax = MODE == kBcast2;
    constexpr int kOut = MODE == kStats1 ? 0 : KOUT;
    extern __shared__ __align__(16) float sm[];
    const int d = p.d, n = p.n, np = p.np, tt = p.tile;
    float* m0t = sm;                                        // [d][np]  A^T
    float* m1t = m0t + (size_t)d * np;                      // [d][np]  V_A^T or dV_A^T
    float* xs = m1t + (kHasM1 ? (size_t)d * np : 0);        // [tt][d]  rows of the logits operand
    float* ys = xs + (size_t)tt * d;                        // [tt][d]  rows of the second operand
    float* pt = ys + (size_t)tt * d;                        // [tt][np] probabilities
    float* dst = pt + (size_t)tt * np;                      // [tt][np] logit gradients

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slab = blockIdx.x / p.chunks, chunk = blockIdx.x - slab * p.chunks;
    const int head = slab % p.heads;
    const int nt = (n + 31) >> 5;
    const size_t nd = (size_t)n * d;

    for (int i = tid; i < d * np * (kHasM1 ? 2 : 1); i += kBwdThreads) sm[i] = 0.f;
    __syncthreads();
    for (int i = tid; i < n * d; i += kBwdThreads) {
        const int r = i / d, c = i - r * d;
        m0t[c * np + r] = p.m0[slab * nd + i];
        if (kHasM1) m1t[c * np + r] = p.m1[slab * nd + i];
    }

    float lse[NT], dot[NT];                                // per-agent row statistics of the aggregation
    float run_m[NT], run_l[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
        const int r = lane + 32 * t;
        lse[t] = (MODE == kVa1 || MODE == kAgg1) && r < n ? p.lse[(size_t)slab * n + r] : 0.f;
        dot[t] = MODE == kAgg1 && r < n ? p.dot[(size_t)slab * n + r] : 0.f;
        run_m[t] = -INFINITY;
        run_l[t] = 0.f;
    }
    float4 acc0[KOUT], acc1[KOUT];
#pragma unroll
    for (int k = 0; k < KOUT; ++k) acc0[k] = acc1[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int outer_total = n * (d >> 2);

    const T* xg = static_cast<const T*>(p.x) + (size_t)slab * p.N * d;
    const T* yg = MODE == kStats1 ? nullptr : static_cast<const T*>(p.y) + (size_t)slab * p.N * d;
    const T* bias = static_cast<const T*>(p.bias);
    const int tile_end = min((chunk + 1) * p.tiles_per_chunk, p.tiles);

    for (int tile = chunk * p.tiles_per_chunk; tile < tile_end; ++tile) {
        const int tok0 = tile * tt;
        __syncthreads();                                   // previous tile's readers are done
        for (int i = tid; i < tt * d; i += kBwdThreads) {
            const int tok = tok0 + i / d;
            const bool in = tok < p.N;
            xs[i] = in ? ld_f32(xg, (size_t)tok0 * d + i) : 0.f;
            if (MODE != kStats1) ys[i] = in ? ld_f32(yg, (size_t)tok0 * d + i) : 0.f;
        }
        __syncthreads();

        for (int tb = warp * TOK; tb < tt; tb += kBwdWarps * TOK) {      // tokens tb .. tb + TOK - 1 of the tile
            float s[TOK][NT], dp[TOK][NT];
#pragma unroll
            for (int k = 0; k < TOK; ++k)
#pragma unroll
                for (int t = 0; t < NT; ++t) s[k][t] = dp[k][t] = 0.f;
            for (int c = 0; c < d; c += 4) {
                float4 xv[TOK], yv[TOK];
#pragma unroll
                for (int k = 0; k < TOK; ++k) {
                    xv[k] = *reinterpret_cast<const float4*>(xs + (size_t)(tb + k) * d + c);
                    if (kHasM1) yv[k] = *reinterpret_cast<const float4*>(ys + (size_t)(tb + k) * d + c);
                }
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                    for (int t = 0; t < NT; ++t)
                        if (t < nt) {
                            const float a0 = m0t[(c + cc) * np + lane + 32 * t];
                            const float a1 = kHasM1 ? m1t[(c + cc) * np + lane + 32 * t] : 0.f;
#pragma unroll
                            for (int k = 0; k < TOK; ++k) {
                                s[k][t] = fmaf(f4c(xv[k], cc), a0, s[k][t]);
                                if (kHasM1) dp[k][t] = fmaf(f4c(yv[k], cc), a1, dp[k][t]);
                            }
                        }
            }
#pragma unroll
            for (int k = 0; k < TOK; ++k) {
                const int tl = tb + k, tok = tok0 + tl;
                const bool valid = tok < p.N;
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    const int r = lane + 32 * t;
                    if (t < nt && r < n && valid) {
                        float b = 0.f;
                        if (bias)
                            b = kRowSoftmax ? ld_f32(bias, ((size_t)head * p.N + tok) * n + r)
                                            : ld_f32(bias, ((size_t)head * n + r) * p.N + tok);
                        s[k][t] = fmaf(p.scale, s[k][t], b);
                    } else {
                        s[k][t] = -INFINITY;
                    }
                }
                if (MODE == kStats1) {
#pragma unroll
                    for (int t = 0; t < NT; ++t)
                        if (s[k][t] > -INFINITY) {
                            const float m = fmaxf(run_m[t], s[k][t]);
                            run_l[t] = run_l[t] * expf(run_m[t] - m) + expf(s[k][t] - m);
                            run_m[t] = m;
                        }
                } else {
                    float prob[NT], rdot[NT];
                    if (kRowSoftmax) {
                        float m = -INFINITY;
#pragma unroll
                        for (int t = 0; t < NT; ++t) m = fmaxf(m, s[k][t]);
                        m = warp_max(m);
                        float l = 0.f;
#pragma unroll
                        for (int t = 0; t < NT; ++t) {
                            prob[t] = valid && s[k][t] > -INFINITY ? expf(s[k][t] - m) : 0.f;
                            l += prob[t];
                        }
                        l = warp_sum(l);
                        const float inv = valid ? 1.f / l : 0.f;
                        float rd = 0.f;
#pragma unroll
                        for (int t = 0; t < NT; ++t) {
                            prob[t] *= inv;
                            rd = fmaf(prob[t], dp[k][t], rd);
                        }
                        rd = warp_sum(rd);
#pragma unroll
                        for (int t = 0; t < NT; ++t) rdot[t] = rd;
                    } else {
#pragma unroll
                        for (int t = 0; t < NT; ++t) {
                            prob[t] = s[k][t] > -INFINITY ? expf(s[k][t] - lse[t]) : 0.f;
                            rdot[t] = dot[t];
                        }
                    }
#pragma unroll
                    for (int t = 0; t < NT; ++t) {
                        const int r = lane + 32 * t;
                        if (t < nt) {
                            pt[(size_t)tl * np + r] = prob[t];
                            if (kHasM1) {
                                const float g = prob[t] * (dp[k][t] - rdot[t]);
                                dst[(size_t)tl * np + r] = g;
                                if (p.dbias && valid && r < n) {
                                    float* o = kRowSoftmax ? p.dbias + ((size_t)head * p.N + tok) * n + r
                                                           : p.dbias + ((size_t)head * n + r) * p.N + tok;
                                    atomicAdd(o, g);
                                }
                            }
                        }
                    }
                }
            }
            if (kHasM1) {
                __syncwarp();
                for (int c = lane; c < d; c += 32) {
                    float a0[TOK], a1[TOK];
#pragma unroll
                    for (int k = 0; k < TOK; ++k) a0[k] = a1[k] = 0.f;
                    for (int r = 0; r < n; ++r) {
                        const float w0 = m0t[c * np + r];
                        const float w1 = MODE == kAgg1 ? m1t[c * np + r] : 0.f;
#pragma unroll
                        for (int k = 0; k < TOK; ++k) {
                            a0[k] = fmaf(dst[(size_t)(tb + k) * np + r], w0, a0[k]);
                            if (MODE == kAgg1) a1[k] = fmaf(pt[(size_t)(tb + k) * np + r], w1, a1[k]);
                        }
                    }
#pragma unroll
                    for (int k = 0; k < TOK; ++k) {
                        const int tok = tok0 + tb + k;
                        if (tok < p.N) {
                            p.row0[((size_t)slab * p.N + tok) * d + c] = p.scale * a0[k];
                            if (MODE == kAgg1) p.row1[((size_t)slab * p.N + tok) * d + c] = a1[k];
                        }
                    }
                }
            }
        }
        if (MODE != kStats1) __syncthreads();
        // sums over the tile's tokens of (per-agent weight) x (token row): thread owns (r, 4 channels)
#pragma unroll
        for (int k = 0; k < kOut; ++k) {
            const int o = tid + kBwdThreads * k;
            if (o < outer_total) {
                const int c4 = o / n, r = o - c4 * n;
                for (int tl = 0; tl < tt; ++tl) {
                    const float4 xv = *reinterpret_cast<const float4*>(xs + (size_t)tl * d + 4 * c4);
                    const float4 yv = *reinterpret_cast<const float4*>(ys + (size_t)tl * d + 4 * c4);
                    const float w = pt[(size_t)tl * np + r];
                    if (MODE == kVa1 || MODE == kBcast2) {
                        acc0[k].x = fmaf(w, yv.x, acc0[k].x); acc0[k].y = fmaf(w, yv.y, acc0[k].y);
                        acc0[k].z = fmaf(w, yv.z, acc0[k].z); acc0[k].w = fmaf(w, yv.w, acc0[k].w);
                    }
                    if (kHasM1) {
                        const float g = dst[(size_t)tl * np + r];
                        acc1[k].x = fmaf(g, xv.x, acc1[k].x); acc1[k].y = fmaf(g, xv.y, acc1[k].y);
                        acc1[k].z = fmaf(g, xv.z, acc1[k].z); acc1[k].w = fmaf(g, xv.w, acc1[k].w);
                    }
                }
            }
        }
    }

    if (MODE == kStats1) {
        // combine the warps' running states per agent, in warp order
        __syncthreads();
        float* red = pt;                                   // [warps][np][2]
#pragma unroll
        for (int t = 0; t < NT; ++t)
            if (t < nt) {
                red[((size_t)warp * np + lane + 32 * t) * 2] = run_m[t];
                red[((size_t)warp * np + lane + 32 * t) * 2 + 1] = run_l[t];
            }
        __syncthreads();
        for (int r = tid; r < n; r += kBwdThreads) {
            float m = -INFINITY, l = 0.f;
            for (int w = 0; w < kBwdWarps; ++w) {
                const float mw = red[((size_t)w * np + r) * 2], lw = red[((size_t)w * np + r) * 2 + 1];
                if (lw > 0.f) {
                    const float mm = fmaxf(m, mw);
                    l = l * expf(m - mm) + lw * expf(mw - mm);
                    m = mm;
                }
            }
            float* o = p.part + (((size_t)slab * p.chunks + chunk) * n + r) * 2;
            o[0] = m; o[1] = l;
        }
    }
#pragma unroll
    for (int k = 0; k < kOut; ++k) {
        const int o = tid + kBwdThreads * k;
        if (o < outer_total) {
            const int c4 = o / n, r = o - c4 * n;
            const size_t at = slab * nd + (size_t)r * d + 4 * c4;
            if (MODE == kVa1 || MODE == kBcast2) {
                atomicAdd(p.outer0 + at, acc0[k].x); atomicAdd(p.outer0 + at + 1, acc0[k].y);
                atomicAdd(p.outer0 + at + 2, acc0[k].z); atomicAdd(p.outer0 + at + 3, acc0[k].w);
            }
            if (kHasM1) {
                atomicAdd(p.outer1 + at, p.scale * acc1[k].x); atomicAdd(p.outer1 + at + 1, p.scale * acc1[k].y);
                atomicAdd(p.outer1 + at + 2, p.scale * acc1[k].z); atomicAdd(p.outer1 + at + 3, p.scale * acc1[k].w);
            }
        }
    }
}

// Agent tokens in fp32: mean of Q over the window of each pooled cell (text under Eq. 6).
template <typename T>
__global__ void bwd_pool_kernel(BwdArgs p, const void* qv, float* a) {
    const size_t total = (size_t)p.slabs * p.n * p.d;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int c = (int)(i % p.d);
    const int r = (int)((i / p.d) % p.n);
    const int slab = (int)(i / ((size_t)p.d * p.n));
    const int ay = r / p.pw, ax = r - ay * p.pw;
    const int y0 = (ay * p.H) / p.ph, y1 = ((ay + 1) * p.H + p.ph - 1) / p.ph;
    const int x0 = (ax * p.W) / p.pw, x1 = ((ax + 1) * p.W + p.pw - 1) / p.pw;
    const T* q = static_cast<const T*>(qv) + (size_t)slab * p.N * p.d;
    float acc = 0.f;
    for (int y = y0; y < y1; ++y)
        for (int x = x0; x < x1; ++x) acc += ld_f32(q, ((size_t)y * p.W + x) * p.d + c);
    a[i] = acc / (float)((y1 - y0) * (x1 - x0));
}

// lse[slab][r] = log sum_j exp(S1[r][j]) from the per-chunk (max, sum) pairs, in chunk order.
__global__ void bwd_lse_kernel(BwdArgs p, float* lse) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;          // slab * n + r
    if (i >= p.slabs * p.n) return;
    const int slab = i / p.n, r = i - slab * p.n;
    float m = -INFINITY, l = 0.f;
    for (int ch = 0; ch < p.chunks; ++ch) {
        const float* q = p.part + (((size_t)slab * p.chunks + ch) * p.n + r) * 2;
        if (q[1] > 0.f) {
            const float mm = fmaxf(m, q[0]);
            l = l * expf(m - mm) + q[1] * expf(q[0] - mm);
            m = mm;
        }
    }
    lse[i] = m + logf(l);
}

// dot[slab][r] = dV_A[r] . V_A[r]  (= sum_j P1[r][j] (dV_A[r] . V[j]))
__global__ void bwd_dot_kernel(BwdArgs p, const float* va, const float* dva, float* dot) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.slabs * p.n) return;
    float acc = 0.f;
    for (int c = 0; c < p.d; ++c) acc = fmaf(dva[(size_t)i * p.d + c], va[(size_t)i * p.d + c], acc);
    dot[i] = acc;
}

// Four consecutive elements of a token row as fp32.
template <typename T> __device__ __forceinline__ float4 ld4_f32(const T* p);
template <> __device__ __forceinline__ float4 ld4_f32<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <> __device__ __forceinline__ float4 ld4_f32<__nv_bfloat16>(const __nv_bfloat16* p) {
    const uint2 w = *reinterpret_cast<const uint2*>(p);
    const float2 a = unpack2<__nv_bfloat16>(w.x), b = unpack2<__nv_bfloat16>(w.y);
    return make_float4(a.x, a.y, b.x, b.y);
}
template <> __device__ __forceinline__ float4 ld4_f32<__half>(const __half* p) {
    const uint2 w = *reinterpret_cast<const uint2*>(p);
    const float2 a = unpack2<__half>(w.x), b = unpack2<__half>(w.y);
    return make_float4(a.x, a.y, b.x, b.y);
}

// Per token of the grid (the same for every slab): the pooled cells whose window contains it (at most two per
// axis; bounds as in bwd_pool_kernel), the reciprocal of each window's size, and the token's grid position.
// Three int4 per token: (count, agent0, agent1, agent2), (agent3, inv0, inv1, inv2), (inv3, y, x, -).
__global__ void bwd_window_table_kernel(BwdArgs p, int4* tab) {
    const int tok = blockIdx.x * blockDim.x + threadIdx.x;
    if (tok >= p.N) return;
    const int y = tok / p.W, x = tok - y * p.W;
    int ays[2], hy[2], axs[2], wx[2], ny = 0, nx = 0;
    const int ayc = (y * p.ph) / p.H, axc = (x * p.pw) / p.W;
    for (int ay = ayc; ay <= min(ayc + 1, p.ph - 1); ++ay) {
        const int y0 = (ay * p.H) / p.ph, y1 = ((ay + 1) * p.H + p.ph - 1) / p.ph;
        if (y >= y0 && y < y1) { ays[ny] = ay; hy[ny] = y1 - y0; ++ny; }
    }
    for (int ax = axc; ax <= min(axc + 1, p.pw - 1); ++ax) {
        const int x0 = (ax * p.W) / p.pw, x1 = ((ax + 1) * p.W + p.pw - 1) / p.pw;
        if (x >= x0 && x < x1) { axs[nx] = ax; wx[nx] = x1 - x0; ++nx; }
    }
    int agent[4] = {0, 0, 0, 0};
    float inv[4] = {0.f, 0.f, 0.f, 0.f};
    int cnt = 0;
    for (int a = 0; a < ny; ++a)
        for (int b = 0; b < nx; ++b) {
            agent[cnt] = ays[a] * p.pw + axs[b];
            inv[cnt] = 1.f / (float)(hy[a] * wx[b]);
            ++cnt;
        }
    tab[3 * tok] = make_int4(cnt, agent[0], agent[1], agent[2]);
    tab[3 * tok + 1] = make_int4(agent[3], __float_as_int(inv[0]), __float_as_int(inv[1]), __float_as_int(inv[2]));
    tab[3 * tok + 2] = make_int4(__float_as_int(inv[3]), y, x, 0);
}

// Token-wise tail, one pass over the tokens:
//   dQ  += Pooling^T(dA)   each window spreads its agent's gradient evenly over its tokens
//   dV  += DWC^T(dO)       tap (u, v) of output token (y - u + 1, x - v + 1) read V[y][x]
//   dWd += corr(dO, V)     dWd[c][u][v] = sum over tokens of dO[y - u + 1][x - v + 1][c] * V[y][x][c]
// (the last two use the same nine neighbours of dO).  Block = (slab, token chunk); thread = (token lane,
// 4 channels); the filter gradient is summed per thread, reduced per block and added with atomics.
template <typename T>
__global__ void __launch_bounds__(256) bwd_tail_kernel(BwdArgs p, const int4* tab, const float* da, const void* gov,
                                                       const void* vv, const void* wdv, float* dq, float* dv,
                                                       float* dwd, int chunks) {
    __shared__ __align__(16) float sw[9 * 128];
    __shared__ float4 red[256 * 9];
    const int slab = blockIdx.x / chunks, chunk = blockIdx.x - slab * chunks;
    const int head = slab % p.heads;
    const int d4 = p.d >> 2;
    const int lanes = 256 / d4;                                   // token lanes (d <= 128: at least 8)
    const int c4 = threadIdx.x % d4, tlane = threadIdx.x / d4, c = 4 * c4;
    const int per = (p.N + chunks - 1) / chunks;
    const int t0 = chunk * per, t1 = min(t0 + per, p.N);
    if (wdv) {
        const T* w = static_cast<const T*>(wdv) + (size_t)head * p.d * 9;
        for (int i = threadIdx.x; i < p.d * 9; i += 256) {
            const int cc = i / 9, k = i - cc * 9;
            sw[k * p.d + cc] = ld_f32(w, i);
        }
        __syncthreads();
    }
    const T* go = static_cast<const T*>(gov) + (size_t)slab * p.N * p.d + c;
    const T* v = static_cast<const T*>(vv) + (size_t)slab * p.N * p.d + c;
    float4 accw[9];
#pragma unroll
    for (int k = 0; k < 9; ++k) accw[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (tlane < lanes)
        for (int tok = t0 + tlane; tok < t1; tok += lanes) {
            const int4 e0 = tab[3 * tok], e1 = tab[3 * tok + 1], e2 = tab[3 * tok + 2];
            const int agent[4] = {e0.y, e0.z, e0.w, e1.x};
            const float inv[4] = {__int_as_float(e1.y), __int_as_float(e1.z), __int_as_float(e1.w), __int_as_float(e2.x)};
            const size_t st = (size_t)slab * p.N + tok;
            float4* qo = reinterpret_cast<float4*>(dq + st * p.d + c);
            float4 qv = *qo;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < e0.x) {
                    const float4 a = *reinterpret_cast<const float4*>(da + ((size_t)slab * p.n + agent[k]) * p.d + c);
                    qv.x = fmaf(a.x, inv[k], qv.x); qv.y = fmaf(a.y, inv[k], qv.y);
                    qv.z = fmaf(a.z, inv[k], qv.z); qv.w = fmaf(a.w, inv[k], qv.w);
                }
            *qo = qv;
            if (wdv) {
                const int y = e2.y, x = e2.z;
                float4* vo = reinterpret_cast<float4*>(dv + st * p.d + c);
                float4 acc = *vo;
                float4 vt = make_float4(0.f, 0.f, 0.f, 0.f);
                if (dwd) vt = ld4_f32<T>(v + (size_t)tok * p.d);
#pragma unroll
                for (int u = 0; u < 3; ++u)
#pragma unroll
                    for (int w = 0; w < 3; ++w) {
                        const int yo = y - u + 1, xo = x - w + 1;
                        if (yo < 0 || yo >= p.H || xo < 0 || xo >= p.W) continue;
                        const float4 gv = ld4_f32<T>(go + ((size_t)yo * p.W + xo) * p.d);
                        const float4 wv = *reinterpret_cast<const float4*>(sw + (u * 3 + w) * p.d + c);
                        acc.x = fmaf(wv.x, gv.x, acc.x); acc.y = fmaf(wv.y, gv.y, acc.y);
                        acc.z = fmaf(wv.z, gv.z, acc.z); acc.w = fmaf(wv.w, gv.w, acc.w);
                        float4& a = accw[u * 3 + w];
                        a.x = fmaf(gv.x, vt.x, a.x); a.y = fmaf(gv.y, vt.y, a.y);
                        a.z = fmaf(gv.z, vt.z, a.z); a.w = fmaf(gv.w, vt.w, a.w);
                    }
                *vo = acc;
            }
        }
    if (!dwd) return;
#pragma unroll
    for (int k = 0; k < 9; ++k) red[threadIdx.x * 9 + k] = accw[k];
    __syncthreads();
    for (int o = threadIdx.x; o < p.d * 9; o += 256) {           // o = c * 9 + tap, the layout of dWd
        const int cc = o / 9, k = o - cc * 9;
        const int q4 = cc >> 2, e = cc & 3;
        float s = 0.f;
        for (int l = 0; l < lanes; ++l) {
            const float4 t = red[(l * d4 + q4) * 9 + k];
            s += e == 0 ? t.x : e == 1 ? t.y : e == 2 ? t.z : t.w;
        }
        atomicAdd(dwd + (size_t)head * p.d * 9 + o, s);
    }
}

template <typename T, int MODE, int NT, int KOUT, int TOK>
cudaError_t launch_tile_cfg(const BwdArgs& a, cudaStream_t st) {
    const bool m1 = MODE == kBcast2 || MODE == kAgg1;
    const size_t smem = ((size_t)a.d * a.np * (m1 ? 2 : 1) + 2 * (size_t)a.tile * a.d + 2 * (size_t)a.tile * a.np) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(bwd_tile_kernel<T, MODE, NT, KOUT, TOK>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    bwd_tile_kernel<T, MODE, NT, KOUT, TOK><<<a.slabs * a.chunks, kBwdThreads, smem, st>>>(a);
    return cudaGetLastError();
}

// Three register budgets: few agents (four tokens per warp at once, two blocks per SM), up to 128 agents,
// and the general case.
template <typename T, int MODE>
cudaError_t launch_tile(const BwdArgs& a, cudaStream_t st) {
    switch (backward_variant(a.n, a.d)) {
        case 0:  return launch_tile_cfg<T, MODE, 2, 4, 4>(a, st);
        case 1:  return launch_tile_cfg<T, MODE, 4, 8, 2>(a, st);
        default: return launch_tile_cfg<T, MODE, kMaxLaneAgents, kMaxOuter, 1>(a, st);
    }
}

template <typename T>
cudaError_t backward_typed(const BwdCall& c, BwdArgs a, cudaStream_t st) {
    const size_t sn = (size_t)a.slabs * a.n, snd = sn * a.d;
    cudaError_t e;
#define AA_TRY(x) do { e = (x); if (e != cudaSuccess) return e; } while (0)
    AA_TRY(cudaMemsetAsync(c.ws_va, 0, c.clear_bytes, st));               // V_A, dV_A, dA are contiguous
    const size_t bias_elems = (size_t)a.heads * a.n * a.N;
    if (c.db1) AA_TRY(cudaMemsetAsync(c.db1, 0, bias_elems * sizeof(float), st));
    if (c.db2) AA_TRY(cudaMemsetAsync(c.db2, 0, bias_elems * sizeof(float), st));
    if (c.dwd) AA_TRY(cudaMemsetAsync(c.dwd, 0, (size_t)a.heads * a.d * 9 * sizeof(float), st));

    bwd_pool_kernel<T><<<(unsigned)((snd + 255) / 256), 256, 0, st>>>(a, c.q, c.ws_a);
    AA_TRY(cudaGetLastError());
    bwd_window_table_kernel<<<(unsigned)((a.N + 255) / 256), 256, 0, st>>>(a, c.ws_tab);
    AA_TRY(cudaGetLastError());
    // aggregation forward: row statistics, then V_A
    a.x = c.k; a.y = c.v; a.bias = c.b1; a.m0 = c.ws_a; a.m1 = nullptr; a.scale = c.scale1;
    a.part = c.ws_part; a.dbias = nullptr;
    if (c.use_mma) {
        BwdArgs m = a;
        m.np = c.plan_mma.np; m.tile = c.plan_mma.tile; m.tiles = c.plan_mma.tiles;
        m.chunks = c.plan_mma.chunks; m.tiles_per_chunk = c.plan_mma.tiles_per_chunk;
        AA_TRY(launch_backward_fwd1_mma(c.dtype, m, c.ws_va, c.ws_lse, st));
        a.lse = c.ws_lse;
    } else {
        AA_TRY((launch_tile<T, kStats1>(a, st)));
        bwd_lse_kernel<<<(unsigned)((sn + 255) / 256), 256, 0, st>>>(a, c.ws_lse);
        AA_TRY(cudaGetLastError());
        a.lse = c.ws_lse; a.outer0 = c.ws_va;
        AA_TRY((launch_tile<T, kVa1>(a, st)));
    }
    // broadcast backward
    a.x = c.q; a.y = c.d_out; a.bias = c.b2; a.m0 = c.ws_a; a.m1 = c.ws_va; a.scale = c.scale2;
    a.outer0 = c.ws_dva; a.outer1 = c.ws_da; a.row0 = c.dq; a.row1 = nullptr; a.dbias = c.db2;
    if (c.use_mma) {
        BwdArgs m = a;
        m.np = c.plan_mma.np; m.tile = c.plan_mma.tile; m.tiles = c.plan_mma.tiles;
        m.chunks = c.plan_mma.chunks; m.tiles_per_chunk = c.plan_mma.tiles_per_chunk;
        AA_TRY(launch_backward_mma(c.dtype, true, m, st));
    } else {
        AA_TRY((launch_tile<T, kBcast2>(a, st)));
    }
    bwd_dot_kernel<<<(unsigned)((sn + 255) / 256), 256, 0, st>>>(a, c.ws_va, c.ws_dva, c.ws_dot);
    AA_TRY(cudaGetLastError());
    // aggregation backward
    a.x = c.k; a.y = c.v; a.bias = c.b1; a.m0 = c.ws_a; a.m1 = c.ws_dva; a.scale = c.scale1;
    a.lse = c.ws_lse; a.dot = c.ws_dot;
    a.outer0 = nullptr; a.outer1 = c.ws_da; a.row0 = c.dk; a.row1 = c.dv; a.dbias = c.db1;
    if (c.use_mma) {
        BwdArgs m = a;
        m.np = c.plan_mma.np; m.tile = c.plan_mma.tile; m.tiles = c.plan_mma.tiles;
        m.chunks = c.plan_mma.chunks; m.tiles_per_chunk = c.plan_mma.tiles_per_chunk;
        AA_TRY(launch_backward_mma(c.dtype, false, m, st));
    } else {
        AA_TRY((launch_tile<T, kAgg1>(a, st)));
    }
    // pooling and depthwise terms
    {
        int chunks = (4 * c.sm_count + a.slabs - 1) / a.slabs;          // short loops (they are load-latency bound), few atomics
        chunks = max(1, min(chunks, (a.N + 63) / 64));
        bwd_tail_kernel<T><<<a.slabs * chunks, 256, 0, st>>>(a, c.ws_tab, c.ws_da, c.d_out, c.v, c.wd, c.dq, c.dv, c.dwd,
                                                              chunks);
        AA_TRY(cudaGetLastError());
    }
#undef AA_TRY
    return cudaSuccess;
}

}  // namespace

// Shared-memory need of the widest tile kernel for `tile` tokens per tile.
static size_t bwd_smem_bytes(int n, int d, int tile) {
    const int np = (n + 31) / 32 * 32 + 1;
    return ((size_t)d * np * 2 + 2 * (size_t)tile * d + 2 * (size_t)tile * np) * sizeof(float);
}

bool plan_backward(int slabs, int n, int N, int d, int sm_count, BwdPlan* out) {
    if (n > 32 * kMaxLaneAgents || (size_t)n * d > (size_t)4 * kMaxOuter * kBwdThreads || d % 4) return false;
    if (slabs > 65535 || d > 128) return false;                 // the token-wise tail indexes slabs with gridDim.y
    int tile = 32;
    while (tile >= 8 && bwd_smem_bytes(n, d, tile) > 227u * 1024u) tile >>= 1;
    if (tile < 8) return false;
    BwdPlan pl;
    pl.tile = tile;
    pl.np = (n + 31) / 32 * 32 + 1;
    pl.tiles = (N + tile - 1) / tile;
    // one wave of blocks where the slabs allow it: two blocks per SM fit for few agents, else one
    const int slots = sm_count * (backward_variant(n, d) == 0 ? 2 : 1);
    int chunks = slots >= slabs ? slots / slabs : 1;
    chunks = max(1, min(chunks, pl.tiles));
    pl.tiles_per_chunk = (pl.tiles + chunks - 1) / chunks;
    pl.chunks = (pl.tiles + pl.tiles_per_chunk - 1) / pl.tiles_per_chunk;
    *out = pl;
    return true;
}

int backward_launch_count(bool use_mma) { return use_mma ? 8 : 9; }

cudaError_t launch_backward(int dtype, const BwdCall& c, cudaStream_t st) {
    BwdArgs a;
    memset(&a, 0, sizeof(a));
    a.slabs = c.slabs; a.heads = c.heads; a.N = c.H * c.W; a.H = c.H; a.W = c.W; a.d = c.d; a.n = c.n;
    a.ph = c.p; a.pw = c.p;
    a.np = c.plan.np; a.tile = c.plan.tile; a.tiles = c.plan.tiles;
    a.chunks = c.plan.chunks; a.tiles_per_chunk = c.plan.tiles_per_chunk;
    switch (dtype) {
        case kF32:  return backward_typed<float>(c, a, st);
        case kBF16: return backward_typed<__nv_bfloat16>(c, a, st);
        case kF16:  return backward_typed<__half>(c, a, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace aa
