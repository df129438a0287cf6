// Agent broadcast O = softmax(scale2 * Q A^T + B2) V_A (Eq. 3, Eq. 5) on tensor cores, with the
// depthwise 3x3 term DWC(V) of Eq. 6 added in the epilogue so that O is written exactly once.
//
// Grid: (query tiles of 128 tokens, slabs).  The slab's agents A and agent features V_A stay
// resident in shared memory; each of the 8 warps owns 16 query rows, computes their logits
// against all agents in chunks of 64 (online softmax over the chunks, row statistics by quad
// shuffles), multiplies by V_A, then re-maps its 16 x d result through a private shared-memory
// patch to (token, 8-channel) items for the stencil and a 16-byte coalesced store.
#include "common.cuh"
#include "kernels.h"

namespace aa {

namespace {
constexpr int QT = 128;                      // queries per block
constexpr int AC = 64;                       // agents per chunk
__host__ __device__ inline int dk_of2(int d) { return d <= 32 ? 32 : d <= 48 ? 48 : d <= 64 ? 64 : 128; }
}  // namespace

template <typename T, int DK>
__global__ void __launch_bounds__(256) broadcast_mma_kernel(AttnArgs p, int n_pad) {
    constexpr int PA = DK + 8;                // pitch (elements) of A, V_A and Q rows
    constexpr int PO = DK + 8;                // pitch (floats) of the per-warp output patch
    extern __shared__ __align__(16) unsigned char smem_raw[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.y, head = slab % p.heads;
    const int N = p.rows, n = p.cols, d = p.d;
    const int i0 = blockIdx.x * QT + warp * 16;          // first query row of this warp

    T* sA = reinterpret_cast<T*>(smem_raw);                       // [n_pad][PA]
    T* sVA = sA + (size_t)n_pad * PA;                              // [n_pad][PA]
    float* sW = reinterpret_cast<float*>(sVA + (size_t)n_pad * PA);   // [9][DK] filter taps
    float* sPatch = sW + 9 * DK + (size_t)warp * 16 * PO;          // [16][PO] per warp
    T* sQ = reinterpret_cast<T*>(sPatch);                          // [16][PA], aliases the patch

    {   // zero everything once (pad rows / pad columns must be finite zeros)
        const size_t total16 = ((size_t)2 * n_pad * PA * 2 + (9 * DK + (size_t)8 * 16 * PO) * 4) / 16;
        uint4* z = reinterpret_cast<uint4*>(smem_raw);
        for (size_t i = tid; i < total16; i += 256) z[i] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();

    const int cpr = d / 8;
    const T* gA = static_cast<const T*>(p.km) + (size_t)slab * n * d;
    const T* gVA = static_cast<const T*>(p.vm) + (size_t)slab * n * d;
    const T* gQ = static_cast<const T*>(p.qm) + (size_t)slab * N * d;
    for (int e = tid; e < n * cpr; e += 256) {
        const int r = e / cpr, c = e - r * cpr;
        cp_async16(sA + r * PA + c * 8, gA + (size_t)r * d + c * 8, 16);
        cp_async16(sVA + r * PA + c * 8, gVA + (size_t)r * d + c * 8, 16);
    }
    for (int e = lane; e < 16 * cpr; e += 32) {
        const int r = e / cpr, c = e - r * cpr;
        const bool ok = (i0 + r) < N;
        cp_async16(sQ + r * PA + c * 8, gQ + (ok ? ((size_t)(i0 + r) * d + c * 8) : 0), ok ? 16 : 0);
    }
    cp_async_commit();
    const bool has_dwc = p.dwc_w != nullptr;
    if (has_dwc) {
        const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * d * 9;
        for (int e = tid; e < 9 * d; e += 256) {
            const int c = e / 9, tap = e - c * 9;
            sW[tap * DK + c] = Elem<T>::to_f32(w[e]);
        }
    }
    cp_async_wait<0>();
    __syncthreads();

    const int g = lane >> 2, t4 = lane & 3;
    uint32_t qf[DK / 16][4];
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks)
        ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3],
                    sQ + ((lane & 7) + ((lane >> 3) & 1) * 8) * PA + ks * 16 + (lane >> 4) * 8);
    __syncwarp();                              // Q rows are in registers; the patch may be reused

    const float scale_log2 = p.scale * kLog2e;
    const T* gB = p.bias ? static_cast<const T*>(p.bias) + (size_t)head * N * n : nullptr;
    const int row_a = i0 + g, row_b = i0 + g + 8;

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float acc[DK / 8][4];
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) { acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f; }

    for (int a0 = 0; a0 < n_pad; a0 += AC) {
        if (a0 >= n) break;
        float sc[AC / 8][4];
#pragma unroll
        for (int j = 0; j < AC / 8; ++j) { sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < DK / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < AC / 16; ++np) {
                if (a0 + np * 16 < n_pad) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(b0, b1, b2, b3,
                                sA + (a0 + np * 16 + (lane & 7) + (lane >> 4) * 8) * PA + ks * 16 + ((lane >> 3) & 1) * 8);
                    mma16816<T>(sc[2 * np], qf[ks], b0, b1);
                    mma16816<T>(sc[2 * np + 1], qf[ks], b2, b3);
                }
            }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int j = 0; j < AC / 8; ++j) {
            const int col = a0 + 8 * j + 2 * t4;
            const bool ok0 = col < n, ok1 = (col + 1) < n;
            float b00 = 0.f, b01 = 0.f, b10 = 0.f, b11 = 0.f;
            if (gB) {
                if (row_a < N) {
                    if (ok0) b00 = Elem<T>::to_f32(__ldg(gB + (size_t)row_a * n + col)) * kLog2e;
                    if (ok1) b01 = Elem<T>::to_f32(__ldg(gB + (size_t)row_a * n + col + 1)) * kLog2e;
                }
                if (row_b < N) {
                    if (ok0) b10 = Elem<T>::to_f32(__ldg(gB + (size_t)row_b * n + col)) * kLog2e;
                    if (ok1) b11 = Elem<T>::to_f32(__ldg(gB + (size_t)row_b * n + col + 1)) * kLog2e;
                }
            }
            sc[j][0] = ok0 ? fmaf(sc[j][0], scale_log2, b00) : -INFINITY;
            sc[j][1] = ok1 ? fmaf(sc[j][1], scale_log2, b01) : -INFINITY;
            sc[j][2] = ok0 ? fmaf(sc[j][2], scale_log2, b10) : -INFINITY;
            sc[j][3] = ok1 ? fmaf(sc[j][3], scale_log2, b11) : -INFINITY;
            mx0 = fmaxf(mx0, fmaxf(sc[j][0], sc[j][1]));
            mx1 = fmaxf(mx1, fmaxf(sc[j][2], sc[j][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);      // finite: every chunk has an agent
        const float corr0 = fast_exp2(m0 - mn0), corr1 = fast_exp2(m1 - mn1);
        m0 = mn0; m1 = mn1;
        l0 *= corr0; l1 *= corr1;
#pragma unroll
        for (int j = 0; j < DK / 8; ++j) {
            acc[j][0] *= corr0; acc[j][1] *= corr0; acc[j][2] *= corr1; acc[j][3] *= corr1;
        }
        uint32_t pk[AC / 8][2];
#pragma unroll
        for (int j = 0; j < AC / 8; ++j) {
            pk[j][0] = pack2<T>(fast_exp2(sc[j][0] - mn0), fast_exp2(sc[j][1] - mn0));
            pk[j][1] = pack2<T>(fast_exp2(sc[j][2] - mn1), fast_exp2(sc[j][3] - mn1));
            const float2 q0 = unpack2<T>(pk[j][0]), q1 = unpack2<T>(pk[j][1]);
            l0 += q0.x + q0.y;
            l1 += q1.x + q1.y;
        }
#pragma unroll
        for (int kk = 0; kk < AC / 16; ++kk) {
            if (a0 + kk * 16 < n_pad) {
                const uint32_t pa[4] = {pk[2 * kk][0], pk[2 * kk][1], pk[2 * kk + 1][0], pk[2 * kk + 1][1]};
#pragma unroll
                for (int np = 0; np < DK / 16; ++np) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(b0, b1, b2, b3,
                                      sVA + (a0 + kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PA + np * 16 + (lane >> 4) * 8);
                    mma16816<T>(acc[2 * np], pa, b0, b1);
                    mma16816<T>(acc[2 * np + 1], pa, b2, b3);
                }
            }
        }
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float inv0 = 1.f / l0, inv1 = 1.f / l1;

    // re-map the warp's 16 x d result through its patch
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) {
        const int col = 8 * j + 2 * t4;
        *reinterpret_cast<float2*>(sPatch + g * PO + col) = make_float2(acc[j][0] * inv0, acc[j][1] * inv0);
        *reinterpret_cast<float2*>(sPatch + (g + 8) * PO + col) = make_float2(acc[j][2] * inv1, acc[j][3] * inv1);
    }
    __syncwarp();

    const T* gV = has_dwc ? static_cast<const T*>(p.dwc_v) + (size_t)slab * N * d : nullptr;
    T* gO = static_cast<T*>(p.out) + (size_t)slab * N * d;
    const int H = p.H, W = p.W;
    for (int item = lane; item < 16 * cpr; item += 32) {
        const int r = item / cpr, ch = item - r * cpr;
        const int tok = i0 + r;
        if (tok >= N) continue;
        float o[8];
        {
            const float4 x0 = *reinterpret_cast<const float4*>(sPatch + r * PO + ch * 8);
            const float4 x1 = *reinterpret_cast<const float4*>(sPatch + r * PO + ch * 8 + 4);
            o[0] = x0.x; o[1] = x0.y; o[2] = x0.z; o[3] = x0.w;
            o[4] = x1.x; o[5] = x1.y; o[6] = x1.z; o[7] = x1.w;
        }
        if (has_dwc) {   // depthwise 3x3 cross-correlation with zero padding (Eq. 6)
            const int y = tok / W, x = tok - y * W;
#pragma unroll
            for (int u = 0; u < 3; ++u) {
                const int yy = y + u - 1;
                if (yy < 0 || yy >= H) continue;
#pragma unroll
                for (int v = 0; v < 3; ++v) {
                    const int xx = x + v - 1;
                    if (xx < 0 || xx >= W) continue;
                    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(gV + (size_t)(yy * W + xx) * d) + ch);
                    float f[8];
                    unpack16<T>(raw, f);
                    const float4 w0 = *reinterpret_cast<const float4*>(sW + (u * 3 + v) * DK + ch * 8);
                    const float4 w1 = *reinterpret_cast<const float4*>(sW + (u * 3 + v) * DK + ch * 8 + 4);
                    o[0] = fmaf(w0.x, f[0], o[0]); o[1] = fmaf(w0.y, f[1], o[1]);
                    o[2] = fmaf(w0.z, f[2], o[2]); o[3] = fmaf(w0.w, f[3], o[3]);
                    o[4] = fmaf(w1.x, f[4], o[4]); o[5] = fmaf(w1.y, f[5], o[5]);
                    o[6] = fmaf(w1.z, f[6], o[6]); o[7] = fmaf(w1.w, f[7], o[7]);
                }
            }
        }
        *(reinterpret_cast<uint4*>(gO + (size_t)tok * d) + ch) = pack16<T>(o);
    }
}

template <typename T, int DK>
static cudaError_t launch_bc(const AttnArgs& p, cudaStream_t st) {
    const int n_pad = (p.cols + 15) / 16 * 16;
    const size_t smem = (size_t)2 * n_pad * (DK + 8) * 2 + (9 * DK + (size_t)8 * 16 * (DK + 8)) * 4;
    auto kern = broadcast_mma_kernel<T, DK>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((p.rows + QT - 1) / QT, p.slabs);
    kern<<<grid, 256, smem, st>>>(p, n_pad);
    return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_bc_t(const AttnArgs& p, cudaStream_t st) {
    switch (dk_of2(p.d)) {
        case 32:  return launch_bc<T, 32>(p, st);
        case 48:  return launch_bc<T, 48>(p, st);
        case 64:  return launch_bc<T, 64>(p, st);
        case 128: return launch_bc<T, 128>(p, st);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_broadcast_mma(int dtype, const AttnArgs& p, cudaStream_t st) {
    if (dtype == kBF16) return launch_bc_t<__nv_bfloat16>(p, st);
    if (dtype == kF16)  return launch_bc_t<__half>(p, st);
    return cudaErrorInvalidValue;
}

}  // namespace aa
