// Agent tokens by average pooling of Q over the token grid (text under Eq. 6: A = Pooling(Q)).
//
// One warp owns one pooled cell of one slab.  Its lanes are laid out as (token sub-lane, 16-byte
// channel chunk), so a warp-wide load covers whole contiguous token rows of the window; sums are
// kept in fp32 and reduced across the token sub-lanes in a fixed order (no atomics: results are
// bit-reproducible).
#include "common.cuh"
#include "kernels.h"

namespace aa {

template <typename T>
__global__ void __launch_bounds__(256) pool_kernel(PoolArgs p) {
    constexpr int VEC = Elem<T>::kVec;
    __shared__ float s_red[8][32][VEC];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = p.ph * p.pw;
    const long long cell = (long long)blockIdx.x * 8 + warp;       // slab * n + agent
    if (cell >= (long long)p.slabs * n) return;
    const int slab = (int)(cell / n), a = (int)(cell - (long long)slab * n);
    const int ay = a / p.pw, ax = a - ay * p.pw;
    const int y0 = (ay * p.H) / p.ph, y1 = ((ay + 1) * p.H + p.ph - 1) / p.ph;
    const int x0 = (ax * p.W) / p.pw, x1 = ((ax + 1) * p.W + p.pw - 1) / p.pw;
    const int ww = x1 - x0, cnt = (y1 - y0) * ww;
    const int cpt = p.d / VEC;                    // 16-byte chunks per token
    const int tpl = 32 / cpt;                     // tokens covered by one warp-wide load
    const int cg = lane % cpt, tsub = lane / cpt;
    const T* q = static_cast<const T*>(p.q) + tok_offset(p.lq, slab, p.heads, 0);

    float acc[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[k] = 0.f;
    if (tsub < tpl) {
#pragma unroll 4
        for (int i = tsub; i < cnt; i += tpl) {
            const int wy = i / ww, wx = i - wy * ww;
            const size_t tok = (size_t)(y0 + wy) * p.W + (x0 + wx);
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(q + tok * (size_t)p.lq.st) + cg);
            float f[VEC];
            unpack16<T>(raw, f);
#pragma unroll
            for (int k = 0; k < VEC; ++k) acc[k] += f[k];
        }
    }
#pragma unroll
    for (int k = 0; k < VEC; ++k) s_red[warp][lane][k] = acc[k];
    __syncwarp();
    const float inv = 1.f / (float)cnt;
    T* out = static_cast<T*>(p.a) + (size_t)cell * p.d;
    for (int c = lane; c < p.d; c += 32) {
        const int g = c / VEC, k = c - g * VEC;
        float s = 0.f;
        for (int t = 0; t < tpl; ++t) s += s_red[warp][t * cpt + g][k];
        out[c] = Elem<T>::from_f32(s * inv);
    }
}

cudaError_t launch_pool(int dtype, const PoolArgs& p, cudaStream_t st) {
    const long long cells = (long long)p.slabs * p.ph * p.pw;
    const unsigned blocks = (unsigned)((cells + 7) / 8);
    switch (dtype) {
        case kF32:  pool_kernel<float><<<blocks, 256, 0, st>>>(p); break;
        case kBF16: pool_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(p); break;
        case kF16:  pool_kernel<__half><<<blocks, 256, 0, st>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace aa
