// Dense agent bias from its three components (App. B): B = (B'_c + B'_r + B'_b).reshape(n, N), with
// the column bias repeated over rows, the row bias repeated over columns and the block bias resized
// to the token grid by bilinear interpolation (half-pixel centres, edge clamp).  One thread per
// output element; fp32 arithmetic, one rounding to the storage type.
#include "common.cuh"
#include "kernels.h"

namespace aa {

template <typename T>
__global__ void __launch_bounds__(256) compose_bias_kernel(ComposeArgs p) {
    const int N = p.h * p.w;
    const long long total = (long long)p.heads * p.n * N;
    const long long e = (long long)blockIdx.x * 256 + threadIdx.x;
    if (e >= total) return;
    // enumerate outputs in the order they are stored, so that stores coalesce
    int head, a, t;
    if (p.transpose) { head = (int)(e / ((long long)N * p.n)); const int r = (int)(e - (long long)head * N * p.n); t = r / p.n; a = r - t * p.n; }
    else             { head = (int)(e / ((long long)p.n * N)); const int r = (int)(e - (long long)head * p.n * N); a = r / N; t = r - a * N; }
    const int y = t / p.w, x = t - y * p.w;
    const size_t ha = (size_t)head * p.n + a;
    float v = 0.f;
    if (p.col) v += Elem<T>::to_f32(static_cast<const T*>(p.col)[ha * p.w + x]);
    if (p.row) v += Elem<T>::to_f32(static_cast<const T*>(p.row)[ha * p.h + y]);
    if (p.blk) {
        float sy = fmaxf(0.f, ((float)y + 0.5f) * (float)p.h0 / (float)p.h - 0.5f);
        float sx = fmaxf(0.f, ((float)x + 0.5f) * (float)p.w0 / (float)p.w - 0.5f);
        int y0 = min((int)sy, p.h0 - 1), x0 = min((int)sx, p.w0 - 1);
        const int y1 = y0 < p.h0 - 1 ? y0 + 1 : y0, x1 = x0 < p.w0 - 1 ? x0 + 1 : x0;
        const float ly = fminf(sy - (float)y0, 1.f), lx = fminf(sx - (float)x0, 1.f);
        const T* b = static_cast<const T*>(p.blk) + ha * p.h0 * p.w0;
        const float b00 = Elem<T>::to_f32(b[y0 * p.w0 + x0]), b01 = Elem<T>::to_f32(b[y0 * p.w0 + x1]);
        const float b10 = Elem<T>::to_f32(b[y1 * p.w0 + x0]), b11 = Elem<T>::to_f32(b[y1 * p.w0 + x1]);
        v += (1.f - ly) * ((1.f - lx) * b00 + lx * b01) + ly * ((1.f - lx) * b10 + lx * b11);
    }
    static_cast<T*>(p.out)[e] = Elem<T>::from_f32(v);
}

cudaError_t launch_compose_bias(int dtype, const ComposeArgs& p, cudaStream_t st) {
    const long long total = (long long)p.heads * p.n * p.h * p.w;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    switch (dtype) {
        case kF32:  compose_bias_kernel<float><<<blocks, 256, 0, st>>>(p); break;
        case kBF16: compose_bias_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(p); break;
        case kF16:  compose_bias_kernel<__half><<<blocks, 256, 0, st>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace aa
