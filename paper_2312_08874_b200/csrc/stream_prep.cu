// First kernel of the streaming path for small agent counts: everything the two attention kernels need
// besides Q, K and V themselves.
//   * agents A = Pooling(Q) (text under Eq. 6): one warp per (slab, agent) window, 16-byte loads with eight in
//     flight per lane, fp32 sums in a fixed order; written as A and as scale1 * A, scale2 * A (each rounded
//     once from the fp32 mean), the operands of the logit products of Eq. 3.  A caller's agents are only scaled.
//   * agent biases (Eq. 5): B1 clamped to +-30000, transposed to [N][64] (pad columns zero); B2 clamped and
//     padded to 64 columns with -60000.  The attention kernels add the bias inside the
//     tensor-core contraction (a product with an identity block), where an infinite entry would turn 0 * inf into NaN for every other agent; and the pad
//     columns make the agents past n drop out of the broadcast softmax without any masking instructions.
//   * the depthwise filter as diagonal operand slices: the broadcast kernel evaluates the 3x3 term on the tensor
//     core as nine products of a shifted V tile with diag(w[:, tap]).
//   * the arrival counters of the aggregation are cleared.
#include "stream_common.cuh"

namespace aa {

namespace {
constexpr int NT = 256;

template <typename T>
__global__ void __launch_bounds__(NT, 4) stream_prep_kernel(const StreamArgs p, int bias_blocks) {
    pdl_launch_dependents();          // the aggregation kernel may set itself up while this one runs
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = p.H * p.W, n = p.n;
    if (blockIdx.x == 0)
        for (int e = tid; e < p.slabs; e += NT) p.tickets[e] = 0u;
    // the bias blocks come first in the grid: they are few, latency-bound, and would otherwise form the kernel's tail
    if ((int)blockIdx.x >= bias_blocks) {
        const long long wi = (long long)(blockIdx.x - bias_blocks) * (NT / 32) + warp;
        if (wi >= (long long)p.slabs * n) return;
        const int slab = (int)(wi / n), a = (int)(wi - (long long)slab * n);
        const int c = lane & 7, ts = lane >> 3;
        float acc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;
        float inv = 1.f;
        if (p.a_user) {
            if (ts == 0) unpack16<T>(__ldg(reinterpret_cast<const uint4*>(static_cast<const T*>(p.a_user) + ((size_t)slab * n + a) * 64) + c), acc);
        } else {
            const int win_h = p.H / p.p, win_w = p.W / p.p, cnt = win_h * win_w;
            const int y0 = (a / p.p) * win_h, x0 = (a % p.p) * win_w;
            // lane (c, ts) walks the window's tokens ts, ts + 4, ... in row-major order; (wy, wx) is kept
            // incrementally, so the loads of a batch cost an add and a compare each
            const uint4* gq = reinterpret_cast<const uint4*>(static_cast<const T*>(p.q) + ((size_t)slab * N + (size_t)y0 * p.W + x0) * 64) + c;
            inv = 1.f / (float)cnt;
            int wy = ts / win_w, wx = ts - wy * win_w;
            float2 acc2[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) acc2[k] = make_float2(0.f, 0.f);
            for (int ib = ts; ib < cnt; ib += 32) {          // eight loads in flight per lane, four blocks per SM
                uint4 raw[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    raw[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (ib + 4 * u < cnt) raw[u] = __ldg(gq + ((size_t)wy * p.W + wx) * 8);
                    wx += 4;
                    while (wx >= win_w) { wx -= win_w; ++wy; }
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    acc2[0] = fadd2(acc2[0], unpack2<T>(raw[u].x));
                    acc2[1] = fadd2(acc2[1], unpack2<T>(raw[u].y));
                    acc2[2] = fadd2(acc2[2], unpack2<T>(raw[u].z));
                    acc2[3] = fadd2(acc2[3], unpack2<T>(raw[u].w));
                }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) { acc[2 * k] = acc2[k].x; acc[2 * k + 1] = acc2[k].y; }
        }
#pragma unroll
        for (int o = 8; o < 32; o <<= 1) {
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], o);
        }
        if (ts == 0) {
            float m[8], s1[8], s2[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) { m[k] = acc[k] * inv; s1[k] = m[k] * p.scale1; s2[k] = m[k] * p.scale2; }
            const size_t off = ((size_t)slab * n + a) * 64;
            if (!p.a_user) *(reinterpret_cast<uint4*>(static_cast<T*>(p.a_ws) + off) + c) = pack16<T>(m);
            *(reinterpret_cast<uint4*>(static_cast<T*>(p.a1s) + off) + c) = pack16<T>(s1);
            *(reinterpret_cast<uint4*>(static_cast<T*>(p.a2s) + off) + c) = pack16<T>(s2);
        }
        return;
    }
    // ---- bias blocks
    const long long t0 = (long long)blockIdx.x * NT + tid, step = (long long)bias_blocks * NT;
    if (p.b1) {
        // B1 [heads][n][N] -> transposed, padded [heads][N][64] (pad columns zero): a K-major operand tile per 128 tokens
        const long long vecs = (long long)p.heads * N * 8;
        const T* src = static_cast<const T*>(p.b1);
        uint4* dst = static_cast<uint4*>(p.b1c);
        for (long long e = t0; e < vecs; e += step) {
            const long long rowi = e >> 3;                                 // head * N + token
            const int head = (int)(rowi / N), tok = (int)(rowi - (long long)head * N);
            const int c0 = (int)(e & 7) * 8;
            float f[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int col = c0 + k;
                f[k] = col < n ? fminf(fmaxf(Elem<T>::to_f32(src[((size_t)head * n + col) * N + tok]), -Pair<T>::kBig), Pair<T>::kBig) : 0.f;
            }
            dst[e] = pack16<T>(f);
        }
    }
    if (p.dwc_w) {
        // depthwise filter -> per tap a [16][64] K-major operand tile (128-byte rows, 128-byte swizzle) holding four
        // diagonal 16 x 16 slices: row j, column 16 g + k is w[16 g + j][tap] where j == k, else 0
        const long long elems = (long long)p.heads * 9 * 16 * 64;
        const T* src = static_cast<const T*>(p.dwc_w);
        unsigned char* dst = static_cast<unsigned char*>(p.wt);
        for (long long e = t0; e < elems; e += step) {
            const int col = (int)(e & 63), j = (int)((e >> 6) & 15);
            const int ht = (int)(e >> 10), head = ht / 9, tap = ht - head * 9;
            const int g = col >> 4, k = col & 15;
            const T v = (j == k) ? src[((size_t)head * 64 + 16 * g + j) * 9 + tap] : Elem<T>::from_f32(0.f);
            *reinterpret_cast<T*>(dst + (size_t)ht * 2048 + j * 128 + ((((col >> 3) ^ j) & 7) << 4) + (col & 7) * 2) = v;
        }
    }
    {
        const int hb = p.b2 ? p.heads : 1;
        const long long vecs = (long long)hb * N * 8;
        const T* src = static_cast<const T*>(p.b2);
        uint4* dst = static_cast<uint4*>(p.b2p);
        for (long long e = t0; e < vecs; e += step) {
            const long long rowi = e >> 3;                                 // head * N + token
            const int c0 = (int)(e & 7) * 8;
            float f[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int col = c0 + k;
                float v = -Pair<T>::kPad;
                if (col < n) v = src ? fminf(fmaxf(Elem<T>::to_f32(src[rowi * n + col]), -Pair<T>::kBig), Pair<T>::kBig) : 0.f;
                f[k] = v;
            }
            dst[e] = pack16<T>(f);
        }
    }
}
}  // namespace

cudaError_t launch_stream_prep(int dtype, const StreamArgs& a, cudaStream_t st) {
    const long long windows = (long long)a.slabs * a.n;
    const int pool_blocks = (int)((windows + NT / 32 - 1) / (NT / 32));
    const long long N = (long long)a.H * a.W;
    const long long items = (a.b1 ? (long long)a.heads * N * 8 : 0) + (long long)(a.b2 ? a.heads : 1) * N * 8;
    long long bias_blocks = (items + NT - 1) / NT;            // one output vector per thread where the grid allows it
    if (bias_blocks > 8LL * a.sm_count) bias_blocks = 8LL * a.sm_count;
    if (bias_blocks < 1) bias_blocks = 1;
    const unsigned grid = (unsigned)(pool_blocks + bias_blocks);
    if (dtype == kBF16) stream_prep_kernel<__nv_bfloat16><<<grid, NT, 0, st>>>(a, (int)bias_blocks);
    else if (dtype == kF16) stream_prep_kernel<__half><<<grid, NT, 0, st>>>(a, (int)bias_blocks);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace aa
