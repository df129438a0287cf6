// fp32 FMA kernels for both Softmax attentions of Eq. 3 (any element type, fp32 arithmetic).
//
// This is the path of the fp32 configuration (no tensor-core rounding is acceptable at its
// 1e-4 tolerance) and a cross-check path for the 16-bit types.  One block owns 64 rows of the
// attention (agents in the aggregation, tokens in the broadcast) and walks its columns in tiles
// of 32 with an online softmax; the accumulator lives in registers.
#include "common.cuh"
#include "kernels.h"
#include "merge.cuh"

namespace aa {

namespace {
constexpr int RB = 64;     // rows per block
constexpr int CT = 32;     // columns per tile
constexpr int NT = 256;    // threads
constexpr int MAXACC = RB * 128 / NT;   // accumulator registers per thread at d = 128

inline size_t simt_smem_floats(int d) {
    return (size_t)RB * (d + 1) + (size_t)CT * (d + 1) + (size_t)CT * d + (size_t)RB * (CT + 1)
           + 3 * RB + 9 * (size_t)d;
}
}  // namespace

template <typename T, bool SPLIT>
__global__ void __launch_bounds__(NT) attn_simt_kernel(AttnArgs p, int rows_pad) {
    extern __shared__ float smem[];
    __shared__ int s_flag;
    const int d = p.d, dp = d + 1;
    float* sQ = smem;                       // [RB][dp]
    float* sK = sQ + RB * dp;               // [CT][dp]
    float* sV = sK + CT * dp;               // [CT][d]
    float* sS = sV + CT * d;                // [RB][CT+1]
    float* sCorr = sS + RB * (CT + 1);      // [RB]
    float* sM = sCorr + RB;                 // [RB]
    float* sL = sM + RB;                    // [RB]
    float* sW = sL + RB;                    // [9][d] depthwise filter taps (broadcast only)

    const int tid = threadIdx.x;
    const int rb = blockIdx.x, split = blockIdx.y, slab = blockIdx.z;
    const int head = slab % p.heads;
    const int row0 = rb * RB;
    const T* qm = static_cast<const T*>(p.qm) + ((size_t)slab * p.rows) * d;
    const T* km = static_cast<const T*>(p.km) + ((size_t)slab * p.cols) * d;
    const T* vm = static_cast<const T*>(p.vm) + ((size_t)slab * p.cols) * d;
    const T* bias = p.bias ? static_cast<const T*>(p.bias) + (size_t)head * p.rows * p.cols : nullptr;

    for (int e = tid; e < RB * d; e += NT) {
        const int r = e / d, c = e - r * d;
        sQ[r * dp + c] = (row0 + r < p.rows) ? Elem<T>::to_f32(qm[(size_t)(row0 + r) * d + c]) : 0.f;
    }
    if (tid < RB) { sM[tid] = -INFINITY; sL[tid] = 0.f; }
    if (!SPLIT && p.dwc_w) {
        const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * d * 9;
        for (int e = tid; e < 9 * d; e += NT) {
            const int c = e / 9, tap = e - c * 9;
            sW[tap * d + c] = Elem<T>::to_f32(w[e]);
        }
    }

    const int tiles = (p.cols + CT - 1) / CT;
    const int nsplit = SPLIT ? p.splits : 1;
    const int tps = (tiles + nsplit - 1) / nsplit;
    const int t0 = split * tps, t1 = min(tiles, t0 + tps);
    const int nacc = (RB * d + NT - 1) / NT;

    float acc[MAXACC];
#pragma unroll
    for (int i = 0; i < MAXACC; ++i) acc[i] = 0.f;

    for (int t = t0; t < t1; ++t) {
        const int c0 = t * CT;
        __syncthreads();
        for (int e = tid; e < CT * d; e += NT) {
            const int j = e / d, c = e - j * d;
            const bool ok = (c0 + j) < p.cols;
            sK[j * dp + c] = ok ? Elem<T>::to_f32(km[(size_t)(c0 + j) * d + c]) : 0.f;
            sV[j * d + c]  = ok ? Elem<T>::to_f32(vm[(size_t)(c0 + j) * d + c]) : 0.f;
        }
        __syncthreads();
        {   // logits in log2 units: (scale * q.k + bias) * log2(e)
            const int j = tid & 31, col = c0 + j;
#pragma unroll 1
            for (int i = 0; i < RB / 8; ++i) {
                const int r = (tid >> 5) + 8 * i;
                float dot = 0.f;
                for (int c = 0; c < d; ++c) dot = fmaf(sQ[r * dp + c], sK[j * dp + c], dot);
                float s = dot * p.scale;
                if (bias && col < p.cols && row0 + r < p.rows)
                    s += Elem<T>::to_f32(bias[(size_t)(row0 + r) * p.cols + col]);
                sS[r * (CT + 1) + j] = (col < p.cols) ? s * kLog2e : -INFINITY;
            }
        }
        __syncthreads();
        {   // online softmax: warp w updates rows w, w+8, ...
            const int lane = tid & 31, w = tid >> 5;
#pragma unroll 1
            for (int i = 0; i < RB / 8; ++i) {
                const int r = w + 8 * i;
                const float s = sS[r * (CT + 1) + lane];
                float mx = s;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float m_old = sM[r];
                const float m_new = fmaxf(m_old, mx);
                const float pe = (m_new == -INFINITY) ? 0.f : exp2f(s - m_new);
                float sum = pe;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                const float corr = (m_new == -INFINITY) ? 1.f : exp2f(m_old - m_new);
                __syncwarp();
                sS[r * (CT + 1) + lane] = pe;
                if (lane == 0) { sM[r] = m_new; sL[r] = sL[r] * corr + sum; sCorr[r] = corr; }
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < MAXACC; ++i) {
            if (i < nacc) {
                const int e = tid + NT * i;
                if (e < RB * d) {
                    const int r = e / d, c = e - r * d;
                    float a = acc[i] * sCorr[r];
                    for (int j = 0; j < CT; ++j) a = fmaf(sS[r * (CT + 1) + j], sV[j * d + c], a);
                    acc[i] = a;
                }
            }
        }
    }
    __syncthreads();

    if (SPLIT) {
        const size_t pf = partial_floats(rows_pad, d);
        float* slab_parts = p.partials + (size_t)slab * p.splits * pf;
        float* part = slab_parts + (size_t)split * pf;
        if (tid < RB) { part[row0 + tid] = sM[tid]; part[rows_pad + row0 + tid] = sL[tid]; }
#pragma unroll
        for (int i = 0; i < MAXACC; ++i) {
            if (i < nacc) {
                const int e = tid + NT * i;
                if (e < RB * d) {
                    const int r = e / d, c = e - r * d;
                    part[2 * (size_t)rows_pad + (size_t)(row0 + r) * d + c] = acc[i];
                }
            }
        }
        if (arrive_is_last(p.tickets + slab, gridDim.x * gridDim.y, &s_flag))
            merge_partials<T>(slab_parts, p.splits, rows_pad, d, p.rows, d,
                              static_cast<T*>(p.out) + (size_t)slab * p.rows * d);
    } else {
        T* out = static_cast<T*>(p.out) + (size_t)slab * p.rows * d;
        const T* v = p.dwc_w ? static_cast<const T*>(p.dwc_v) + (size_t)slab * p.rows * d : nullptr;
#pragma unroll
        for (int i = 0; i < MAXACC; ++i) {
            if (i < nacc) {
                const int e = tid + NT * i;
                const int r = e / d, c = e - r * d;
                const int tok = row0 + r;
                if (e < RB * d && tok < p.rows) {
                    float o = acc[i] / sL[r];
                    if (v) {   // depthwise 3x3 cross-correlation, zero padding (Eq. 6)
                        const int y = tok / p.W, x = tok - y * p.W;
                        for (int u = 0; u < 3; ++u) {
                            const int yy = y + u - 1;
                            if (yy < 0 || yy >= p.H) continue;
                            for (int vv = 0; vv < 3; ++vv) {
                                const int xx = x + vv - 1;
                                if (xx < 0 || xx >= p.W) continue;
                                o = fmaf(sW[(u * 3 + vv) * d + c],
                                         Elem<T>::to_f32(v[(size_t)(yy * p.W + xx) * d + c]), o);
                            }
                        }
                    }
                    out[(size_t)tok * d + c] = Elem<T>::from_f32(o);
                }
            }
        }
    }
}

AggPlan plan_aggregate_simt(int slabs, int n_agents, int n_tokens, int d, int sm_count) {
    AggPlan pl;
    pl.row_blocks = (n_agents + RB - 1) / RB;
    pl.rows_pad = pl.row_blocks * RB;
    pl.dpad = d;
    const int tiles = (n_tokens + CT - 1) / CT;
    const int blocks1 = slabs * pl.row_blocks;
    int splits = (4 * sm_count + blocks1 - 1) / blocks1;
    if (splits < 1) splits = 1;
    if (splits > tiles) splits = tiles;
    if (splits > 64) splits = 64;
    const int tps = (tiles + splits - 1) / splits;
    pl.splits = (tiles + tps - 1) / tps;          // no empty split
    pl.parts = pl.splits;
    return pl;
}

template <typename T>
static cudaError_t launch_agg_t(const AttnArgs& p, const AggPlan& plan, cudaStream_t st) {
    const size_t smem = simt_smem_floats(p.d) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(attn_simt_kernel<T, true>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid(plan.row_blocks, plan.splits, p.slabs);
    attn_simt_kernel<T, true><<<grid, NT, smem, st>>>(p, plan.rows_pad);
    return cudaGetLastError();
}
template <typename T>
static cudaError_t launch_bc_t(const AttnArgs& p, cudaStream_t st) {
    const size_t smem = simt_smem_floats(p.d) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(attn_simt_kernel<T, false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((p.rows + RB - 1) / RB, 1, p.slabs);
    attn_simt_kernel<T, false><<<grid, NT, smem, st>>>(p, 0);
    return cudaGetLastError();
}

cudaError_t launch_aggregate_simt(int dtype, const AttnArgs& p, const AggPlan& plan, cudaStream_t st) {
    AttnArgs q = p;
    q.splits = plan.splits;
    switch (dtype) {
        case kF32:  return launch_agg_t<float>(q, plan, st);
        case kBF16: return launch_agg_t<__nv_bfloat16>(q, plan, st);
        case kF16:  return launch_agg_t<__half>(q, plan, st);
    }
    return cudaErrorInvalidValue;
}
cudaError_t launch_broadcast_simt(int dtype, const AttnArgs& p, cudaStream_t st) {
    switch (dtype) {
        case kF32:  return launch_bc_t<float>(p, st);
        case kBF16: return launch_bc_t<__nv_bfloat16>(p, st);
        case kF16:  return launch_bc_t<__half>(p, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace aa
