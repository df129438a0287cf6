// Agent aggregation V_A = softmax(scale1 * A K^T + B1) V (Eq. 3, Eq. 5) on tensor cores,
// 16-bit operands, fp32 accumulation.
//
// Grid: (splits, slabs).  A block streams its share of the slab's key/value tiles (64 tokens
// each, plus the matching B1 tile) through a multi-stage shared-memory ring, keeps the n agent
// rows resident, and runs a flash-style online softmax: warp (wm, wk) owns agent rows
// 16*wm .. 16*wm+15 and the wk-th slice of every key tile, with its own (max, sum, acc) state.
// Every warp writes its state as one partial; the last block of the slab merges all partials in
// a fixed order (merge.cuh).
#include "common.cuh"
#include "kernels.h"
#include "merge.cuh"

namespace aa {

namespace {
constexpr int KT = 64;                       // tokens per tile

__host__ __device__ inline int dk_of(int d) { return d <= 32 ? 32 : d <= 48 ? 48 : d <= 64 ? 64 : 128; }
inline int nwk_of(int rows_pad) { return rows_pad <= 32 ? 4 : rows_pad <= 64 ? 2 : 1; }

struct AggSmem {
    size_t a_bytes, k_bytes, b_bytes, stage_bytes, total;
    int stages;
};
inline AggSmem agg_smem(int rows_pad, int dk, bool bias, size_t limit) {
    AggSmem s;
    s.a_bytes = (size_t)rows_pad * (dk + 8) * 2;
    s.k_bytes = (size_t)KT * (dk + 8) * 2;
    s.b_bytes = bias ? (size_t)rows_pad * (KT + 8) * 2 : 0;
    s.stage_bytes = 2 * s.k_bytes + s.b_bytes;
    s.stages = 4;
    while (s.stages > 2 && s.a_bytes + s.stages * s.stage_bytes > limit) --s.stages;
    s.total = s.a_bytes + s.stages * s.stage_bytes;
    return s;
}
}  // namespace

template <typename T, int DK, int NWK>
__global__ void __launch_bounds__(512) aggregate_mma_kernel(AttnArgs p, int rows_pad, int stages) {
    constexpr int PA = DK + 8;                // row pitch (elements) of A, K, V tiles: conflict-free ldmatrix
    constexpr int PB = KT + 8;                // row pitch of the bias tile
    constexpr int KW = KT / NWK;              // keys per warp per tile
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x;
    const int nwm = rows_pad / 16;
    const int wm = warp % nwm, wk = warp / nwm;
    const int split = blockIdx.x, slab = blockIdx.y;
    const int head = slab % p.heads;
    const int n = p.rows, N = p.cols, d = p.d;
    const bool has_bias = p.bias != nullptr;

    const size_t a_bytes = (size_t)rows_pad * PA * 2;
    const size_t k_bytes = (size_t)KT * PA * 2;
    const size_t b_bytes = has_bias ? (size_t)rows_pad * PB * 2 : 0;
    const size_t stage_bytes = 2 * k_bytes + b_bytes;
    T* sA = reinterpret_cast<T*>(smem_raw);
    auto stage_k = [&](int s) { return reinterpret_cast<T*>(smem_raw + a_bytes + s * stage_bytes); };
    auto stage_v = [&](int s) { return reinterpret_cast<T*>(smem_raw + a_bytes + s * stage_bytes + k_bytes); };
    auto stage_b = [&](int s) { return reinterpret_cast<T*>(smem_raw + a_bytes + s * stage_bytes + 2 * k_bytes); };

    const T* gA = static_cast<const T*>(p.qm) + (size_t)slab * n * d;
    const T* gK = static_cast<const T*>(p.km) + (size_t)slab * N * d;
    const T* gV = static_cast<const T*>(p.vm) + (size_t)slab * N * d;
    const T* gB = has_bias ? static_cast<const T*>(p.bias) + (size_t)head * n * N : nullptr;
    const bool bias_vec = has_bias && (N % 8 == 0);     // bias rows start on 16-byte boundaries

    // zero the whole dynamic region once: pad columns, pad rows and unused bias rows stay zero
    {
        const size_t total16 = (a_bytes + (size_t)stages * stage_bytes) / 16;
        uint4* z = reinterpret_cast<uint4*>(smem_raw);
        for (size_t i = tid; i < total16; i += nthreads) z[i] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();

    const int cpr = d / 8;                    // 16-byte chunks per row of A, K, V
    // agents (resident)
    for (int e = tid; e < n * cpr; e += nthreads) {
        const int r = e / cpr, c = e - r * cpr;
        cp_async16(sA + r * PA + c * 8, gA + (size_t)r * d + c * 8, 16);
    }

    const int tiles = (N + KT - 1) / KT;
    const int tps = (tiles + p.splits - 1) / p.splits;
    const int t0 = split * tps, t1 = min(tiles, t0 + tps);

    auto load_tile = [&](int t, int s) {
        const int c0 = t * KT;
        T* sK = stage_k(s);
        T* sV = stage_v(s);
        for (int e = tid; e < KT * cpr; e += nthreads) {
            const int j = e / cpr, c = e - j * cpr;
            const int key = c0 + j;
            const bool ok = key < N;
            const size_t off = ok ? ((size_t)key * d + c * 8) : 0;
            cp_async16(sK + j * PA + c * 8, gK + off, ok ? 16 : 0);
            cp_async16(sV + j * PA + c * 8, gV + off, ok ? 16 : 0);
        }
        if (has_bias) {
            T* sB = stage_b(s);
            if (bias_vec) {
                for (int e = tid; e < n * (KT / 8); e += nthreads) {
                    const int r = e / (KT / 8), c = e - r * (KT / 8);
                    const int key = c0 + c * 8;
                    int bytes = (N - key) * 2;
                    bytes = bytes < 0 ? 0 : (bytes > 16 ? 16 : bytes);
                    cp_async16(sB + r * PB + c * 8, gB + (bytes ? ((size_t)r * N + key) : 0), bytes);
                }
            } else {
                for (int e = tid; e < n * KT; e += nthreads) {
                    const int r = e / KT, j = e - r * KT;
                    const int key = c0 + j;
                    sB[r * PB + j] = key < N ? gB[(size_t)r * N + key] : Elem<T>::from_f32(0.f);
                }
            }
        }
    };

    // prologue
    for (int s = 0; s < stages - 1; ++s) {
        if (t0 + s < t1) load_tile(t0 + s, s);
        cp_async_commit();
    }

    const int g = lane >> 2, t4 = lane & 3;
    const int r0 = wm * 16;
    const int kw0 = wk * KW;
    const float scale_log2 = p.scale * kLog2e;

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float acc[DK / 8][4];
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) { acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f; }
    uint32_t af[DK / 16][4];
    bool a_loaded = false;

    for (int t = t0; t < t1; ++t) {
        const int it = t - t0;
        // tile t was committed as group `it`; at most stages-2 younger groups may stay in flight
        if (stages == 4) cp_async_wait<2>(); else if (stages == 3) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncthreads();
        {
            const int tn = t + stages - 1;
            if (tn < t1) load_tile(tn, (it + stages - 1) % stages);
            cp_async_commit();
        }
        if (!a_loaded) {
#pragma unroll
            for (int ks = 0; ks < DK / 16; ++ks)
                ldmatrix_x4(af[ks][0], af[ks][1], af[ks][2], af[ks][3],
                            sA + (r0 + (lane & 7) + ((lane >> 3) & 1) * 8) * PA + ks * 16 + (lane >> 4) * 8);
            a_loaded = true;
        }
        const int s = it % stages;
        const T* sK = stage_k(s);
        const T* sV = stage_v(s);
        const T* sB = stage_b(s);
        const int c0 = t * KT;

        float sc[KW / 8][4];
#pragma unroll
        for (int j = 0; j < KW / 8; ++j) { sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < DK / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < KW / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3,
                            sK + (kw0 + np * 16 + (lane & 7) + (lane >> 4) * 8) * PA + ks * 16 + ((lane >> 3) & 1) * 8);
                mma16816<T>(sc[2 * np], af[ks], b0, b1);
                mma16816<T>(sc[2 * np + 1], af[ks], b2, b3);
            }
        }
        // logits (log2 units) + bias, mask keys beyond N
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int j = 0; j < KW / 8; ++j) {
            const int col = kw0 + 8 * j + 2 * t4;
            float b00 = 0.f, b01 = 0.f, b10 = 0.f, b11 = 0.f;
            if (has_bias) {
                const float2 u0 = unpack2<T>(*reinterpret_cast<const uint32_t*>(sB + (r0 + g) * PB + col));
                const float2 u1 = unpack2<T>(*reinterpret_cast<const uint32_t*>(sB + (r0 + g + 8) * PB + col));
                b00 = u0.x * kLog2e; b01 = u0.y * kLog2e; b10 = u1.x * kLog2e; b11 = u1.y * kLog2e;
            }
            const bool ok0 = (c0 + col) < N, ok1 = (c0 + col + 1) < N;
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
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float base0 = (mn0 == -INFINITY) ? 0.f : mn0;
        const float base1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float corr0 = fast_exp2(m0 - base0), corr1 = fast_exp2(m1 - base1);
        m0 = mn0; m1 = mn1;
        l0 *= corr0; l1 *= corr1;
#pragma unroll
        for (int j = 0; j < DK / 8; ++j) {
            acc[j][0] *= corr0; acc[j][1] *= corr0; acc[j][2] *= corr1; acc[j][3] *= corr1;
        }
        // probabilities, rounded to the operand type; the row sum uses the rounded values
        uint32_t pk[KW / 8][2];
#pragma unroll
        for (int j = 0; j < KW / 8; ++j) {
            pk[j][0] = pack2<T>(fast_exp2(sc[j][0] - base0), fast_exp2(sc[j][1] - base0));
            pk[j][1] = pack2<T>(fast_exp2(sc[j][2] - base1), fast_exp2(sc[j][3] - base1));
            const float2 q0 = unpack2<T>(pk[j][0]), q1 = unpack2<T>(pk[j][1]);
            l0 += q0.x + q0.y;
            l1 += q1.x + q1.y;
        }
#pragma unroll
        for (int kk = 0; kk < KW / 16; ++kk) {
            const uint32_t pa[4] = {pk[2 * kk][0], pk[2 * kk][1], pk[2 * kk + 1][0], pk[2 * kk + 1][1]};
#pragma unroll
            for (int np = 0; np < DK / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(b0, b1, b2, b3,
                                  sV + (kw0 + kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PA + np * 16 + (lane >> 4) * 8);
                mma16816<T>(acc[2 * np], pa, b0, b1);
                mma16816<T>(acc[2 * np + 1], pa, b2, b3);
            }
        }
    }
    cp_async_wait<0>();

    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    const int parts = p.splits * NWK;
    const size_t pf = partial_floats(rows_pad, DK);
    float* slab_parts = p.partials + (size_t)slab * parts * pf;
    float* part = slab_parts + (size_t)(split * NWK + wk) * pf;
    if (t4 == 0) {
        part[r0 + g] = m0;            part[r0 + g + 8] = m1;
        part[rows_pad + r0 + g] = l0; part[rows_pad + r0 + g + 8] = l1;
    }
    float* pacc = part + 2 * (size_t)rows_pad;
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) {
        const int col = 8 * j + 2 * t4;
        *reinterpret_cast<float2*>(pacc + (size_t)(r0 + g) * DK + col) = make_float2(acc[j][0], acc[j][1]);
        *reinterpret_cast<float2*>(pacc + (size_t)(r0 + g + 8) * DK + col) = make_float2(acc[j][2], acc[j][3]);
    }
    if (arrive_is_last(p.tickets + slab, gridDim.x, &s_flag))
        merge_partials<T>(slab_parts, parts, rows_pad, DK, n, d, static_cast<T*>(p.out) + (size_t)slab * n * d);
}

AggPlan plan_aggregate_mma(int slabs, int n_agents, int n_tokens, int d, int sm_count) {
    AggPlan pl;
    pl.rows_pad = (n_agents + 15) / 16 * 16;
    pl.dpad = dk_of(d);
    pl.row_blocks = 1;
    const int tiles = (n_tokens + KT - 1) / KT;
    int splits = (3 * sm_count + slabs - 1) / slabs;      // about three blocks per SM in total
    if (splits < 1) splits = 1;
    if (splits > (tiles + 1) / 2) splits = (tiles + 1) / 2;   // at least two tiles per block
    if (splits < 1) splits = 1;
    if (splits > 64) splits = 64;
    const int tps = (tiles + splits - 1) / splits;
    pl.splits = (tiles + tps - 1) / tps;
    pl.parts = pl.splits * nwk_of(pl.rows_pad);
    return pl;
}

template <typename T, int DK, int NWK>
static cudaError_t launch_agg(const AttnArgs& p, const AggPlan& plan, cudaStream_t st) {
    const AggSmem sm = agg_smem(plan.rows_pad, DK, p.bias != nullptr, 220 * 1024);
    auto kern = aggregate_mma_kernel<T, DK, NWK>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm.total);
    if (e != cudaSuccess) return e;
    dim3 grid(plan.splits, p.slabs);
    const int threads = 32 * (plan.rows_pad / 16) * NWK;
    kern<<<grid, threads, sm.total, st>>>(p, plan.rows_pad, sm.stages);
    return cudaGetLastError();
}

template <typename T, int DK>
static cudaError_t launch_agg_dk(const AttnArgs& p, const AggPlan& plan, cudaStream_t st) {
    switch (nwk_of(plan.rows_pad)) {
        case 4: return launch_agg<T, DK, 4>(p, plan, st);
        case 2: return launch_agg<T, DK, 2>(p, plan, st);
        default: return launch_agg<T, DK, 1>(p, plan, st);
    }
}

template <typename T>
static cudaError_t launch_agg_t(const AttnArgs& p, const AggPlan& plan, cudaStream_t st) {
    switch (plan.dpad) {
        case 32:  return launch_agg_dk<T, 32>(p, plan, st);
        case 48:  return launch_agg_dk<T, 48>(p, plan, st);
        case 64:  return launch_agg_dk<T, 64>(p, plan, st);
        case 128: return launch_agg_dk<T, 128>(p, plan, st);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_aggregate_mma(int dtype, const AttnArgs& p, const AggPlan& plan, cudaStream_t st) {
    AttnArgs q = p;
    q.splits = plan.splits;
    if (dtype == kBF16) return launch_agg_t<__nv_bfloat16>(q, plan, st);
    if (dtype == kF16)  return launch_agg_t<__half>(q, plan, st);
    return cudaErrorInvalidValue;
}

}  // namespace aa
