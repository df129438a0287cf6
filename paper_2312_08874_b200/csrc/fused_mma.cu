// The whole module of Eq. 6 in one persistent kernel, for small agent counts (n <= 64).
//
// Why one kernel: the path reads Q twice (pooling, broadcast) and V twice (aggregation, DWC).
// Run phase by phase over a large batch, the second reads come from HBM.  Here resident blocks
// pull tasks from a queue ordered slab by slab, so a slab's second reads follow its first ones
// within microseconds and are served by L2; HBM sees every input once.
//
//   G task (slab, range of grid rows): start the K/V/B1 tile ring, pool Q over the range (whole
//     pooling windows: these are complete agent rows), publish them, wait until the slab's other G
//     tasks have published theirs, then run the split aggregation over the range (Eq. 3, Eq. 5).
//     The last G task of a slab merges the partial states into V_A and raises the slab's flag.
//   B task (slab, 128-token tile): start loading Q, the V rows with their 3x3 halo and the B2 tile,
//     wait for the slab's flag, load A and V_A, then broadcast + DWC (Eq. 3, Eq. 5, Eq. 6).
//
// Every wait is bounded: after kSpinLimit polls the block records a timeout in the status word
// and carries on (the result is then wrong, but nothing hangs).  Queue order guarantees progress:
// a task only waits for tasks that precede it or for its own slab's G siblings, which are adjacent
// in the queue, and the grid holds at least as many resident blocks as a slab has G tasks.
#include "common.cuh"
#include "kernels.h"
#include "merge.cuh"

#include <cstring>

namespace aa {

namespace {
constexpr int KT = 64;            // tokens per aggregation tile
constexpr int QT = 128;           // tokens per broadcast tile
constexpr int NT = 256;           // threads per block (8 warps)
constexpr int RP = 64;            // agent rows, padded
constexpr int STAGES = 3;
constexpr int MAXW = 64;          // widest grid the halo buffer is sized for
constexpr unsigned kSpinLimit = 1u << 20;
constexpr int kTimeoutAgents = 1, kTimeoutFeatures = 2;

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Thread 0 polls until *ctr >= target; gives up after kSpinLimit polls and records `code`.
__device__ __forceinline__ void wait_counter(const unsigned* ctr, unsigned target, int* status, int code) {
    if (threadIdx.x == 0) {
        unsigned spins = 0;
        while (ld_acquire(ctr) < target) {
            if (++spins > kSpinLimit) { atomicExch(status, code); break; }
            // once any block has given up, the others stop waiting too
            if ((spins & 255u) == 0 && ld_acquire(reinterpret_cast<const unsigned*>(status)) != 0u) break;
            __nanosleep(40);
        }
    }
    __syncthreads();
}
// Publish: all of this block's prior global writes become visible before the counter moves.
__device__ __forceinline__ void publish_add(unsigned* ctr) {
    __syncthreads();
    if (threadIdx.x == 0) { __threadfence(); atomicAdd(ctr, 1u); }
}

template <int DK> struct FusedSmem {
    static constexpr int PA = DK + 8;                               // padded row pitch (elements)
    static constexpr int PB = KT + 8;                               // B1 tile row pitch
    static constexpr size_t kA = (size_t)RP * PA * 2;               // resident agents
    static constexpr size_t kVA = kA;                               // resident agent features
    static constexpr size_t kCommon = kA + kVA;
    // G layout
    static constexpr size_t kTile = (size_t)KT * PA * 2;
    static constexpr size_t kB1 = (size_t)RP * PB * 2;
    static constexpr size_t kStage = 2 * kTile + kB1;
    static constexpr size_t kG = STAGES * kStage;
    // B layout
    static constexpr int PO = DK + 8;                               // fp32 patch pitch (floats)
    static constexpr size_t kPatch = (size_t)8 * 16 * PO * 4;       // per-warp [16][PO] fp32 (Q rows alias it)
    static constexpr size_t kHalo = (size_t)(QT + 2 * MAXW + 2) * DK * 2;
    static constexpr size_t kB2 = (size_t)QT * RP * 2;
    static constexpr size_t kW = (size_t)9 * DK * 4;
    static constexpr size_t kB = kPatch + kHalo + kB2 + kW;
    static constexpr size_t kTotal = kCommon + (kG > kB ? kG : kB);
};

// Flat global -> shared copy of `bytes` (a multiple of 2) with the widest cp.async the source
// alignment allows; the tail and 2-byte-aligned sources go through plain loads.
__device__ __forceinline__ void copy_flat(unsigned char* dst, const unsigned char* src, int bytes, int tid) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(src);
    if ((a & 15) == 0) {
        const int n16 = bytes >> 4;
        for (int i = tid; i < n16; i += NT) cp_async16(dst + 16 * i, src + 16 * i, 16);
        for (int i = (n16 << 4) + 2 * tid; i < bytes; i += 2 * NT)
            *reinterpret_cast<unsigned short*>(dst + i) = *reinterpret_cast<const unsigned short*>(src + i);
    } else {
        for (int i = 2 * tid; i < bytes; i += 2 * NT)
            *reinterpret_cast<unsigned short*>(dst + i) = *reinterpret_cast<const unsigned short*>(src + i);
    }
}
}  // namespace

// Faster merge for the fused kernel: one thread per (agent row, 4 channels), float4 loads.
template <typename T>
__device__ __forceinline__ void merge_partials_vec(const float* parts_base, int parts, int dpad, int rows,
                                                   int d, T* out) {
    const size_t pf = partial_floats(RP, dpad);
    const int cq = d / 4;
    for (int e = threadIdx.x; e < rows * cq; e += NT) {
        const int r = e / cq, c = (e - r * cq) * 4;
        float m = -INFINITY;
        for (int j = 0; j < parts; ++j) m = fmaxf(m, __ldcg(parts_base + j * pf + r));
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
        float den = 0.f;
#pragma unroll 4
        for (int j = 0; j < parts; ++j) {
            const float* pj = parts_base + j * pf;
            const float mj = __ldcg(pj + r);
            const float w = (mj == -INFINITY) ? 0.f : exp2f(mj - m);
            den += w * __ldcg(pj + RP + r);
            const float4 a = __ldcg(reinterpret_cast<const float4*>(pj + 2 * RP + (size_t)r * dpad + c));
            num.x += w * a.x; num.y += w * a.y; num.z += w * a.z; num.w += w * a.w;
        }
        const float inv = 1.f / den;
        T* o = out + (size_t)r * d + c;
        o[0] = Elem<T>::from_f32(num.x * inv); o[1] = Elem<T>::from_f32(num.y * inv);
        o[2] = Elem<T>::from_f32(num.z * inv); o[3] = Elem<T>::from_f32(num.w * inv);
    }
}

// ---------------------------------------------------------------------------------- G task
template <typename T, int DK>
__device__ __forceinline__ void run_g_task(const FusedArgs& p, int slab, int sub, unsigned char* smem,
                                           int* s_flag) {
    using L = FusedSmem<DK>;
    constexpr int PA = L::PA, PB = L::PB;
    constexpr int NWK = 2, KW = KT / NWK;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp & 3, wk = warp >> 2;
    const int head = slab % p.heads;
    const int N = p.H * p.W, n = p.n, W = p.W;
    const int win_h = p.H / p.p, win_w = p.W / p.p;
    const int gr0 = sub * p.plan.rows_per_g, gr1 = min(p.H, gr0 + p.plan.rows_per_g);
    const int t_begin = gr0 * W, t_end = gr1 * W;
    const int tiles = (t_end - t_begin + KT - 1) / KT;
    const bool has_bias = p.b1 != nullptr;
    const bool bias_vec = has_bias && (N % 8 == 0) && (t_begin % 8 == 0);

    T* sA = reinterpret_cast<T*>(smem);
    unsigned char* ring = smem + L::kCommon;
    auto stage_k = [&](int s) { return reinterpret_cast<T*>(ring + s * L::kStage); };
    auto stage_v = [&](int s) { return reinterpret_cast<T*>(ring + s * L::kStage + L::kTile); };
    auto stage_b = [&](int s) { return reinterpret_cast<T*>(ring + s * L::kStage + 2 * L::kTile); };

    const T* gQ = static_cast<const T*>(p.q) + (size_t)slab * N * DK;
    const T* gK = static_cast<const T*>(p.k) + (size_t)slab * N * DK;
    const T* gV = static_cast<const T*>(p.v) + (size_t)slab * N * DK;
    const T* gB = has_bias ? static_cast<const T*>(p.b1) + (size_t)head * n * N : nullptr;
    T* gA = static_cast<T*>(p.a_ws) + (size_t)slab * n * DK;
    constexpr int cpr = DK / 8;

    auto load_tile = [&](int t, int s) {
        const int c0 = t_begin + t * KT;
        T* sK = stage_k(s);
        T* sV = stage_v(s);
        for (int e = tid; e < KT * cpr; e += NT) {
            const int j = e / cpr, c = e - j * cpr;
            const int key = c0 + j;
            const bool ok = key < t_end;
            const size_t off = ok ? ((size_t)key * DK + c * 8) : 0;
            cp_async16(sK + j * PA + c * 8, gK + off, ok ? 16 : 0);
            cp_async16(sV + j * PA + c * 8, gV + off, ok ? 16 : 0);
        }
        if (has_bias) {
            T* sB = stage_b(s);
            if (bias_vec) {
                for (int e = tid; e < n * (KT / 8); e += NT) {
                    const int r = e / (KT / 8), c = e - r * (KT / 8);
                    const int key = c0 + c * 8;
                    int bytes = (t_end - key) * 2;
                    bytes = bytes < 0 ? 0 : (bytes > 16 ? 16 : bytes);
                    cp_async16(sB + r * PB + c * 8, gB + (bytes ? ((size_t)r * N + key) : 0), bytes);
                }
            } else {
                for (int e = tid; e < n * KT; e += NT) {
                    const int r = e / KT, j = e - r * KT;
                    const int key = c0 + j;
                    sB[r * PB + j] = key < t_end ? gB[(size_t)r * N + key] : Elem<T>::from_f32(0.f);
                }
            }
        }
    };

    // 1. start the ring
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < tiles) load_tile(s, s);
        cp_async_commit();
    }

    // 2. pool this range of Q: whole windows, i.e. complete rows of A (text under Eq. 6)
    {
        const int ar0 = gr0 / win_h, ar1 = gr1 / win_h;
        const int nwin = (ar1 - ar0) * p.p;
        const int cnt = win_h * win_w;
        constexpr int tpl = 32 / cpr;
        const int cg = lane % cpr, tsub = lane / cpr;
        const float inv = 1.f / (float)cnt;
        for (int wi = warp; wi < nwin; wi += NT / 32) {
            const int ay = ar0 + wi / p.p, ax = wi % p.p;
            const int y0 = ay * win_h, x0 = ax * win_w;
            float acc[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] = 0.f;
#pragma unroll 4
            for (int i = tsub; i < cnt; i += tpl) {
                const int wy = i / win_w, wx = i - wy * win_w;
                const size_t tok = (size_t)(y0 + wy) * W + (x0 + wx);
                const uint4 raw = __ldg(reinterpret_cast<const uint4*>(gQ + tok * DK) + cg);
                float f[8];
                unpack16<T>(raw, f);
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] += f[k];
            }
#pragma unroll
            for (int o = cpr; o < 32; o <<= 1) {
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], o);
            }
            if (tsub == 0) {
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] *= inv;
                *(reinterpret_cast<uint4*>(gA + (size_t)(ay * p.p + ax) * DK) + cg) = pack16<T>(acc);
            }
        }
    }
    // 3. publish these agent rows, wait for the slab's other G tasks
    publish_add(p.counters + slab);
    wait_counter(p.counters + slab, (unsigned)p.plan.g_tasks, p.status, kTimeoutAgents);

    // 4. all agents of the slab -> shared memory (L2 reads; rows >= n stay zero)
    for (int e = tid; e < n * cpr; e += NT) {
        const int r = e / cpr, c = e - r * cpr;
        cp_async16(sA + r * PA + c * 8, gA + (size_t)r * DK + c * 8, 16);
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();

    const int g = lane >> 2, t4 = lane & 3;
    const int r0 = wm * 16, kw0 = wk * KW;
    const float scale_log2 = p.scale1 * kLog2e;
    uint32_t af[DK / 16][4];
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks)
        ldmatrix_x4(af[ks][0], af[ks][1], af[ks][2], af[ks][3],
                    sA + (r0 + (lane & 7) + ((lane >> 3) & 1) * 8) * PA + ks * 16 + (lane >> 4) * 8);

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float acc[DK / 8][4];
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) { acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f; }

    // 5. online-softmax aggregation over the range
    for (int it = 0; it < tiles; ++it) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        if (it + STAGES - 1 < tiles) load_tile(it + STAGES - 1, (it + STAGES - 1) % STAGES);
        cp_async_commit();
        const int s = it % STAGES;
        const T* sK = stage_k(s);
        const T* sV = stage_v(s);
        const T* sB = stage_b(s);
        const int c0 = t_begin + it * KT;

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
            const bool ok0 = (c0 + col) < t_end, ok1 = (c0 + col + 1) < t_end;
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

    // 6. partial state of this warp; the slab's last G task merges and raises the slab's flag
    const int parts = p.plan.parts;
    const size_t pf = partial_floats(RP, DK);
    float* slab_parts = p.partials + (size_t)slab * parts * pf;
    float* part = slab_parts + (size_t)(sub * NWK + wk) * pf;
    if (t4 == 0) {
        part[r0 + g] = m0;      part[r0 + g + 8] = m1;
        part[RP + r0 + g] = l0; part[RP + r0 + g + 8] = l1;
    }
    float* pacc = part + 2 * RP;
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) {
        const int col = 8 * j + 2 * t4;
        *reinterpret_cast<float2*>(pacc + (size_t)(r0 + g) * DK + col) = make_float2(acc[j][0], acc[j][1]);
        *reinterpret_cast<float2*>(pacc + (size_t)(r0 + g + 8) * DK + col) = make_float2(acc[j][2], acc[j][3]);
    }
    unsigned* ticket = p.counters + p.slabs + slab;
    if (arrive_is_last(ticket, (unsigned)p.plan.g_tasks, s_flag)) {
        merge_partials_vec<T>(slab_parts, parts, DK, n, DK, static_cast<T*>(p.va_ws) + (size_t)slab * n * DK);
        publish_add(p.counters + 2 * p.slabs + slab);
    }
    __syncthreads();     // the ring is free for the next task
}

// ---------------------------------------------------------------------------------- B task
template <typename T, int DK>
__device__ __forceinline__ void run_b_task(const FusedArgs& p, int slab, int tile, unsigned char* smem) {
    using L = FusedSmem<DK>;
    constexpr int PA = L::PA, PO = L::PO;
    constexpr int cpr = DK / 8;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int head = slab % p.heads;
    const int N = p.H * p.W, n = p.n, W = p.W, H = p.H;
    const int n_pad = (n + 15) & ~15;
    const int q0 = tile * QT;
    const int i0 = q0 + warp * 16;
    const bool has_dwc = p.dwc_w != nullptr;
    const bool has_b2 = p.b2 != nullptr;

    T* sA = reinterpret_cast<T*>(smem);
    T* sVA = reinterpret_cast<T*>(smem + L::kA);
    unsigned char* base = smem + L::kCommon;
    float* sPatch = reinterpret_cast<float*>(base) + (size_t)warp * 16 * PO;
    T* sQ = reinterpret_cast<T*>(sPatch);                           // [16][PA], aliases the patch
    T* sH = reinterpret_cast<T*>(base + L::kPatch);                 // V rows h0..h1, [tokens][DK]
    T* sB2 = reinterpret_cast<T*>(base + L::kPatch + L::kHalo);     // [rows][n] flat
    float* sW = reinterpret_cast<float*>(base + L::kPatch + L::kHalo + L::kB2);   // [9][DK]

    const T* gQ = static_cast<const T*>(p.q) + (size_t)slab * N * DK;
    const T* gV = static_cast<const T*>(p.v) + (size_t)slab * N * DK;
    const int h0 = max(0, q0 - W - 1), h1 = min(N, q0 + QT + W + 1);

    // 1. loads that do not depend on the aggregation
    for (int e = lane; e < 16 * cpr; e += 32) {
        const int r = e / cpr, c = e - r * cpr;
        const bool ok = (i0 + r) < N;
        cp_async16(sQ + r * PA + c * 8, gQ + (ok ? ((size_t)(i0 + r) * DK + c * 8) : 0), ok ? 16 : 0);
    }
    if (has_dwc) {
        const int chunks = (h1 - h0) * cpr;
        const T* src = gV + (size_t)h0 * DK;
        for (int e = tid; e < chunks; e += NT) cp_async16(sH + e * 8, src + e * 8, 16);
        const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * DK * 9;
        for (int e = tid; e < 9 * DK; e += NT) {
            const int c = e / 9, tap = e - c * 9;
            sW[tap * DK + c] = Elem<T>::to_f32(w[e]);
        }
    }
    if (has_b2) {
        const int rows = min(QT, N - q0);
        const T* src = static_cast<const T*>(p.b2) + ((size_t)head * N + q0) * n;
        copy_flat(reinterpret_cast<unsigned char*>(sB2), reinterpret_cast<const unsigned char*>(src),
                  rows * n * 2, tid);
    }
    cp_async_commit();

    // 2. wait for the slab's agent features, then fetch A and V_A (L2)
    wait_counter(p.counters + 2 * p.slabs + slab, 1u, p.status, kTimeoutFeatures);
    {
        const T* gA = static_cast<const T*>(p.a_ws) + (size_t)slab * n * DK;
        const T* gVA = static_cast<const T*>(p.va_ws) + (size_t)slab * n * DK;
        for (int e = tid; e < n * cpr; e += NT) {
            const int r = e / cpr, c = e - r * cpr;
            cp_async16(sA + r * PA + c * 8, gA + (size_t)r * DK + c * 8, 16);
            cp_async16(sVA + r * PA + c * 8, gVA + (size_t)r * DK + c * 8, 16);
        }
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();

    // 3. logits of 16 queries per warp against all agents, softmax over agents, times V_A
    const int g = lane >> 2, t4 = lane & 3;
    uint32_t qf[DK / 16][4];
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks)
        ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3],
                    sQ + ((lane & 7) + ((lane >> 3) & 1) * 8) * PA + ks * 16 + (lane >> 4) * 8);
    __syncwarp();

    const float scale_log2 = p.scale2 * kLog2e;
    const int lr_a = warp * 16 + g, lr_b = lr_a + 8;           // rows within the tile
    float sc[RP / 8][4];
#pragma unroll
    for (int j = 0; j < RP / 8; ++j) { sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks) {
#pragma unroll
        for (int np = 0; np < RP / 16; ++np) {
            if (np * 16 < n_pad) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3,
                            sA + (np * 16 + (lane & 7) + (lane >> 4) * 8) * PA + ks * 16 + ((lane >> 3) & 1) * 8);
                mma16816<T>(sc[2 * np], qf[ks], b0, b1);
                mma16816<T>(sc[2 * np + 1], qf[ks], b2, b3);
            }
        }
    }
    float mx0 = -INFINITY, mx1 = -INFINITY;
    const bool row_a_ok = (q0 + lr_a) < N, row_b_ok = (q0 + lr_b) < N;
#pragma unroll
    for (int j = 0; j < RP / 8; ++j) {
        const int col = 8 * j + 2 * t4;
        const bool ok0 = col < n, ok1 = (col + 1) < n;
        float b00 = 0.f, b01 = 0.f, b10 = 0.f, b11 = 0.f;
        if (has_b2) {
            if (row_a_ok) {
                if (ok0) b00 = Elem<T>::to_f32(sB2[lr_a * n + col]) * kLog2e;
                if (ok1) b01 = Elem<T>::to_f32(sB2[lr_a * n + col + 1]) * kLog2e;
            }
            if (row_b_ok) {
                if (ok0) b10 = Elem<T>::to_f32(sB2[lr_b * n + col]) * kLog2e;
                if (ok1) b11 = Elem<T>::to_f32(sB2[lr_b * n + col + 1]) * kLog2e;
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
    float l0 = 0.f, l1 = 0.f;
    uint32_t pk[RP / 8][2];
#pragma unroll
    for (int j = 0; j < RP / 8; ++j) {
        pk[j][0] = pack2<T>(fast_exp2(sc[j][0] - mx0), fast_exp2(sc[j][1] - mx0));
        pk[j][1] = pack2<T>(fast_exp2(sc[j][2] - mx1), fast_exp2(sc[j][3] - mx1));
        const float2 u0 = unpack2<T>(pk[j][0]), u1 = unpack2<T>(pk[j][1]);
        l0 += u0.x + u0.y;
        l1 += u1.x + u1.y;
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    float acc[DK / 8][4];
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) { acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < RP / 16; ++kk) {
        if (kk * 16 < n_pad) {
            const uint32_t pa[4] = {pk[2 * kk][0], pk[2 * kk][1], pk[2 * kk + 1][0], pk[2 * kk + 1][1]};
#pragma unroll
            for (int np = 0; np < DK / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(b0, b1, b2, b3,
                                  sVA + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PA + np * 16 + (lane >> 4) * 8);
                mma16816<T>(acc[2 * np], pa, b0, b1);
                mma16816<T>(acc[2 * np + 1], pa, b2, b3);
            }
        }
    }
    const float inv0 = 1.f / l0, inv1 = 1.f / l1;
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) {
        const int col = 8 * j + 2 * t4;
        *reinterpret_cast<float2*>(sPatch + g * PO + col) = make_float2(acc[j][0] * inv0, acc[j][1] * inv0);
        *reinterpret_cast<float2*>(sPatch + (g + 8) * PO + col) = make_float2(acc[j][2] * inv1, acc[j][3] * inv1);
    }
    __syncwarp();

    // 4. (token, 8 channels) items: add the depthwise 3x3 term from the V rows in shared memory, store
    T* gO = static_cast<T*>(p.out) + (size_t)slab * N * DK;
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
        if (has_dwc) {
            const int y = tok / W, x = tok - y * W;
#pragma unroll
            for (int u = 0; u < 3; ++u) {
                const int yy = y + u - 1;
                if (yy < 0 || yy >= H) continue;
#pragma unroll
                for (int v = 0; v < 3; ++v) {
                    const int xx = x + v - 1;
                    if (xx < 0 || xx >= W) continue;
                    const uint4 raw = *(reinterpret_cast<const uint4*>(sH + (size_t)(yy * W + xx - h0) * DK) + ch);
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
        *(reinterpret_cast<uint4*>(gO + (size_t)tok * DK) + ch) = pack16<T>(o);
    }
    __syncthreads();     // shared memory is free for the next task
}

// ---------------------------------------------------------------------------------- kernel
template <typename T, int DK>
__global__ void __launch_bounds__(NT, 2) fused_kernel(const __grid_constant__ FusedArgs p) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ int s_task, s_flag;
    const int tid = threadIdx.x;
    {   // zero once: rows >= n of the resident A / V_A must be finite zeros for the whole kernel
        uint4* z = reinterpret_cast<uint4*>(smem);
        for (int i = tid; i < (int)(FusedSmem<DK>::kTotal / 16); i += NT) z[i] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    const int G = p.plan.g_tasks, B = p.plan.b_tasks, Lg = p.plan.lag, S = p.slabs;
    const int count0 = Lg * G, count1 = (S - Lg) * (G + B);
    const int total = S * (G + B);
    unsigned* queue = p.counters + 3 * (size_t)S;
    for (;;) {
        if (tid == 0) s_task = (int)atomicAdd(queue, 1u);
        __syncthreads();
        const int task = s_task;
        __syncthreads();
        if (task >= total) break;
        // queue order: step i holds the G tasks of slab i (i < S) and the B tasks of slab i - lag (i >= lag)
        int slab, sub;
        bool is_g;
        if (task < count0) {
            slab = task / G; sub = task - slab * G; is_g = true;
        } else if (task - count0 < count1) {
            const int t = task - count0;
            const int step = t / (G + B), r = t - step * (G + B);
            is_g = r < G;
            slab = is_g ? (Lg + step) : step;
            sub = is_g ? r : (r - G);
        } else {
            const int t = task - count0 - count1;
            const int step = t / B;
            slab = S - Lg + step; sub = t - step * B; is_g = false;
        }
        if (is_g) run_g_task<T, DK>(p, slab, sub, smem, &s_flag);
        else      run_b_task<T, DK>(p, slab, sub, smem);
    }
}

template <typename T, int DK>
static int fused_occupancy() {
    int occ = 0;
    auto kern = fused_kernel<T, DK>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FusedSmem<DK>::kTotal) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, NT, FusedSmem<DK>::kTotal) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return occ;
}

// Shape part of the plan (no CUDA calls): eligibility, task counts, partial states per slab.
static bool fused_shape_plan(int dtype, int H, int W, int d, int n_agents, FusedPlan* pl) {
    memset(pl, 0, sizeof(*pl));
    if (dtype != kBF16 && dtype != kF16) return false;
    if (d != 32 && d != 64) return false;
    if (n_agents < 1 || n_agents > RP || W > MAXW || H < 1) return false;
    int p = 1;
    while (p * p < n_agents) ++p;
    if (p * p != n_agents || H % p != 0 || W % p != 0) return false;
    const int win_h = H / p;
    // about 448 tokens per G task, in whole agent rows
    int k = (448 + win_h * W / 2) / (win_h * W);
    if (k < 1) k = 1;
    if (k > p) k = p;
    pl->rows_per_g = k * win_h;
    pl->g_tasks = (p + k - 1) / k;
    pl->b_tasks = (H * W + QT - 1) / QT;
    pl->parts = pl->g_tasks * 2;
    return pl->g_tasks <= 32;
}

int fused_parts_per_slab(int dtype, int H, int W, int d, int n_agents) {
    FusedPlan pl;
    return fused_shape_plan(dtype, H, W, d, n_agents, &pl) ? pl.parts : 0;
}

FusedPlan plan_fused(int dtype, int slabs, int H, int W, int d, int n_agents, int sm_count) {
    FusedPlan pl;
    if (!fused_shape_plan(dtype, H, W, d, n_agents, &pl)) { pl.ok = false; return pl; }
    int occ;
    if (dtype == kBF16) occ = d == 64 ? fused_occupancy<__nv_bfloat16, 64>() : fused_occupancy<__nv_bfloat16, 32>();
    else                occ = d == 64 ? fused_occupancy<__half, 64>() : fused_occupancy<__half, 32>();
    if (occ < 1) return pl;
    if (occ > 2) occ = 2;
    const long long total = (long long)slabs * (pl.g_tasks + pl.b_tasks);
    long long grid = (long long)occ * sm_count;
    if (grid > total) grid = total;
    pl.grid = (int)grid;
    if (pl.grid < pl.g_tasks || pl.g_tasks > 32) return pl;      // progress needs a resident block per G sibling
    int lag = (3 * pl.grid / 2 + pl.g_tasks + pl.b_tasks - 1) / (pl.g_tasks + pl.b_tasks) + 1;
    if (lag > slabs) lag = slabs;
    pl.lag = lag;
    pl.smem = d == 64 ? FusedSmem<64>::kTotal : FusedSmem<32>::kTotal;
    pl.ok = true;
    return pl;
}

template <typename T, int DK>
static cudaError_t launch_fused_t(const FusedArgs& a, cudaStream_t st) {
    fused_kernel<T, DK><<<a.plan.grid, NT, FusedSmem<DK>::kTotal, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_fused(int dtype, const FusedArgs& a, cudaStream_t st) {
    if (dtype == kBF16) return a.d == 64 ? launch_fused_t<__nv_bfloat16, 64>(a, st) : launch_fused_t<__nv_bfloat16, 32>(a, st);
    if (dtype == kF16)  return a.d == 64 ? launch_fused_t<__half, 64>(a, st) : launch_fused_t<__half, 32>(a, st);
    return cudaErrorInvalidValue;
}

}  // namespace aa
