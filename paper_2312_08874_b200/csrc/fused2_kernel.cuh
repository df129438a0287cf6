// The whole module of Eq. 6 in one persistent, role-specialised kernel for small agent counts
// (n <= 64, d = 64, 16-bit elements): one block of sixteen warps per SM.
//
//   warps 0-7   "row warps":     own the 128 lanes of tensor memory, two threads per lane (each 32 of
//                                the 64 logit columns).  Aggregation: online softmax per agent row on
//                                logits that tcgen05.mma left in tensor memory.  Broadcast: softmax over
//                                the agents per query row; the normalised row goes to the stencil warps.
//   warps 8-13  "stencil warps": depthwise 3x3 term (Eq. 6) and the store of O, one tile behind the row
//                                warps; they also pool and merge together with the row warps.
//   warp 14     "producer":      one lane issues every TMA / bulk copy, ahead of the others through
//                                full/empty mbarriers.
//   warp 15     "MMA issuer":    one lane issues every tcgen05.mma and its commits.
//
// Blocks take tasks from a device-side queue.  Four kinds, ordered so that a task only ever waits for
// tasks of an EARLIER stage of the queue (no circular waits, any grid size makes progress):
//   P (slab, range of grid rows): pool Q over the range (complete agent rows; text under Eq. 6).
//   G (slab, range): stream K, V and B1 tiles of 64 tokens through a six-slot TMA ring.  A step takes
//     two tiles: rows 0-63 of the 128-row MMA work on the first, rows 64-127 on the second (the agent
//     operand is stacked twice), and each row is shared by two threads that own 32 tokens each with
//     their own running maximum and their own accumulator, so no reduction crosses threads.
//     Logits: S = (scale1 A) K^T + I B1: the bias enters through a second K-block whose A operand is an
//     identity matrix (Eq. 5 inside the contraction).  V_A partial = P V with P written back to shared
//     memory as the A operand (Eq. 3).  The range's partial state goes to the workspace.
//   M (slab): merge the slab's partial states into V_A (fixed order: bit-reproducible).
//   B (slab, run of broadcast tiles): per tile of whole grid rows (<= 128 tokens) S = Q A^T by
//     tcgen05.mma, softmax with B2 per query row (Eq. 5), O = P V_A, then the depthwise term on the V
//     rows that a ring of row slots keeps in shared memory.  Loads run two tiles ahead, the softmax one
//     tile ahead of the stencil.
// Stages interleave groups of slabs (P of group g+3, G of g+2, M of g+1, B of g) sized so that the Q and
// V of the groups in flight stay in L2.
//
// Every wait is bounded (mbarrier waits and flag polls give up, set the status word and a block-wide
// flag that makes every later wait return at once), so a logic error ends as a status code, not as a
// hang.  No TMA multicast, no clusters.
#pragma once
#include "common.cuh"
#include "kernels.h"
#include "merge.cuh"
#include "tma.cuh"
#include "umma.cuh"

namespace aa {
namespace f2 {

constexpr int DK = 64;            // head dim
constexpr int KT = 64;            // tokens per aggregation tile
constexpr int QT = 128;           // most tokens per broadcast tile
constexpr int RP = 64;            // agent rows, padded
constexpr int NR = 256;           // row warps 0-7
constexpr int NX = 192;           // stencil warps 8-13
constexpr int NCOMP = NR + NX;    // compute threads
constexpr int NT = NCOMP + 64;    // + producer warp + MMA issuer warp: 512 threads, 128 registers each
constexpr int kWarpProd = 14, kWarpMma = 15;
constexpr int RING = 6;           // aggregation ring slots (one tile each)
constexpr int MAXW = 64, MINW = 8;
constexpr int kVTokens = 400;     // V row slots: (2R + 2)(W + 2) tokens at most
constexpr unsigned kSpinLimit = 1u << 20;
constexpr unsigned kBarLimit = 1u << 22;
constexpr int kTimeoutAgents = 1, kTimeoutFeatures = 2, kTimeoutTile = 3, kTimeoutLoads = 4, kTimeoutRole = 6;
constexpr float kTau = 5.5f;      // a row's reference maximum moves only when exceeded by this much (natural units)

// ------------------------------------------------------------------ shared-memory map (bytes)
constexpr int kTile = KT * 128;                       // swizzled [64][64] tile of 16-bit elements
constexpr int OFF_W = 0;                              // filter taps [9][64] fp32
constexpr int OFF_BAR = 2304;                         // mbarriers (8 bytes each)
constexpr int kNumBars = 40;
constexpr int OFF_UNION = 3072;
// aggregation
constexpr int G_ASTACK = OFF_UNION;                   // [128][128 B]: scaled agents, twice
constexpr int G_IDENT = G_ASTACK + 2 * kTile;         // [128][128 B]: identity, twice
constexpr int G_P = G_IDENT + 2 * kTile;              // [128][128 B]: probabilities of the step
constexpr int G_RING = G_P + 2 * kTile;               // RING x (K | V | B1)
constexpr int kSlot = 3 * kTile;
constexpr int G_END = G_RING + RING * kSlot;
// broadcast
constexpr int PO = DK + 4;                            // patch pitch (floats)
constexpr int kPatch = QT * PO * 4;
constexpr int kB2Buf = QT * RP * 2 + 64;
constexpr int B_A = OFF_UNION;                        // [64][128 B] agents (B operand of S)
constexpr int B_VA = B_A + kTile;                     // [64][128 B] agent features (B operand of O)
constexpr int B_Q = B_VA + kTile;                     // 2 x [128][128 B] query tiles
constexpr int B_P = B_Q + 4 * kTile;                  // [128][128 B] probabilities
constexpr int B_PATCH = B_P + 2 * kTile;              // 2 x [128][PO] fp32
constexpr int B_B2 = B_PATCH + 2 * kPatch;            // 2 x bias tiles (flat rows of n elements)
constexpr int B_V = B_B2 + 2 * kB2Buf;                // V row slots
constexpr int B_END = B_V + kVTokens * 128;
constexpr int kSmemBytes = (G_END > B_END ? G_END : B_END) + 1024;   // + slack to align the base to 1024
static_assert(OFF_W + 9 * DK * 4 <= OFF_BAR && OFF_BAR + 8 * kNumBars <= OFF_UNION, "common area");
static_assert(OFF_UNION % 1024 == 0 && kTile % 1024 == 0 && B_V % 128 == 0 && B_B2 % 16 == 0 && kB2Buf % 16 == 0, "alignment");
static_assert(kSmemBytes <= 232448, "shared memory per block");
static_assert(kSmemBytes > 116 * 1024, "one block per SM: each block takes all 512 tensor-memory columns");

// mbarrier indices                   count     waiter
constexpr int BAR_FULL = 0;          // [RING]  tx        MMA issuer      tile landed
constexpr int BAR_EMPTY = 6;         // [RING]  commit    producer        tile consumed
constexpr int BAR_S_FULL = 12;       // [2]     commit    row warps       logits ready
constexpr int BAR_S_EMPTY = 14;      // [2]     256       MMA issuer      logits read
constexpr int BAR_PG_FULL = 16;      //         256       MMA issuer      aggregation: P of the step written
constexpr int BAR_PB_FULL = 17;      //         1         MMA issuer      broadcast: P of the tile written
constexpr int BAR_PV = 18;           //         commit    row warps       P V product done
constexpr int BAR_AG = 19;           //         tx        MMA issuer      agents (and features) landed
constexpr int BAR_PREP = 20;         //         1         MMA issuer      identity / plain-load bias tiles written
constexpr int BAR_IN_FULL = 21;      // [2]     tx        MMA issuer      Q and B2 tile landed
constexpr int BAR_IN_EMPTY = 23;     // [2]     256       producer        Q and B2 tile consumed
constexpr int BAR_PATCH_FULL = 25;   // [2]     256       stencil warps   normalised rows written
constexpr int BAR_PATCH_EMPTY = 27;  // [2]     256       row warps       patch consumed
constexpr int BAR_V_FULL = 29;       // [2]     tx        stencil warps   V rows of a tile landed
constexpr int BAR_V_EMPTY = 31;      // [2]     256       producer        V rows of a tile consumed
constexpr int kBarsUsed = 33;
static_assert(kBarsUsed <= kNumBars, "barriers");
__host__ __device__ constexpr uint32_t bar_count(int i) {
    return ((i >= BAR_S_EMPTY && i <= BAR_PG_FULL) || (i >= BAR_IN_EMPTY && i < BAR_PATCH_EMPTY)) ? (uint32_t)NR
           : ((i >= BAR_PATCH_EMPTY && i < BAR_V_FULL) || i >= BAR_V_EMPTY) ? (uint32_t)NX : 1u;
}

// tensor-memory columns (512 allocated)
constexpr uint32_t TM_GS = 0;        // aggregation logits: 2 buffers x 128 columns (two tiles per step)
constexpr uint32_t TM_GO = 256;      // aggregation accumulators: 4 x 64 columns, index 2 * (stack half) + (token half)
constexpr uint32_t TM_BS = 0;        // broadcast logits: 2 x 64
constexpr uint32_t TM_BO = 128;      // broadcast outputs: 2 x 64

struct Role {
    int* status;          // device status word
    int* dead;            // shared flag: some wait of this block gave up
    uint32_t bars;        // shared address of mbarrier 0
    uint64_t ph;          // parity to wait for next, one bit per mbarrier (each role tracks the ones it waits on)
    uint32_t tmem;
};
__device__ __forceinline__ uint32_t bar_addr(const Role& ro, int i) { return ro.bars + 8u * (uint32_t)i; }

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_shared_volatile(const int* p) { return *reinterpret_cast<const volatile int*>(p); }

// Bounded wait of ONE thread for the next phase of mbarrier i (this thread's parity bit flips either way).
__device__ __forceinline__ void wait_bar_one(Role& ro, int i, int code) {
    const uint32_t parity = (uint32_t)(ro.ph >> i) & 1u;
    ro.ph ^= 1ull << i;
    if (ld_shared_volatile(ro.dead)) return;
    const uint32_t bar = bar_addr(ro, i);
    for (unsigned tries = 0; tries < kBarLimit; ++tries) {
        if (mbar_try_wait(bar, parity)) return;
        if (tries > 4) __nanosleep(32);
        if ((tries & 255u) == 255u && ld_shared_volatile(ro.dead)) return;
    }
    *reinterpret_cast<volatile int*>(ro.dead) = 1;
    atomicCAS(ro.status, 0, code);
}
// The same for a whole (converged) warp: lane 0 polls, so that waiting warps leave the shared-memory
// pipeline to the working ones; the warp barrier passes the acquired data on to the other lanes.
__device__ __forceinline__ void wait_bar(Role& ro, int i, int code) {
    if ((threadIdx.x & 31) == 0) {
        wait_bar_one(ro, i, code);
    } else {
        ro.ph ^= 1ull << i;
    }
    __syncwarp();
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
// Bounded poll of a global counter by one thread.
__device__ __forceinline__ void poll_counter(Role& ro, const unsigned* ctr, unsigned target, int code) {
    if (ld_shared_volatile(ro.dead)) return;
    unsigned spins = 0;
    while (ld_acquire(ctr) < target) {
        if (++spins > kSpinLimit) {
            *reinterpret_cast<volatile int*>(ro.dead) = 1;
            atomicCAS(ro.status, 0, code);
            return;
        }
        if ((spins & 255u) == 0 && (ld_acquire(reinterpret_cast<const unsigned*>(ro.status)) != 0u || ld_shared_volatile(ro.dead))) return;
        __nanosleep(40);
    }
}
// Thread 0 polls, then the whole block (all 288 threads) passes a barrier.
__device__ __forceinline__ void wait_counter_block(Role& ro, const unsigned* ctr, unsigned target, int code) {
    if (threadIdx.x == 0) poll_counter(ro, ctr, target, code);
    __syncthreads();
}
__device__ __forceinline__ void publish_add(unsigned* ctr) {
    __syncthreads();
    if (threadIdx.x == 0) { __threadfence(); atomicAdd(ctr, 1u); }
}
__device__ __forceinline__ void sync_rows() { asm volatile("bar.sync 1, 256;\n" ::: "memory"); }      // warps 0-7
__device__ __forceinline__ void sync_stencil() { asm volatile("bar.sync 2, %0;\n" ::"n"(NX) : "memory"); }     // warps 8-13
__device__ __forceinline__ void sync_compute() { asm volatile("bar.sync 3, %0;\n" ::"n"(NCOMP) : "memory"); }  // warps 0-13

__device__ __forceinline__ int swz(int row, int col) {
    return row * 128 + ((((col >> 3) ^ row) & 7) << 4) + (col & 7) * 2;
}
// 32 consecutive fp32 columns of this thread's tensor-memory row <- registers
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }

template <int H_, int W_, int P_> struct Shape {
    static constexpr int kH = H_, kW = W_, kP = P_;
    static constexpr bool kFixed = (H_ > 0);
};
using ShapeAny = Shape<0, 0, 0>;

// Optional per-task timestamps (debug builds only): define AA_FUSED2_TRACE and hand a device buffer to
// aa_fused2_trace_buffer; record (block, task slot < 32) holds eight values: entries 0-5 are globaltimer
// marks of thread 0, entry 6 the task kind + 1, entry 7 the task index.
#ifdef AA_FUSED2_TRACE
__device__ unsigned long long* g_trace2 = nullptr;
__device__ __forceinline__ void trace_put(int slot, int entry, unsigned long long v) {
    if (g_trace2 && slot < 32) g_trace2[((size_t)blockIdx.x * 32 + slot) * 8 + entry] = v;
}
__device__ __forceinline__ void trace_mark(int slot, int entry) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    trace_put(slot, entry, t);
}
#define TR(entry) if (threadIdx.x == 0) trace_mark(slot, entry)
#else
#define TR(entry)
#endif

// ---------------------------------------------------------------------------------- P task
// Pool Q over a range of grid rows that covers whole pooling windows: complete rows of A.  Each window
// is split over `nsplit` warps (by token index inside the window); the parts meet in shared memory.
template <typename T, typename SH>
__device__ __forceinline__ void run_p_task(const FusedArgs& p, int slab, int sub, unsigned char* smem, int slot) {
    constexpr int cpr = DK / 8;               // 16-byte chunks per token row
    constexpr int tpl = 32 / cpr;             // tokens per warp-wide load
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = SH::kFixed ? SH::kH : p.H, W = SH::kFixed ? SH::kW : p.W, P = SH::kFixed ? SH::kP : p.p;
    const int N = H * W, n = SH::kFixed ? SH::kP * SH::kP : p.n;
    const int win_h = H / P, win_w = W / P;
    const int gr0 = sub * p.plan.rows_per_g, gr1 = min(H, gr0 + p.plan.rows_per_g);
    const int ar0 = gr0 / win_h, ar1 = gr1 / win_h;
    const int nwin = (ar1 - ar0) * P;
    const int cnt = win_h * win_w;
    int nsplit = (NCOMP / 32) / nwin;
    if (nsplit < 1) nsplit = 1;
    if (nsplit > 8) nsplit = 8;
    while (nsplit > 1 && tpl * nsplit > cnt) --nsplit;        // at least one load per part
    const T* gQ = static_cast<const T*>(p.q) + (size_t)slab * N * DK;
    T* gAg = static_cast<T*>(p.ag_ws) + (size_t)slab * RP * DK;     // scale1 * A, rows >= n zero
    T* gAb = static_cast<T*>(p.ab_ws) + (size_t)slab * RP * DK;     // A, rows >= n zero
    float* sPart = reinterpret_cast<float*>(smem + OFF_UNION);      // [window][part][64]
    TR(0);
    if (warp < NCOMP / 32) {
        const int cg = lane % cpr, tsub = lane / cpr;
        for (int item = warp; item < nwin * nsplit; item += NCOMP / 32) {
            const int wi = item / nsplit, part = item - wi * nsplit;
            const int ay = ar0 + wi / P, ax = wi % P;
            const int y0 = ay * win_h, x0 = ax * win_w;
            float acc[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] = 0.f;
            for (int ib = tsub + part * tpl; ib < cnt; ib += 8 * tpl * nsplit) {    // eight loads in flight per lane
                uint4 raw[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = ib + u * tpl * nsplit;
                    raw[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (i < cnt) {
                        const int wy = i / win_w, wx = i - wy * win_w;
                        const size_t tok = (size_t)(y0 + wy) * W + (x0 + wx);
                        raw[u] = __ldg(reinterpret_cast<const uint4*>(gQ + tok * DK) + cg);
                    }
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float f[8];
                    unpack16<T>(raw[u], f);
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] += f[k];
                }
            }
#pragma unroll
            for (int o = cpr; o < 32; o <<= 1) {
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], o);
            }
            if (tsub == 0) {
                float* d = sPart + ((size_t)wi * nsplit + part) * DK + cg * 8;
                *reinterpret_cast<float4*>(d) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                *reinterpret_cast<float4*>(d + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
            }
        }
        sync_compute();
        const float inv = 1.f / (float)cnt;
        for (int e = tid; e < nwin * cpr; e += NCOMP) {
            const int wi = e / cpr, c8 = e - wi * cpr;
            float a[8], sc[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) a[k] = 0.f;
            for (int part = 0; part < nsplit; ++part) {         // fixed order: bit-reproducible
                const float* d = sPart + ((size_t)wi * nsplit + part) * DK + c8 * 8;
#pragma unroll
                for (int k = 0; k < 8; ++k) a[k] += d[k];
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) { a[k] *= inv; sc[k] = a[k] * p.scale1; }
            const int arow = (ar0 + wi / P) * P + wi % P;
            *(reinterpret_cast<uint4*>(gAb + (size_t)arow * DK) + c8) = pack16<T>(a);
            *(reinterpret_cast<uint4*>(gAg + (size_t)arow * DK) + c8) = pack16<T>(sc);
        }
        if (sub == 0)                        // padded agent rows are zero in both copies
            for (int e = tid; e < (RP - n) * cpr; e += NCOMP) {
                *(reinterpret_cast<uint4*>(gAb + (size_t)n * DK) + e) = make_uint4(0u, 0u, 0u, 0u);
                *(reinterpret_cast<uint4*>(gAg + (size_t)n * DK) + e) = make_uint4(0u, 0u, 0u, 0u);
            }
    }
    publish_add(p.counters + slab);        // block barrier, then one release + add
    fence_proxy_async();
    __syncthreads();
    TR(1);
}

// ---------------------------------------------------------------------------------- M task
// All partial states of the slab -> V_A (log-sum-exp merge in the fixed order of the parts).
template <typename T, typename SH>
__device__ __forceinline__ void run_m_task(const FusedArgs& p, int slab, Role& ro, int slot) {
    const int tid = threadIdx.x;
    const int n = SH::kFixed ? SH::kP * SH::kP : p.n;
    const int parts = p.plan.parts;
    const size_t pf = partial_floats(RP, DK);
    const float* slab_parts = p.partials + (size_t)slab * parts * pf;
    TR(0);
    wait_counter_block(ro, p.counters + p.slabs + slab, (unsigned)p.plan.g_tasks, kTimeoutAgents);
    TR(1);
    if (tid < NCOMP) {
        T* va = static_cast<T*>(p.va2_ws) + (size_t)slab * RP * DK;
        for (int e = tid; e < n * (DK / 4); e += NCOMP) {
            const int r = e / (DK / 4), c = (e % (DK / 4)) * 4;
            float mx = -INFINITY, den = 0.f;
            float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
            for (int q = 0; q < parts; ++q) {
                const float* pq = slab_parts + q * pf;
                const float mq = __ldcg(pq + r);
                const float lq = __ldcg(pq + RP + r);
                const float4 a = __ldcg(reinterpret_cast<const float4*>(pq + 2 * RP + (size_t)r * DK + c));
                const float mn = fmaxf(mx, mq);
                const float bs = (mn == -INFINITY) ? 0.f : mn;
                const float c0 = exp2f(mx - bs), c1 = exp2f(mq - bs);
                den = den * c0 + lq * c1;
                num.x = num.x * c0 + a.x * c1; num.y = num.y * c0 + a.y * c1;
                num.z = num.z * c0 + a.z * c1; num.w = num.w * c0 + a.w * c1;
                mx = mn;
            }
            const float inv = 1.f / den;
            uint2 o;
            o.x = pack2<T>(num.x * inv, num.y * inv);
            o.y = pack2<T>(num.z * inv, num.w * inv);
            *reinterpret_cast<uint2*>(va + (size_t)r * DK + c) = o;
        }
        // padded feature rows are zero (0 * NaN is not 0)
        for (int e = tid; e < (RP - n) * (DK / 8); e += NCOMP)
            *(reinterpret_cast<uint4*>(va + (size_t)n * DK) + e) = make_uint4(0u, 0u, 0u, 0u);
    }
    publish_add(p.counters + 2 * p.slabs + slab);
    __syncthreads();
    TR(2);
}

// ---------------------------------------------------------------------------------- G task
template <typename T, typename SH>
__device__ __forceinline__ void run_g_task(const FusedArgs& p, int slab, int sub, unsigned char* smem, Role& ro, int slot) {
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int head = slab % p.heads;
    const int H = SH::kFixed ? SH::kH : p.H, W = SH::kFixed ? SH::kW : p.W;
    const int N = H * W, n = SH::kFixed ? SH::kP * SH::kP : p.n;
    const int gr0 = sub * p.plan.rows_per_g, gr1 = min(H, gr0 + p.plan.rows_per_g);
    const int t_begin = gr0 * W, t_end = gr1 * W;
    const int tiles = (t_end - t_begin + KT - 1) / KT;
    const int steps = (tiles + 1) >> 1;
    const bool has_bias = SH::kFixed ? true : (p.b1 != nullptr);
    const bool bias_tma = has_bias && p.b1_tma;
    const bool prep = has_bias;                    // identity operand (and plain-load bias tiles) to build

    const uint32_t ring_u32 = smem_u32(smem + G_RING);
    const uint32_t astack = smem_u32(smem + G_ASTACK), ident = smem_u32(smem + G_IDENT), sP = smem_u32(smem + G_P);
    const size_t pf = partial_floats(RP, DK);
    TR(0);

    if (warp == kWarpProd) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const uint32_t tile_tx = 2 * kTile + (bias_tma ? kTile : 0);
            auto fill = [&](int t) {
                const int s = t % RING, c0 = t_begin + t * KT;
                const uint32_t bar = bar_addr(ro, BAR_FULL + s), dst = ring_u32 + s * kSlot;
                mbar_arrive_expect_tx(bar, tile_tx);
                tma_load_2d(dst, &p.tm_k, 0, slab * N + c0, bar);
                tma_load_2d(dst + kTile, &p.tm_v, 0, slab * N + c0, bar);
                if (bias_tma) tma_load_2d(dst + 2 * kTile, &p.tm_b1, c0, head * n, bar);
            };
            for (int t = 0; t < tiles && t < RING; ++t) fill(t);
            // the slab's agents: every P task of the slab has published its rows
            poll_counter(ro, p.counters + slab, (unsigned)p.plan.g_tasks, kTimeoutAgents);
            {
                const uint32_t bar = bar_addr(ro, BAR_AG);
                mbar_arrive_expect_tx(bar, 2 * kTile);
                tma_load_2d(astack, &p.tm_ag, 0, slab * RP, bar);
                tma_load_2d(astack + kTile, &p.tm_ag, 0, slab * RP, bar);
            }
            for (int t = RING; t < tiles; ++t) {
                wait_bar_one(ro, BAR_EMPTY + t % RING, kTimeoutRole);
                fill(t);
            }
            for (int t = max(0, tiles - RING); t < tiles; ++t) wait_bar_one(ro, BAR_EMPTY + t % RING, kTimeoutRole);
        }
        __syncwarp();
    } else if (warp == kWarpMma) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idK = umma_idesc(fmt, 128, 64, 0), idMN = umma_idesc(fmt, 128, 64, 1);
            const uint64_t dA = umma_desc_sw128(astack), dI = umma_desc_sw128(ident), dP = umma_desc_sw128(sP);
            const uint64_t dRing = umma_desc_sw128(ring_u32);
            // descriptor start addresses count 16-byte units: + 2 per 32 bytes (one K-step of a K-major
            // operand), + 128 per 2048 bytes (one K-step of an MN-major operand)
            auto issue_S = [&](int j) {
                const int nt2 = min(2, tiles - 2 * j);
                if (j >= 2) wait_bar_one(ro, BAR_S_EMPTY + (j & 1), kTimeoutRole);
                for (int h2 = 0; h2 < nt2; ++h2) wait_bar_one(ro, BAR_FULL + (2 * j + h2) % RING, kTimeoutTile);
                tc_fence_after_sync();
                for (int h2 = 0; h2 < nt2; ++h2) {
                    const uint32_t d = ro.tmem + TM_GS + 128 * (j & 1) + 64 * h2;
                    const uint64_t dK = dRing + (uint64_t)(((2 * j + h2) % RING) * (kSlot >> 4));
                    const uint64_t dB = dK + (uint64_t)((2 * kTile) >> 4);
#pragma unroll
                    for (int kk = 0; kk < DK / 16; ++kk) umma_f16(d, dA + 2 * kk, dK + 2 * kk, idK, kk > 0);
                    if (has_bias) {
#pragma unroll
                        for (int kk = 0; kk < RP / 16; ++kk) umma_f16(d, dI + 2 * kk, dB + 128 * kk, idMN, 1u);
                    }
                }
                umma_commit(bar_addr(ro, BAR_S_FULL + (j & 1)));
            };
            if (prep) wait_bar_one(ro, BAR_PREP, kTimeoutRole);
            wait_bar_one(ro, BAR_AG, kTimeoutLoads);
            unsigned started = 0u;                    // accumulators that hold a product already
            issue_S(0);
            for (int j = 0; j < steps; ++j) {
                if (j + 1 < steps) issue_S(j + 1);
                wait_bar_one(ro, BAR_PG_FULL, kTimeoutRole);
                tc_fence_after_sync();
                const int nt2 = min(2, tiles - 2 * j);
                for (int h2 = 0; h2 < nt2; ++h2) {
                    const int t = 2 * j + h2, sl = t % RING;
                    const int ntok = min(KT, t_end - (t_begin + t * KT));
                    const uint64_t dV = dRing + (uint64_t)(sl * (kSlot >> 4)) + (uint64_t)(kTile >> 4);
                    for (int c = 0; c < 2; ++c) {
                        if (32 * c >= ntok) break;
                        const int a = 2 * h2 + c;
                        const uint32_t d = ro.tmem + TM_GO + 64 * a;
#pragma unroll
                        for (int k2 = 0; k2 < 2; ++k2) {
                            const int kk = 2 * c + k2;
                            umma_f16(d, dP + 2 * kk, dV + 128 * kk, idMN, (((started >> a) & 1u) || k2 > 0) ? 1u : 0u);
                        }
                        started |= 1u << a;
                    }
                    umma_commit(bar_addr(ro, BAR_EMPTY + sl));
                }
                umma_commit(bar_addr(ro, BAR_PV));
            }
            for (int j = max(0, steps - 2); j < steps; ++j) wait_bar_one(ro, BAR_S_EMPTY + (j & 1), kTimeoutRole);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ compute warps
        if (prep) {
            // identity, stacked twice: row r has a one at k = r % 64 (the A operand of the bias K-block)
            const unsigned short one = Elem<T>::kIsBf16 ? 0x3F80u : 0x3C00u;
            for (int idx = tid; idx < 128 * 8; idx += NCOMP) {
                const int row = idx >> 3, c = idx & 7;
                const int lc = c ^ (row & 7);                 // logical 16-byte chunk: k = 8 lc .. 8 lc + 7
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                const int k = row & 63;
                if ((k >> 3) == lc) {
                    const uint32_t w = (uint32_t)one << (16 * (k & 1));
                    const int wi = (k & 7) >> 1;
                    if (wi == 0) v.x = w; else if (wi == 1) v.y = w; else if (wi == 2) v.z = w; else v.w = w;
                }
                *reinterpret_cast<uint4*>(smem + G_IDENT + row * 128 + c * 16) = v;
            }
            if (!bias_tma) {                 // the plan guarantees tiles <= RING here
                const T* gB = static_cast<const T*>(p.b1) + (size_t)head * n * N;
                for (int t = 0; t < tiles; ++t) {
                    unsigned char* sB = smem + G_RING + (t % RING) * kSlot + 2 * kTile;
                    const int c0 = t_begin + t * KT;
                    for (int e = tid; e < RP * KT; e += NCOMP) {
                        const int rr = e / KT, j = e - rr * KT;
                        const int key = c0 + j;
                        *reinterpret_cast<T*>(sB + swz(rr, j)) =
                            (rr < n && key < t_end) ? gB[(size_t)rr * N + key] : Elem<T>::from_f32(0.f);
                    }
                }
            }
            fence_proxy_async();             // the tensor core reads these through the async proxy
            sync_compute();
            if (tid == 0) mbar_arrive(bar_addr(ro, BAR_PREP));
        }
        if (warp < NR / 32) {
            // -------------------------------------------------------------- row warps
            const int row = tid & 127, ch = tid >> 7;          // tensor-memory lane, token half of the tile
            const int half = row >> 6;                         // stack half: which tile of the step
            const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
            const uint32_t tO = ro.tmem + TM_GO + 64 * (2 * half + ch) + lane_base;
            float m_ref = -INFINITY, l = 0.f;
            bool started = false;
            for (int j = 0; j < steps; ++j) {
                const int buf = j & 1;
                wait_bar(ro, BAR_S_FULL + buf, kTimeoutTile);
                tc_fence_after_sync();
                const int t = 2 * j + half;
                int valid = 0;
                if (t < tiles) valid = min(32, t_end - (t_begin + t * KT + 32 * ch));
                const bool tv = valid > 0;                     // uniform per warp
                float s[32];
                {
                    uint32_t ra[32];
                    tmem_ld32(ro.tmem + TM_GS + 128 * buf + 64 * half + 32 * ch + lane_base, ra);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 32; ++k) s[k] = __uint_as_float(ra[k]);
                }
                tc_fence_before_sync();
                mbar_arrive(bar_addr(ro, BAR_S_EMPTY + buf));
                uint32_t pk[16];
                float corr = 1.f;
                bool resc = false;
                if (tv) {
                    if (valid < 32) {
#pragma unroll
                        for (int k = 0; k < 32; ++k) if (k >= valid) s[k] = -INFINITY;
                    }
                    float mx0 = fmaxf(s[0], s[1]), mx1 = fmaxf(s[2], s[3]), mx2 = fmaxf(s[4], s[5]), mx3 = fmaxf(s[6], s[7]);
#pragma unroll
                    for (int k = 8; k < 32; k += 8) {
                        mx0 = fmaxf(mx0, fmaxf(s[k], s[k + 1]));     mx1 = fmaxf(mx1, fmaxf(s[k + 2], s[k + 3]));
                        mx2 = fmaxf(mx2, fmaxf(s[k + 4], s[k + 5])); mx3 = fmaxf(mx3, fmaxf(s[k + 6], s[k + 7]));
                    }
                    const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                    if (mx > m_ref + kTau) {                   // also the first tile of the row (m_ref = -inf)
                        corr = fast_exp2((m_ref - mx) * kLog2e);
                        resc = started;
                        m_ref = mx;
                        l *= corr;
                    }
                    const float nb = -m_ref * kLog2e;
                    float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
#pragma unroll
                    for (int k = 0; k < 16; k += 2) {
                        const float p0 = fast_exp2(fmaf(s[2 * k], kLog2e, nb));       // exp2(-inf) = 0 past the range
                        const float p1 = fast_exp2(fmaf(s[2 * k + 1], kLog2e, nb));
                        const float p2 = fast_exp2(fmaf(s[2 * k + 2], kLog2e, nb));
                        const float p3 = fast_exp2(fmaf(s[2 * k + 3], kLog2e, nb));
                        sum0 += p0; sum1 += p1; sum2 += p2; sum3 += p3;
                        pk[k] = pack2<T>(p0, p1);
                        pk[k + 1] = pack2<T>(p2, p3);
                    }
                    l += (sum0 + sum1) + (sum2 + sum3);
                    started = true;
                }
                if (j > 0) { wait_bar(ro, BAR_PV, kTimeoutTile); tc_fence_after_sync(); }
                if (__any_sync(0xffffffffu, resc)) {           // rare: the reference maximum of some row moved
                    uint32_t ra[32];
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        tmem_ld32(tO + 32 * hh, ra);
                        tmem_ld_wait();
#pragma unroll
                        for (int k = 0; k < 32; ++k) ra[k] = __float_as_uint(__uint_as_float(ra[k]) * corr);
                        tmem_st32(tO + 32 * hh, ra);
                    }
                    tmem_st_wait();
                }
                if (tv) {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        *reinterpret_cast<uint4*>(smem + G_P + row * 128 + (((4 * ch + c) ^ (row & 7)) << 4)) =
                            make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                }
                fence_proxy_async();
                tc_fence_before_sync();
                mbar_arrive(bar_addr(ro, BAR_PG_FULL));
            }
            wait_bar(ro, BAR_PV, kTimeoutTile);
            tc_fence_after_sync();
            TR(1);
            // the four states of an agent row (stack half x token half) meet in shared memory
            float* sX = reinterpret_cast<float*>(smem + G_RING);        // [4][64][68]: row, m, l
            {
                uint32_t ra[32], rb[32];
                tmem_ld32(tO, ra);
                tmem_ld32(tO + 32, rb);
                tmem_ld_wait();
                float* x = sX + ((size_t)(2 * half + ch) * 64 + (row & 63)) * 68;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    *reinterpret_cast<float4*>(x + 4 * k) = started
                        ? make_float4(__uint_as_float(ra[4 * k]), __uint_as_float(ra[4 * k + 1]), __uint_as_float(ra[4 * k + 2]), __uint_as_float(ra[4 * k + 3]))
                        : make_float4(0.f, 0.f, 0.f, 0.f);
                    *reinterpret_cast<float4*>(x + 32 + 4 * k) = started
                        ? make_float4(__uint_as_float(rb[4 * k]), __uint_as_float(rb[4 * k + 1]), __uint_as_float(rb[4 * k + 2]), __uint_as_float(rb[4 * k + 3]))
                        : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                x[64] = m_ref; x[65] = started ? l : 0.f;
            }
            tc_fence_before_sync();
            sync_rows();
            {
                const int a = tid & 63, q = tid >> 6;          // agent row, quarter of the channels
                float mm = -INFINITY;
#pragma unroll
                for (int st = 0; st < 4; ++st) mm = fmaxf(mm, sX[((size_t)st * 64 + a) * 68 + 64]);
                const float bs = (mm == -INFINITY) ? 0.f : mm;
                float wgt[4], lsum = 0.f;
#pragma unroll
                for (int st = 0; st < 4; ++st) {
                    wgt[st] = fast_exp2((sX[((size_t)st * 64 + a) * 68 + 64] - bs) * kLog2e);     // exp2(-inf) = 0
                    lsum += sX[((size_t)st * 64 + a) * 68 + 65] * wgt[st];
                }
                float* part = p.partials + ((size_t)slab * p.plan.parts + sub) * pf;
                if (q == 0) { part[a] = mm * kLog2e; part[RP + a] = lsum; }      // the merge works in log2 units
                float* pacc = part + 2 * RP + (size_t)a * DK + 16 * q;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int st = 0; st < 4; ++st) {
                        const float4 xv = *reinterpret_cast<const float4*>(sX + ((size_t)st * 64 + a) * 68 + 16 * q + 4 * k);
                        acc.x += xv.x * wgt[st]; acc.y += xv.y * wgt[st]; acc.z += xv.z * wgt[st]; acc.w += xv.w * wgt[st];
                    }
                    *reinterpret_cast<float4*>(pacc + 4 * k) = acc;
                }
            }
        }
    }
    TR(2);
    publish_add(p.counters + p.slabs + slab);       // block barrier (the ring is drained), release + add
    fence_proxy_async();   // this task's plain shared-memory writes precede the next task's TMA writes
    __syncthreads();
    TR(3);
}

// ---------------------------------------------------------------------------------- B task
// A run of broadcast tiles of one slab.  Tile = R whole grid rows (R W <= 128 tokens).  V rows live in
// NSLOT = 2R + 2 row slots of W + 2 tokens (zero columns at x = -1 and x = W): grid row y sits in slot
// (y - y_first + 1) mod NSLOT, so consecutive tiles share their halo rows and only R new rows per tile
// are fetched.
template <typename T, typename SH>
__device__ __forceinline__ void run_b_task(const FusedArgs& p, int slab, int run, unsigned char* smem, Role& ro,
                                           int* s_whead, float (*s_red)[128], int slot) {
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int head = slab % p.heads;
    const int H = SH::kFixed ? SH::kH : p.H, W = SH::kFixed ? SH::kW : p.W;
    const int N = H * W, n = SH::kFixed ? SH::kP * SH::kP : p.n;
    const int n16 = (n + 15) >> 4;
    const int R = SH::kFixed ? (QT / SH::kW > 16 ? 16 : (QT / SH::kW > SH::kH ? SH::kH : QT / SH::kW)) : p.plan.rows_per_b;
    const int NSLOT = 2 * R + 2, HP = W + 2;
    const int tile0 = run * p.plan.tb;
    const int nt = min(p.plan.tb, p.plan.b_tiles - tile0);
    const int y_first = tile0 * R;
    const bool has_dwc = SH::kFixed ? true : (p.dwc_w != nullptr);
    const bool has_b2 = SH::kFixed ? true : (p.b2 != nullptr);

    float* sW = reinterpret_cast<float*>(smem + OFF_W);
    T* sV = reinterpret_cast<T*>(smem + B_V);
    const T* gV = static_cast<const T*>(p.v) + (size_t)slab * N * DK;
    const size_t b2_total = (size_t)p.heads * N * n * 2;           // bytes of the whole B2 array
    const size_t b2_head_off = (size_t)head * N * n * 2;
    auto slot_of = [&](int y) { return (y - y_first + 1) % NSLOT; };
    TR(0);

    if (warp == kWarpProd) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            poll_counter(ro, p.counters + 2 * p.slabs + slab, 1u, kTimeoutFeatures);     // the slab's M task is done
            {
                const uint32_t bar = bar_addr(ro, BAR_AG);
                mbar_arrive_expect_tx(bar, 2 * kTile);
                tma_load_2d(smem_u32(smem + B_A), &p.tm_ab, 0, slab * RP, bar);
                tma_load_2d(smem_u32(smem + B_VA), &p.tm_va2, 0, slab * RP, bar);
            }
            for (int i = 0; i < nt; ++i) {
                const int b = i & 1;
                const int y0 = y_first + i * R, rows = min(R, H - y0);
                const int q0 = y0 * W, TQ = rows * W;
                if (i >= 2) wait_bar_one(ro, BAR_IN_EMPTY + b, kTimeoutRole);
                {
                    // B2 rows of the tile: the 16-byte aligned span that covers them, clipped to the array
                    uint32_t nb2 = 0;
                    size_t lo = 0;
                    if (has_b2) {
                        const size_t beg = b2_head_off + (size_t)q0 * n * 2, end = beg + (size_t)TQ * n * 2;
                        lo = beg & ~(size_t)15;
                        size_t hi = (end + 15) & ~(size_t)15;
                        if (hi > (b2_total & ~(size_t)15)) hi = b2_total & ~(size_t)15;
                        nb2 = hi > lo ? (uint32_t)(hi - lo) : 0u;
                    }
                    const uint32_t bar = bar_addr(ro, BAR_IN_FULL + b);
                    mbar_arrive_expect_tx(bar, (uint32_t)QT * 128 + nb2);
                    tma_load_2d(smem_u32(smem + B_Q + b * 2 * kTile), &p.tm_q, 0, slab * N + q0, bar);
                    if (nb2) bulk_load_1d(smem_u32(smem + B_B2 + b * kB2Buf), reinterpret_cast<const unsigned char*>(p.b2) + lo, nb2, bar);
                }
                if (has_dwc) {
                    if (i >= 2) wait_bar_one(ro, BAR_V_EMPTY + b, kTimeoutRole);
                    int ylo = (i == 0) ? y0 - 1 : y0 + 1, yhi = y0 + rows;
                    if (ylo < 0) ylo = 0;
                    if (yhi > H - 1) yhi = H - 1;
                    const int cnt = yhi >= ylo ? yhi - ylo + 1 : 0;
                    const uint32_t bar = bar_addr(ro, BAR_V_FULL + b);
                    mbar_arrive_expect_tx(bar, (uint32_t)cnt * W * 128);
                    for (int y = ylo; y <= yhi; ++y)
                        bulk_load_1d(smem_u32(sV + ((size_t)slot_of(y) * HP + 1) * DK), gV + (size_t)y * W * DK, W * 128, bar);
                }
            }
            for (int i = max(0, nt - 2); i < nt; ++i) {
                wait_bar_one(ro, BAR_IN_EMPTY + (i & 1), kTimeoutRole);
                if (has_dwc) wait_bar_one(ro, BAR_V_EMPTY + (i & 1), kTimeoutRole);
            }
        }
        __syncwarp();
    } else if (warp == kWarpMma) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idK = umma_idesc(fmt, 128, 64, 0), idMN = umma_idesc(fmt, 128, 64, 1);
            const uint64_t dA = umma_desc_sw128(smem_u32(smem + B_A)), dVA = umma_desc_sw128(smem_u32(smem + B_VA));
            const uint64_t dP = umma_desc_sw128(smem_u32(smem + B_P)), dQ0 = umma_desc_sw128(smem_u32(smem + B_Q));
            auto issue_S = [&](int i) {
                const int b = i & 1;
                if (i >= 2) wait_bar_one(ro, BAR_S_EMPTY + b, kTimeoutRole);
                wait_bar_one(ro, BAR_IN_FULL + b, kTimeoutLoads);
                tc_fence_after_sync();
                const uint64_t dQ = dQ0 + (uint64_t)(b * ((2 * kTile) >> 4));
#pragma unroll
                for (int kk = 0; kk < DK / 16; ++kk) umma_f16(ro.tmem + TM_BS + 64 * b, dQ + 2 * kk, dA + 2 * kk, idK, kk > 0);
                umma_commit(bar_addr(ro, BAR_S_FULL + b));
            };
            wait_bar_one(ro, BAR_AG, kTimeoutLoads);
            issue_S(0);
            for (int i = 0; i < nt; ++i) {
                if (i + 1 < nt) issue_S(i + 1);
                wait_bar_one(ro, BAR_PB_FULL, kTimeoutRole);
                tc_fence_after_sync();
                for (int kk = 0; kk < n16; ++kk) umma_f16(ro.tmem + TM_BO + 64 * (i & 1), dP + 2 * kk, dVA + 128 * kk, idMN, kk > 0);
                umma_commit(bar_addr(ro, BAR_PV));
            }
            for (int i = max(0, nt - 2); i < nt; ++i) wait_bar_one(ro, BAR_S_EMPTY + (i & 1), kTimeoutRole);
        }
        __syncwarp();
    } else if (warp < NR / 32) {
        // ------------------------------------------------------------------ row warps
        const int row = tid & 127, ch = tid >> 7;              // query row of the tile, half of the agent columns
        const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
        const int c0 = 32 * ch;
        for (int i = 0; i < nt; ++i) {
            const int b = i & 1;
            const int y0 = y_first + i * R, rows = min(R, H - y0);
            const int q0 = y0 * W, TQ = rows * W;
            wait_bar(ro, BAR_S_FULL + b, kTimeoutLoads);
            tc_fence_after_sync();
            float s[32];
            {
                uint32_t ra[32];
                tmem_ld32(ro.tmem + TM_BS + 64 * b + c0 + lane_base, ra);
                tmem_ld_wait();
#pragma unroll
                for (int k = 0; k < 32; ++k) s[k] = __uint_as_float(ra[k]);
            }
            tc_fence_before_sync();
            mbar_arrive(bar_addr(ro, BAR_S_EMPTY + b));
            // logits in natural units: t = scale2 * q.a + b2; columns >= n are not agents
            float mx = -INFINITY;
            if (has_b2) {
                // the bulk copy stops at the last 16-byte boundary inside the array: a tile that ends the
                // array fetches the few bytes behind it with plain loads
                const size_t beg = b2_head_off + (size_t)q0 * n * 2, end = beg + (size_t)TQ * n * 2;
                const size_t lo = beg & ~(size_t)15, lim = b2_total & ~(size_t)15;
                if (end > lim) {
                    const size_t g = (lim > lo ? lim : lo) + 2 * (size_t)tid;
                    if (tid < 8 && g < end)
                        *reinterpret_cast<unsigned short*>(smem + B_B2 + b * kB2Buf + (g - lo)) =
                            *reinterpret_cast<const unsigned short*>(reinterpret_cast<const unsigned char*>(p.b2) + g);
                    sync_rows();
                }
                // element index of this thread's first bias value inside the buffer (the copy starts at a 16-byte boundary)
                const uint32_t e0 = (uint32_t)((beg & 15) >> 1) + (uint32_t)row * n + c0;
                const uint32_t* w32 = reinterpret_cast<const uint32_t*>(smem + B_B2 + b * kB2Buf) + (e0 >> 1);
                const int sh = (e0 & 1) * 16;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (c0 + 2 * j < n) {
                        const float2 bb = unpack2<T>(__funnelshift_r(w32[j], w32[j + 1], sh));
                        s[2 * j] = fmaf(s[2 * j], p.scale2, bb.x);
                        s[2 * j + 1] = (c0 + 2 * j + 1 < n) ? fmaf(s[2 * j + 1], p.scale2, bb.y) : -INFINITY;
                        mx = fmaxf(mx, fmaxf(s[2 * j], s[2 * j + 1]));
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (c0 + 2 * j < n) {
                        s[2 * j] = s[2 * j] * p.scale2;
                        s[2 * j + 1] = (c0 + 2 * j + 1 < n) ? s[2 * j + 1] * p.scale2 : -INFINITY;
                        mx = fmaxf(mx, fmaxf(s[2 * j], s[2 * j + 1]));
                    }
                }
            }
            mbar_arrive(bar_addr(ro, BAR_IN_EMPTY + b));     // the Q tile and this thread's bias values are consumed
            s_red[ch][row] = mx;
            sync_rows();
            mx = fmaxf(mx, s_red[ch ^ 1][row]);
            const float nm = -mx * kLog2e;
            float l0 = 0.f, l1 = 0.f;
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (c0 + 2 * j < n) {
                    const float p0 = fast_exp2(fmaf(s[2 * j], kLog2e, nm));
                    const float p1 = fast_exp2(fmaf(s[2 * j + 1], kLog2e, nm));      // exp2(-inf) = 0 past the last agent
                    pk[j] = pack2<T>(p0, p1);
                    const float2 q = unpack2<T>(pk[j]);    // the normaliser sums the rounded weights
                    l0 += q.x; l1 += q.y;
                } else {
                    pk[j] = 0u;
                }
            }
            s_red[2 + ch][row] = l0 + l1;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4*>(smem + B_P + row * 128 + (((4 * ch + c) ^ (row & 7)) << 4)) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            fence_proxy_async();
            sync_rows();
            if (tid == 0) mbar_arrive(bar_addr(ro, BAR_PB_FULL));
            const float inv = 1.f / (l0 + l1 + s_red[2 + (ch ^ 1)][row]);
            wait_bar(ro, BAR_PV, kTimeoutLoads);
            tc_fence_after_sync();
            if (i >= 2) wait_bar(ro, BAR_PATCH_EMPTY + b, kTimeoutRole);
            {
                float* prow = reinterpret_cast<float*>(smem + B_PATCH + b * kPatch) + row * PO + c0;
                uint32_t ra[32];
                tmem_ld32(ro.tmem + TM_BO + 64 * b + c0 + lane_base, ra);
                tmem_ld_wait();
                if (row < TQ) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        *reinterpret_cast<float4*>(prow + 4 * k) =
                            make_float4(__uint_as_float(ra[4 * k]) * inv, __uint_as_float(ra[4 * k + 1]) * inv,
                                        __uint_as_float(ra[4 * k + 2]) * inv, __uint_as_float(ra[4 * k + 3]) * inv);
                }
                tc_fence_before_sync();
            }
            mbar_arrive(bar_addr(ro, BAR_PATCH_FULL + b));
        }
        TR(1);
        for (int i = max(0, nt - 2); i < nt; ++i) wait_bar(ro, BAR_PATCH_EMPTY + (i & 1), kTimeoutRole);
    } else {
        // ------------------------------------------------------------------ stencil warps
        const int t2 = tid - NR;
        if (has_dwc) {
            // zero columns x = -1 and x = W of every slot; the row above the grid if the run starts the slab
            for (int e = t2; e < NSLOT * 2 * (DK / 8); e += NX) {
                const int sl = e / (2 * (DK / 8)), rest = e - sl * 2 * (DK / 8);
                const int side = rest / (DK / 8), c = rest - side * (DK / 8);
                *(reinterpret_cast<uint4*>(sV + ((size_t)sl * HP + (side ? W + 1 : 0)) * DK) + c) = make_uint4(0, 0, 0, 0);
            }
            if (y_first == 0)
                for (int e = t2; e < W * (DK / 8); e += NX) *(reinterpret_cast<uint4*>(sV + DK) + e) = make_uint4(0, 0, 0, 0);
            if (ld_shared_volatile(s_whead) != head) {       // filter taps change only with the head
                const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * DK * 9;
                for (int e = t2; e < 9 * DK; e += NX) {
                    const int c = e / 9, tap = e - c * 9;
                    sW[tap * DK + c] = Elem<T>::to_f32(w[e]);
                }
            }
            sync_stencil();
            if (t2 == 0) *s_whead = head;
        }
        for (int i = 0; i < nt; ++i) {
            const int b = i & 1;
            const int y0 = y_first + i * R, rows = min(R, H - y0);
            const int q0 = y0 * W;
            if (has_dwc) {
                wait_bar(ro, BAR_V_FULL + b, kTimeoutLoads);
                if (y0 + rows >= H) {            // the row below the grid
                    T* z = sV + ((size_t)slot_of(H) * HP + 1) * DK;
                    for (int e = t2; e < W * (DK / 8); e += NX) *(reinterpret_cast<uint4*>(z) + e) = make_uint4(0, 0, 0, 0);
                    sync_stencil();
                }
            }
            wait_bar(ro, BAR_PATCH_FULL + b, kTimeoutRole);
            // depthwise 3x3 term + store: thread = (tile row r, 4-channel group cq, x-segment)
            {
                constexpr int NCQ = DK / 4;
                const float* sPatch = reinterpret_cast<const float*>(smem + B_PATCH + b * kPatch);
                const int npairs = rows * NCQ;
                int nseg = NX / npairs;
                if (nseg < 1) nseg = 1;
                if (nseg > W) nseg = W;
                const int seg_len = (W + nseg - 1) / nseg;
                T* gO = static_cast<T*>(p.out) + ((size_t)slab * N + q0) * DK;
                for (int item = t2; item < npairs * nseg; item += NX) {
                    const int pair = item % npairs, seg = item / npairs;
                    const int r = pair / NCQ, cq = pair - r * NCQ;
                    const int x0 = seg * seg_len, x1 = min(W, x0 + seg_len);
                    if (x0 >= x1) continue;
                    const float* pp = sPatch + (r * W) * PO + cq * 4;
                    T* op = gO + (size_t)(r * W) * DK + cq * 4;
                    if (has_dwc) {
                        float2 w[9][2];                 // taps x two channel pairs
#pragma unroll
                        for (int tap = 0; tap < 9; ++tap) {
                            const float4 t = *reinterpret_cast<const float4*>(sW + tap * DK + cq * 4);
                            w[tap][0] = make_float2(t.x, t.y);
                            w[tap][1] = make_float2(t.z, t.w);
                        }
                        // slots of grid rows y-1, y, y+1; buffer column x+1 is grid column x
                        const int y = y0 + r;
                        const T* hp[3];
#pragma unroll
                        for (int u = 0; u < 3; ++u) hp[u] = sV + (size_t)slot_of(y - 1 + u) * HP * DK + cq * 4;
                        float2 ca[3][2], cb[3][2], cc[3][2];
                        auto load_col = [&](int hx, float2 (&c)[3][2]) {
#pragma unroll
                            for (int u = 0; u < 3; ++u) {
                                const uint2 raw = *reinterpret_cast<const uint2*>(hp[u] + hx * DK);
                                c[u][0] = unpack2<T>(raw.x);
                                c[u][1] = unpack2<T>(raw.y);
                            }
                        };
                        auto emit = [&](int x, const float2 (&lft)[3][2], const float2 (&c)[3][2], const float2 (&rr)[3][2]) {
                            const float4 a4 = *reinterpret_cast<const float4*>(pp + x * PO);
                            float2 o0 = make_float2(a4.x, a4.y), o1 = make_float2(a4.z, a4.w);
#pragma unroll
                            for (int u = 0; u < 3; ++u) {
                                o0 = ffma2(w[u * 3 + 0][0], lft[u][0], o0); o1 = ffma2(w[u * 3 + 0][1], lft[u][1], o1);
                                o0 = ffma2(w[u * 3 + 1][0], c[u][0], o0);   o1 = ffma2(w[u * 3 + 1][1], c[u][1], o1);
                                o0 = ffma2(w[u * 3 + 2][0], rr[u][0], o0);  o1 = ffma2(w[u * 3 + 2][1], rr[u][1], o1);
                            }
                            uint2 outw;
                            outw.x = pack2<T>(o0.x, o0.y);
                            outw.y = pack2<T>(o1.x, o1.y);
                            *reinterpret_cast<uint2*>(op + x * DK) = outw;
                        };
                        load_col(x0, ca);          // grid column x0 - 1
                        load_col(x0 + 1, cb);      // grid column x0
                        int x = x0;
                        while (x < x1) {           // the three window columns rotate roles instead of moving
                            load_col(x + 2, cc); emit(x, ca, cb, cc); if (++x >= x1) break;
                            load_col(x + 2, ca); emit(x, cb, cc, ca); if (++x >= x1) break;
                            load_col(x + 2, cb); emit(x, cc, ca, cb); ++x;
                        }
                    } else {
                        for (int x = x0; x < x1; ++x) {
                            const float4 a4 = *reinterpret_cast<const float4*>(pp + x * PO);
                            uint2 outw;
                            outw.x = pack2<T>(a4.x, a4.y);
                            outw.y = pack2<T>(a4.z, a4.w);
                            *reinterpret_cast<uint2*>(op + x * DK) = outw;
                        }
                    }
                }
            }
            if (has_dwc) {
                fence_proxy_async();           // these slots are next written through the async proxy
                mbar_arrive(bar_addr(ro, BAR_V_EMPTY + b));
            }
            mbar_arrive(bar_addr(ro, BAR_PATCH_EMPTY + b));
        }
    }
    TR(2);
    fence_proxy_async();   // this task's plain shared-memory writes precede the next task's TMA writes
    __syncthreads();       // shared memory is free for the next task
    TR(3);
}

// ---------------------------------------------------------------------------------- kernel
// Queue order: stage t holds the B tasks of slab group t-3, the M tasks of group t-2, the G tasks of
// group t-1 and the P tasks of group t (groups of plan.lag slabs), so every task's inputs come from an
// earlier stage.
template <typename T, typename SH>
__global__ void __launch_bounds__(NT, 1) fused2_kernel(const __grid_constant__ FusedArgs p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_info[4], s_whead, s_dead;
    __shared__ uint32_t s_tmem;
    __shared__ float s_red[4][128];     // per query row: maxima and sums of the two column halves
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x;
    Role ro;
    ro.status = p.status;
    ro.dead = &s_dead;
    ro.bars = smem_u32(smem + OFF_BAR);
    ro.ph = 0ull;
    if (tid == 0) {
        s_whead = -1;
        s_dead = 0;
        for (int i = 0; i < kBarsUsed; ++i) mbar_init(ro.bars + 8 * i, bar_count(i));
        mbar_fence_init();
    }
    if (tid < 32) tmem_alloc<512>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    ro.tmem = s_tmem;
    const int G = p.plan.g_tasks, B = p.plan.b_tasks, Lg = p.plan.lag, S = p.slabs;
    const int NG = (S + Lg - 1) / Lg;
    const int total = S * (2 * G + 1 + B);
    unsigned* queue = p.counters + 3 * (size_t)S;
    int slot = 0;
    for (;;) {
        if (tid == 0) {
            int idx = (int)atomicAdd(queue, 1u);
            int kind = -1, slab = 0, sub = 0;
            if (idx < total) {
                for (int t = 0; t < NG + 3 && kind < 0; ++t) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {           // B, M, G, P
                        const int g = t - 3 + k;
                        if (kind >= 0 || g < 0 || g >= NG) continue;
                        const int ns = min(Lg, S - g * Lg);
                        const int per = k == 0 ? B : (k == 1 ? 1 : G);
                        const int cnt = ns * per;
                        if (idx < cnt) { kind = 3 - k; slab = g * Lg + idx / per; sub = idx % per; }
                        else idx -= cnt;
                    }
                }
            }
            s_info[0] = kind; s_info[1] = slab; s_info[2] = sub;
        }
        __syncthreads();
        const int kind = s_info[0], slab = s_info[1], sub = s_info[2];
        __syncthreads();
        if (kind < 0) break;
        if (kind == 0) run_p_task<T, SH>(p, slab, sub, smem, slot);
        else if (kind == 1) run_g_task<T, SH>(p, slab, sub, smem, ro, slot);
        else if (kind == 2) run_m_task<T, SH>(p, slab, ro, slot);
        else run_b_task<T, SH>(p, slab, sub, smem, ro, &s_whead, s_red, slot);
#ifdef AA_FUSED2_TRACE
        if (tid == 0) { trace_put(slot, 6, (unsigned long long)(kind + 1)); trace_put(slot, 7, (unsigned long long)(slab * 64 + sub)); }
#endif
        ++slot;
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid < 32) tmem_dealloc<512>(ro.tmem);
}

// Per-instantiation host helpers: attribute set-up and launch.
template <typename T, typename SH>
static bool fused2_prepare_of() {
    auto kern = fused2_kernel<T, SH>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return true;
}
template <typename SH>
static bool fused2_prepare_dt(int dtype) {
    return dtype == kBF16 ? fused2_prepare_of<__nv_bfloat16, SH>() : fused2_prepare_of<__half, SH>();
}
template <typename SH>
static cudaError_t fused2_launch_dt(int dtype, const FusedArgs& a, cudaStream_t st) {
    if (dtype == kBF16) fused2_kernel<__nv_bfloat16, SH><<<a.plan.grid, NT, kSmemBytes, st>>>(a);
    else if (dtype == kF16) fused2_kernel<__half, SH><<<a.plan.grid, NT, kSmemBytes, st>>>(a);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace f2
}  // namespace aa
