// The whole module of Eq. 6 in one persistent, role-specialised kernel for small agent counts
// (n <= 64, d = 64, 16-bit elements): one block per SM, nine warps.
//
//   warps 0-3  "row group":   own the 128 lanes of tensor memory.  Aggregation: one thread per agent
//                             row does the online softmax on logits that tcgen05.mma left in tensor
//                             memory.  Broadcast: one thread per query row does the softmax over the
//                             agents and hands the normalised row to the stencil group.
//   warps 4-7  "stencil group": depthwise 3x3 term (Eq. 6) and the store of O, one tile behind the
//                             row group; pooling (together with the row group).
//   warp 8     "producer":    one lane issues every TMA / bulk copy, running ahead of the others
//                             through full/empty mbarriers.
//
// Blocks take tasks from a device-side queue (same order and progress argument as the first fused
// kernel: a task waits only for earlier tasks or for its slab's G siblings, which are adjacent in the
// queue, and the grid holds at least as many blocks as a slab has G tasks).
//
//   G task (slab, range of grid rows): pool Q over the range (complete agent rows), publish, wait for
//     the siblings, then stream K, V and B1 tiles of 64 tokens through a six-slot TMA ring.  A step
//     takes two tiles: rows 0-63 of the 128-row MMA work on the first, rows 64-127 on the second
//     (the agent operand is stacked twice), so all 128 lanes carry useful rows with n <= 64.
//     Logits: S = (scale1 A) K^T + I B1, i.e. the bias enters through a second K-block whose A operand
//     is an identity matrix (Eq. 5 inside the contraction).  V_A partial = P V with P written back to
//     shared memory as the A operand (Eq. 3).  Partial states are merged as in the first kernel.
//   B task (slab, run of broadcast tiles): per tile of whole grid rows (<= 128 tokens) S = Q A^T by
//     tcgen05.mma, softmax with B2 per query row (Eq. 5), O = P V_A, then the depthwise term on the V
//     rows that a ring of row slots keeps in shared memory.  The three roles are pipelined over the
//     run's tiles: loads two tiles ahead, softmax one tile ahead of the stencil.
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
constexpr int NCOMP = 256;        // compute threads (row group + stencil group)
constexpr int NT = NCOMP + 32;    // + producer warp
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
constexpr int OFF_BAR = 2304;                         // mbarriers
constexpr int kNumBars = 32;
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

// mbarrier indices
constexpr int BAR_FULL = 0;          // [RING]  tile landed                     (tx)      waiter: row-group leader
constexpr int BAR_EMPTY = 6;         // [RING]  tile consumed                   (commit)  waiter: producer
constexpr int BAR_S = 12;            // [2]     logits ready                    (commit)  waiter: row group
constexpr int BAR_PV = 14;           //         P V product done                (commit)  waiter: row group
constexpr int BAR_AG = 15;           //         agents (and features) landed    (tx)      waiter: row group
constexpr int BAR_IN_FULL = 16;      // [2]     Q and B2 tile landed            (tx)      waiter: row-group leader
constexpr int BAR_IN_EMPTY = 18;     // [2]     Q and B2 tile consumed          (128)     waiter: producer
constexpr int BAR_PATCH_FULL = 20;   // [2]     normalised rows written         (128)     waiter: stencil group
constexpr int BAR_PATCH_EMPTY = 22;  // [2]     patch consumed                  (128)     waiter: row group
constexpr int BAR_V_FULL = 24;       // [2]     V rows of a tile landed         (tx)      waiter: stencil group
constexpr int BAR_V_EMPTY = 26;      // [2]     V rows of a tile consumed       (128)     waiter: producer
constexpr int kBarsUsed = 28;
static_assert(kBarsUsed <= kNumBars, "barriers");

// tensor-memory columns (512 allocated)
constexpr uint32_t TM_GS = 0;        // aggregation logits: 2 buffers x 128 columns (two tiles per step)
constexpr uint32_t TM_GO = 256;      // aggregation accumulators: rows 0-63 use columns [256, 320), rows 64-127 [320, 384)
constexpr uint32_t TM_BS = 0;        // broadcast logits: 2 x 64
constexpr uint32_t TM_BO = 128;      // broadcast outputs: 2 x 64

struct Role {
    int* status;          // device status word
    int* dead;            // shared flag: some wait of this block gave up
    uint32_t bars;        // shared address of mbarrier 0
    uint32_t ph;          // parity to wait for next, one bit per mbarrier (each role tracks the ones it waits on)
    uint32_t tmem;
};
__device__ __forceinline__ uint32_t bar_addr(const Role& ro, int i) { return ro.bars + 8u * (uint32_t)i; }

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_shared_volatile(const int* p) { return *reinterpret_cast<const volatile int*>(p); }

// Bounded wait for the next phase of mbarrier i (this role's parity bit flips either way).
__device__ __forceinline__ void wait_bar(Role& ro, int i, int code) {
    const uint32_t parity = (ro.ph >> i) & 1u;
    ro.ph ^= 1u << i;
    if (ld_shared_volatile(ro.dead)) return;
    const uint32_t bar = bar_addr(ro, i);
    for (unsigned tries = 0; tries < kBarLimit; ++tries) {
        if (mbar_try_wait(bar, parity)) return;
        if (tries > 16) __nanosleep(20);
        if ((tries & 255u) == 255u && ld_shared_volatile(ro.dead)) return;
    }
    *reinterpret_cast<volatile int*>(ro.dead) = 1;
    atomicCAS(ro.status, 0, code);
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
__device__ __forceinline__ void sync_rows() { asm volatile("bar.sync 1, 128;\n" ::: "memory"); }      // warps 0-3
__device__ __forceinline__ void sync_stencil() { asm volatile("bar.sync 2, 128;\n" ::: "memory"); }   // warps 4-7
__device__ __forceinline__ void sync_compute() { asm volatile("bar.sync 3, 256;\n" ::: "memory"); }   // warps 0-7

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

// ---------------------------------------------------------------------------------- G task
template <typename T, typename SH>
__device__ __forceinline__ void run_g_task(const FusedArgs& p, int slab, int sub, unsigned char* smem, Role& ro) {
    constexpr int cpr = DK / 8;
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool is_prod = warp == 8, is_rows = warp < 4;
    const int head = slab % p.heads;
    const int H = SH::kFixed ? SH::kH : p.H, W = SH::kFixed ? SH::kW : p.W, P = SH::kFixed ? SH::kP : p.p;
    const int N = H * W, n = SH::kFixed ? SH::kP * SH::kP : p.n;
    const int win_h = H / P, win_w = W / P;
    const int gr0 = sub * p.plan.rows_per_g, gr1 = min(H, gr0 + p.plan.rows_per_g);
    const int t_begin = gr0 * W, t_end = gr1 * W;
    const int tiles = (t_end - t_begin + KT - 1) / KT;
    const int steps = (tiles + 1) >> 1;
    const bool has_bias = SH::kFixed ? true : (p.b1 != nullptr);
    const bool bias_tma = has_bias && p.b1_tma;

    const uint32_t ring_u32 = smem_u32(smem + G_RING);
    const uint32_t astack = smem_u32(smem + G_ASTACK), ident = smem_u32(smem + G_IDENT), sP = smem_u32(smem + G_P);
    const T* gQ = static_cast<const T*>(p.q) + (size_t)slab * N * DK;
    const T* gB = has_bias ? static_cast<const T*>(p.b1) + (size_t)head * n * N : nullptr;
    T* gAg = static_cast<T*>(p.ag_ws) + (size_t)slab * RP * DK;     // scale1 * A, rows >= n zero
    T* gAb = static_cast<T*>(p.ab_ws) + (size_t)slab * RP * DK;     // A, rows >= n zero
    const uint32_t tile_tx = 2 * kTile + (bias_tma ? kTile : 0);

    auto fill = [&](int t) {              // producer lane: tile t of the range -> its ring slot
        const int s = t % RING, c0 = t_begin + t * KT;
        const uint32_t bar = bar_addr(ro, BAR_FULL + s), dst = ring_u32 + s * kSlot;
        mbar_arrive_expect_tx(bar, tile_tx);
        tma_load_2d(dst, &p.tm_k, 0, slab * N + c0, bar);
        tma_load_2d(dst + kTile, &p.tm_v, 0, slab * N + c0, bar);
        if (bias_tma) tma_load_2d(dst + 2 * kTile, &p.tm_b1, c0, head * n, bar);
    };

    // ---- phase 0: first ring fills; pooling; identity operand; B1 tiles by plain loads if TMA cannot
    if (is_prod) {
        if (lane == 0)
            for (int t = 0; t < tiles && t < RING; ++t) fill(t);
        __syncwarp();
    } else {
        if (has_bias) {
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
        }
        // pool this range of Q: whole windows, i.e. complete rows of A (text under Eq. 6)
        const int ar0 = gr0 / win_h, ar1 = gr1 / win_h;
        const int nwin = (ar1 - ar0) * P;
        const int cnt = win_h * win_w;
        constexpr int tpl = 32 / cpr;
        const int cg = lane % cpr, tsub = lane / cpr;
        const float inv = 1.f / (float)cnt;
        for (int wi = warp; wi < nwin; wi += NCOMP / 32) {
            const int ay = ar0 + wi / P, ax = wi % P;
            const int y0 = ay * win_h, x0 = ax * win_w;
            float acc[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] = 0.f;
            for (int ib = tsub; ib < cnt; ib += 16 * tpl) {    // sixteen loads in flight per lane
                uint4 raw[16];
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const int i = ib + u * tpl;
                    raw[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (i < cnt) {
                        const int wy = i / win_w, wx = i - wy * win_w;
                        const size_t tok = (size_t)(y0 + wy) * W + (x0 + wx);
                        raw[u] = __ldg(reinterpret_cast<const uint4*>(gQ + tok * DK) + cg);
                    }
                }
#pragma unroll
                for (int u = 0; u < 16; ++u) {
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
                float sc[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) { acc[k] *= inv; sc[k] = acc[k] * p.scale1; }
                *(reinterpret_cast<uint4*>(gAb + (size_t)(ay * P + ax) * DK) + cg) = pack16<T>(acc);
                *(reinterpret_cast<uint4*>(gAg + (size_t)(ay * P + ax) * DK) + cg) = pack16<T>(sc);
            }
        }
        if (sub == 0)                        // padded agent rows are zero in both copies
            for (int e = tid; e < (RP - n) * cpr; e += NCOMP) {
                *(reinterpret_cast<uint4*>(gAb + (size_t)n * DK) + e) = make_uint4(0u, 0u, 0u, 0u);
                *(reinterpret_cast<uint4*>(gAg + (size_t)n * DK) + e) = make_uint4(0u, 0u, 0u, 0u);
            }
    }
    // publish these agent rows, wait for the slab's other G tasks
    publish_add(p.counters + slab);
    wait_counter_block(ro, p.counters + slab, (unsigned)p.plan.g_tasks, kTimeoutAgents);

    // ---- phase 1: the loop over the range
    if (tid == 0) {
        const uint32_t bar = bar_addr(ro, BAR_AG);
        mbar_arrive_expect_tx(bar, 2 * kTile);
        tma_load_2d(astack, &p.tm_ag, 0, slab * RP, bar);
        tma_load_2d(astack + kTile, &p.tm_ag, 0, slab * RP, bar);
    }
    float m_ref = -INFINITY, l = 0.f;
    bool started = false;
    const int half = (tid >> 6) & 1;
    const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
    const uint32_t tO = ro.tmem + TM_GO + 64 * half + lane_base;
    if (is_prod) {
        if (lane == 0) {
            for (int t = RING; t < tiles; ++t) {
                wait_bar(ro, BAR_EMPTY + t % RING, kTimeoutRole);
                fill(t);
            }
            for (int t = max(0, tiles - RING); t < tiles; ++t) wait_bar(ro, BAR_EMPTY + t % RING, kTimeoutRole);
        }
        __syncwarp();
    } else if (is_rows) {
        const uint32_t idK = umma_idesc(fmt, 128, 64, 0), idMN = umma_idesc(fmt, 128, 64, 1);
        auto issue_S = [&](int j) {          // leader: logits of step j (two tiles) -> buffer j & 1
            const int nt2 = min(2, tiles - 2 * j);
            for (int h2 = 0; h2 < nt2; ++h2) wait_bar(ro, BAR_FULL + (2 * j + h2) % RING, kTimeoutTile);
            tc_fence_after_sync();
            for (int h2 = 0; h2 < nt2; ++h2) {
                const uint32_t d = ro.tmem + TM_GS + 128 * (j & 1) + 64 * h2;
                const uint32_t sK = ring_u32 + ((2 * j + h2) % RING) * kSlot, sB = sK + 2 * kTile;
#pragma unroll
                for (int kk = 0; kk < DK / 16; ++kk)
                    umma_f16(d, umma_desc_sw128(astack + kk * 32), umma_desc_sw128(sK + kk * 32), idK, kk > 0);
                if (has_bias) {
#pragma unroll
                    for (int kk = 0; kk < RP / 16; ++kk)
                        umma_f16(d, umma_desc_sw128(ident + kk * 32), umma_desc_sw128(sB + kk * 2048), idMN, 1u);
                }
            }
            umma_commit(bar_addr(ro, BAR_S + (j & 1)));
        };
        wait_bar(ro, BAR_AG, kTimeoutLoads);
        if (tid == 0) issue_S(0);
        for (int j = 0; j < steps; ++j) {
            const int buf = j & 1;
            if (tid == 0 && j + 1 < steps) issue_S(j + 1);
            wait_bar(ro, BAR_S + buf, kTimeoutTile);
            tc_fence_after_sync();
            const int t = 2 * j + half;
            const bool tv = t < tiles;                     // uniform per warp
            uint32_t pk[32];
            float corr = 1.f;
            bool resc = false;
            if (tv) {
                const int valid = min(KT, t_end - (t_begin + t * KT));
                float s[64];
                {
                    uint32_t ra[32], rb[32];
                    const uint32_t ts = ro.tmem + TM_GS + 128 * buf + 64 * half + lane_base;
                    tmem_ld32(ts, ra);
                    tmem_ld32(ts + 32, rb);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 32; ++k) { s[k] = __uint_as_float(ra[k]); s[32 + k] = __uint_as_float(rb[k]); }
                }
                if (valid < KT) {
#pragma unroll
                    for (int k = 0; k < 64; ++k) if (k >= valid) s[k] = -INFINITY;
                }
                float mx = s[0];
#pragma unroll
                for (int k = 1; k < 64; ++k) mx = fmaxf(mx, s[k]);
                if (mx > m_ref + kTau) {                   // also the first tile of the row (m_ref = -inf)
                    corr = fast_exp2((m_ref - mx) * kLog2e);
                    resc = started;
                    m_ref = mx;
                    l *= corr;
                }
                const float nb = -m_ref * kLog2e;
                float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    const float p0 = fast_exp2(fmaf(s[2 * k], kLog2e, nb));       // exp2(-inf) = 0 past the range
                    const float p1 = fast_exp2(fmaf(s[2 * k + 1], kLog2e, nb));
                    sum0 += p0; sum1 += p1;
                    pk[k] = pack2<T>(p0, p1);
                }
                l += sum0 + sum1;
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
                for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<uint4*>(smem + G_P + tid * 128 + ((c ^ (tid & 7)) << 4)) =
                        make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            }
            fence_proxy_async();
            tc_fence_before_sync();
            sync_rows();
            if (tid == 0) {
                tc_fence_after_sync();
                const int nt2 = min(2, tiles - 2 * j);
                for (int h2 = 0; h2 < nt2; ++h2) {
                    const int sl = (2 * j + h2) % RING;
                    const uint32_t sV = ring_u32 + sl * kSlot + kTile;
                    const uint32_t d = ro.tmem + TM_GO + 64 * h2;
#pragma unroll
                    for (int kk = 0; kk < KT / 16; ++kk)
                        umma_f16(d, umma_desc_sw128(sP + kk * 32), umma_desc_sw128(sV + kk * 2048), idMN, (j > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(bar_addr(ro, BAR_EMPTY + sl));
                }
                umma_commit(bar_addr(ro, BAR_PV));
            }
        }
        wait_bar(ro, BAR_PV, kTimeoutTile);
        tc_fence_after_sync();
    }
    __syncthreads();                   // the ring is drained: every MMA of the range has completed

    // ---- phase 2: the two stacked halves combine into one partial state of the range
    const int parts = p.plan.parts;
    const size_t pf = partial_floats(RP, DK);
    float* slab_parts = p.partials + (size_t)slab * parts * pf;
    if (is_rows) {
        float* sX = reinterpret_cast<float*>(smem + G_RING);        // [64][68]: row, m, l of the upper half
        float o[64];
        {
            uint32_t ra[32], rb[32];
            tmem_ld32(tO, ra);
            tmem_ld32(tO + 32, rb);
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                o[k] = started ? __uint_as_float(ra[k]) : 0.f;
                o[32 + k] = started ? __uint_as_float(rb[k]) : 0.f;
            }
        }
        tc_fence_before_sync();
        if (half == 1) {
            float* x = sX + (tid - 64) * 68;
#pragma unroll
            for (int k = 0; k < 16; ++k)
                *reinterpret_cast<float4*>(x + 4 * k) = make_float4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            x[64] = m_ref; x[65] = l;
        }
        sync_rows();
        if (half == 0) {
            const float* x = sX + tid * 68;
            const float om = x[64], ol = x[65];
            const float mm = fmaxf(m_ref, om);
            const float bs = (mm == -INFINITY) ? 0.f : mm;
            const float wa = fast_exp2((m_ref - bs) * kLog2e), wb = fast_exp2((om - bs) * kLog2e);
            float* part = slab_parts + (size_t)sub * pf;
            part[tid] = mm * kLog2e;                       // the merge works in log2 units
            part[RP + tid] = l * wa + ol * wb;
            float* pacc = part + 2 * RP + (size_t)tid * DK;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float4 xv = *reinterpret_cast<const float4*>(x + 4 * k);
                *reinterpret_cast<float4*>(pacc + 4 * k) =
                    make_float4(o[4 * k] * wa + xv.x * wb, o[4 * k + 1] * wa + xv.y * wb,
                                o[4 * k + 2] * wa + xv.z * wb, o[4 * k + 3] * wa + xv.w * wb);
            }
        }
    }
    // when all of the slab's partial states are written, every G task merges its share of the agent
    // rows (fixed order of the parts: bit-reproducible) and counts itself done on the slab's flag
    unsigned* arrived = p.counters + p.slabs + slab;
    publish_add(arrived);
    wait_counter_block(ro, arrived, (unsigned)p.plan.g_tasks, kTimeoutAgents);
    if (!is_prod) {
        const int rows_per = (n + p.plan.g_tasks - 1) / p.plan.g_tasks;
        const int rb = sub * rows_per, re = min(n, rb + rows_per);
        T* va = static_cast<T*>(p.va2_ws) + (size_t)slab * RP * DK;
        for (int e = tid; e < (re - rb) * (DK / 4); e += NCOMP) {
            const int r = rb + e / (DK / 4), c = (e % (DK / 4)) * 4;
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
        if (sub == 0)                        // padded feature rows are zero (0 * NaN is not 0)
            for (int e = tid; e < (RP - n) * cpr; e += NCOMP)
                *(reinterpret_cast<uint4*>(va + (size_t)n * DK) + e) = make_uint4(0u, 0u, 0u, 0u);
    }
    publish_add(p.counters + 2 * p.slabs + slab);
    fence_proxy_async();   // this task's plain shared-memory writes precede the next task's TMA writes
    __syncthreads();
}

// ---------------------------------------------------------------------------------- B task
// A run of broadcast tiles of one slab.  Tile = R whole grid rows (R W <= 128 tokens).  V rows live in
// NSLOT = 2R + 2 row slots of W + 2 tokens (zero columns at x = -1 and x = W): grid row y sits in slot
// (y - y_first + 1) mod NSLOT, so consecutive tiles share their halo rows and only R new rows per tile
// are fetched.
template <typename T, typename SH>
__device__ __forceinline__ void run_b_task(const FusedArgs& p, int slab, int run, unsigned char* smem, Role& ro,
                                           int* s_whead) {
    constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool is_prod = warp == 8, is_rows = warp < 4;
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
    const unsigned char* b2base = has_b2 ? reinterpret_cast<const unsigned char*>(p.b2) + (size_t)head * N * n * 2 : nullptr;
    const size_t b2_total = (size_t)p.heads * N * n * 2;           // bytes of the whole B2 array
    const size_t b2_head_off = (size_t)head * N * n * 2;
    auto slot_of = [&](int y) { return (y - y_first + 1) % NSLOT; };

    if (is_prod) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            poll_counter(ro, p.counters + 2 * p.slabs + slab, (unsigned)p.plan.g_tasks, kTimeoutFeatures);
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
                if (i >= 2) wait_bar(ro, BAR_IN_EMPTY + b, kTimeoutRole);
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
                    if (i >= 2) wait_bar(ro, BAR_V_EMPTY + b, kTimeoutRole);
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
                wait_bar(ro, BAR_IN_EMPTY + (i & 1), kTimeoutRole);
                if (has_dwc) wait_bar(ro, BAR_V_EMPTY + (i & 1), kTimeoutRole);
            }
        }
        __syncwarp();
    } else if (is_rows) {
        // ------------------------------------------------------------------ row group
        const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;
        const uint32_t idK = umma_idesc(fmt, 128, 64, 0), idMN = umma_idesc(fmt, 128, 64, 1);
        const uint32_t sA = smem_u32(smem + B_A), sVA = smem_u32(smem + B_VA), sP = smem_u32(smem + B_P);
        auto issue_S = [&](int i) {
            const int b = i & 1;
            wait_bar(ro, BAR_IN_FULL + b, kTimeoutLoads);
            tc_fence_after_sync();
            const uint32_t sQ = smem_u32(smem + B_Q + b * 2 * kTile);
#pragma unroll
            for (int kk = 0; kk < DK / 16; ++kk)
                umma_f16(ro.tmem + TM_BS + 64 * b, umma_desc_sw128(sQ + kk * 32), umma_desc_sw128(sA + kk * 32), idK, kk > 0);
            umma_commit(bar_addr(ro, BAR_S + b));
        };
        wait_bar(ro, BAR_AG, kTimeoutLoads);
        if (tid == 0) issue_S(0);
        for (int i = 0; i < nt; ++i) {
            const int b = i & 1;
            const int y0 = y_first + i * R, rows = min(R, H - y0);
            const int q0 = y0 * W, TQ = rows * W;
            if (tid == 0 && i + 1 < nt) issue_S(i + 1);
            wait_bar(ro, BAR_S + b, kTimeoutLoads);
            tc_fence_after_sync();
            float s[64];
            {
                uint32_t ra[32], rb[32];
                const uint32_t ts = ro.tmem + TM_BS + 64 * b + lane_base;
                tmem_ld32(ts, ra);
                tmem_ld32(ts + 32, rb);
                tmem_ld_wait();
#pragma unroll
                for (int k = 0; k < 32; ++k) { s[k] = __uint_as_float(ra[k]); s[32 + k] = __uint_as_float(rb[k]); }
            }
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
                // element index of this row's first bias value inside the buffer (the copy starts at a 16-byte boundary)
                const uint32_t e0 = (uint32_t)(((b2_head_off + (size_t)q0 * n * 2) & 15) >> 1) + (uint32_t)tid * n;
                const uint32_t* w32 = reinterpret_cast<const uint32_t*>(smem + B_B2 + b * kB2Buf) + (e0 >> 1);
                const int sh = (e0 & 1) * 16;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (2 * j < n) {
                        const float2 bb = unpack2<T>(__funnelshift_r(w32[j], w32[j + 1], sh));
                        s[2 * j] = fmaf(s[2 * j], p.scale2, bb.x);
                        s[2 * j + 1] = (2 * j + 1 < n) ? fmaf(s[2 * j + 1], p.scale2, bb.y) : -INFINITY;
                        mx = fmaxf(mx, fmaxf(s[2 * j], s[2 * j + 1]));
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (2 * j < n) {
                        s[2 * j] = s[2 * j] * p.scale2;
                        s[2 * j + 1] = (2 * j + 1 < n) ? s[2 * j + 1] * p.scale2 : -INFINITY;
                        mx = fmaxf(mx, fmaxf(s[2 * j], s[2 * j + 1]));
                    }
                }
            }
            mbar_arrive(bar_addr(ro, BAR_IN_EMPTY + b));     // the Q tile and this row's bias values are consumed
            const float nm = -mx * kLog2e;
            float l0 = 0.f, l1 = 0.f;
            uint32_t pk[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                if (2 * j < n) {
                    const float p0 = fast_exp2(fmaf(s[2 * j], kLog2e, nm));
                    const float p1 = fast_exp2(fmaf(s[2 * j + 1], kLog2e, nm));      // exp2(-inf) = 0 past the last agent
                    pk[j] = pack2<T>(p0, p1);
                    const float2 q = unpack2<T>(pk[j]);    // the normaliser sums the rounded weights
                    l0 += q.x; l1 += q.y;
                } else {
                    pk[j] = 0u;
                }
            }
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(smem + B_P + tid * 128 + ((c ^ (tid & 7)) << 4)) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            fence_proxy_async();
            tc_fence_before_sync();
            sync_rows();
            if (tid == 0) {
                tc_fence_after_sync();
                for (int kk = 0; kk < n16; ++kk)
                    umma_f16(ro.tmem + TM_BO + 64 * b, umma_desc_sw128(sP + kk * 32), umma_desc_sw128(sVA + kk * 2048), idMN, kk > 0);
                umma_commit(bar_addr(ro, BAR_PV));
            }
            wait_bar(ro, BAR_PV, kTimeoutLoads);
            tc_fence_after_sync();
            if (i >= 2) wait_bar(ro, BAR_PATCH_EMPTY + b, kTimeoutRole);
            {
                const float inv = 1.f / (l0 + l1);
                float* prow = reinterpret_cast<float*>(smem + B_PATCH + b * kPatch) + tid * PO;
                uint32_t ra[32], rb[32];
                const uint32_t to = ro.tmem + TM_BO + 64 * b + lane_base;
                tmem_ld32(to, ra);
                tmem_ld32(to + 32, rb);
                tmem_ld_wait();
                if (tid < TQ) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        *reinterpret_cast<float4*>(prow + 4 * k) =
                            make_float4(__uint_as_float(ra[4 * k]) * inv, __uint_as_float(ra[4 * k + 1]) * inv,
                                        __uint_as_float(ra[4 * k + 2]) * inv, __uint_as_float(ra[4 * k + 3]) * inv);
                        *reinterpret_cast<float4*>(prow + 32 + 4 * k) =
                            make_float4(__uint_as_float(rb[4 * k]) * inv, __uint_as_float(rb[4 * k + 1]) * inv,
                                        __uint_as_float(rb[4 * k + 2]) * inv, __uint_as_float(rb[4 * k + 3]) * inv);
                    }
                }
                tc_fence_before_sync();
            }
            mbar_arrive(bar_addr(ro, BAR_PATCH_FULL + b));
        }
        for (int i = max(0, nt - 2); i < nt; ++i) wait_bar(ro, BAR_PATCH_EMPTY + (i & 1), kTimeoutRole);
    } else {
        // ------------------------------------------------------------------ stencil group
        const int t2 = tid - 128;
        if (has_dwc) {
            // zero columns x = -1 and x = W of every slot; the row above the grid if the run starts the slab
            for (int e = t2; e < NSLOT * 2 * (DK / 8); e += 128) {
                const int sl = e / (2 * (DK / 8)), rest = e - sl * 2 * (DK / 8);
                const int side = rest / (DK / 8), c = rest - side * (DK / 8);
                *(reinterpret_cast<uint4*>(sV + ((size_t)sl * HP + (side ? W + 1 : 0)) * DK) + c) = make_uint4(0, 0, 0, 0);
            }
            if (y_first == 0)
                for (int e = t2; e < W * (DK / 8); e += 128) *(reinterpret_cast<uint4*>(sV + DK) + e) = make_uint4(0, 0, 0, 0);
            if (ld_shared_volatile(s_whead) != head) {       // filter taps change only with the head
                const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * DK * 9;
                for (int e = t2; e < 9 * DK; e += 128) {
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
                    for (int e = t2; e < W * (DK / 8); e += 128) *(reinterpret_cast<uint4*>(z) + e) = make_uint4(0, 0, 0, 0);
                    sync_stencil();
                }
            }
            wait_bar(ro, BAR_PATCH_FULL + b, kTimeoutRole);
            // depthwise 3x3 term + store: thread = (tile row r, 4-channel group cq, x-segment)
            {
                constexpr int NCQ = DK / 4;
                const float* sPatch = reinterpret_cast<const float*>(smem + B_PATCH + b * kPatch);
                const int npairs = rows * NCQ;
                int nseg = 128 / npairs;
                if (nseg < 1) nseg = 1;
                if (nseg > W) nseg = W;
                const int seg_len = (W + nseg - 1) / nseg;
                T* gO = static_cast<T*>(p.out) + ((size_t)slab * N + q0) * DK;
                for (int item = t2; item < npairs * nseg; item += 128) {
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
    fence_proxy_async();   // this task's plain shared-memory writes precede the next task's TMA writes
    __syncthreads();       // shared memory is free for the next task
}

// ---------------------------------------------------------------------------------- kernel
template <typename T, typename SH>
__global__ void __launch_bounds__(NT, 1) fused2_kernel(const __grid_constant__ FusedArgs p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_task, s_whead, s_dead;
    __shared__ uint32_t s_tmem;
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x;
    Role ro;
    ro.status = p.status;
    ro.dead = &s_dead;
    ro.bars = smem_u32(smem + OFF_BAR);
    ro.ph = 0u;
    if (tid == 0) {
        s_whead = -1;
        s_dead = 0;
        for (int i = 0; i < kBarsUsed; ++i) {
            const bool many = (i >= BAR_IN_EMPTY && i < BAR_V_FULL) || i >= BAR_V_EMPTY;   // arrivals by a whole group
            mbar_init(ro.bars + 8 * i, many ? 128u : 1u);
        }
        mbar_fence_init();
    }
    if (tid < 32) tmem_alloc<512>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    ro.tmem = s_tmem;
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
        if (is_g) run_g_task<T, SH>(p, slab, sub, smem, ro);
        else      run_b_task<T, SH>(p, slab, sub, smem, ro, &s_whead);
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
