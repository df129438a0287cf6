// The whole module of Eq. 6 in one persistent kernel, for small agent counts (n <= 64, d = 64).
//
// Why one kernel: the path reads Q twice (pooling, broadcast) and V twice (aggregation, DWC).
// Run phase by phase over a large batch, the second reads come from HBM.  Here resident blocks
// pull tasks from a queue ordered slab by slab, so a slab's second reads follow its first ones
// within microseconds and are served by L2; HBM sees every input once.
//
//   G task (slab, range of grid rows): start the K/V/B1 tile ring (TMA, 128-byte swizzle), pool Q
//     over the range (whole pooling windows: complete agent rows), publish them, wait until the
//     slab's other G tasks have published theirs, then run the split aggregation over the range
//     (Eq. 3, Eq. 5).  When all G tasks of the slab have written their partial states, each merges
//     its share of the agent rows into V_A and counts itself done on the slab's flag.
//   B task (slab, tile of whole grid rows, <= 128 tokens): start the bulk copies of the V rows
//     (with their 3x3 halo) and of the B2 tile, load Q fragments straight into registers, wait for
//     the slab's flag, fetch A and V_A (TMA), then broadcast + DWC (Eq. 3, Eq. 5, Eq. 6).
//
// Every wait is bounded: flag polls and mbarrier waits give up after a fixed number of tries,
// record a code in the status word and carry on (the result is then wrong, but nothing hangs).
// Queue order guarantees progress: a task only waits for tasks that precede it or for its own
// slab's G siblings, which are adjacent in the queue, and the grid holds at least as many
// resident blocks as a slab has G tasks.  No TMA multicast is used.
#pragma once
#include "common.cuh"
#include "kernels.h"
#include "merge.cuh"
#include "tma.cuh"
#include "umma.cuh"

namespace aa {

namespace {
constexpr int DK = 64;            // head dim handled by this kernel
constexpr int KT = 64;            // tokens per aggregation tile
constexpr int QT = 128;           // most tokens per broadcast tile
constexpr int NT = 256;           // threads per block (8 warps)
constexpr int RP = 64;            // agent rows, padded
constexpr int STAGES = 3;
constexpr int MAXW = 64;          // widest grid the V-row buffer is sized for
constexpr int MINW = 8;
constexpr int kHaloTokens = 264;  // max over 8 <= W <= 64 of (R + 2)(W + 2), R = min(16, 128 / W)
constexpr unsigned kSpinLimit = 1u << 20;      // flag polls
constexpr unsigned kBarLimit = 1u << 22;       // mbarrier try_wait attempts
constexpr int kTimeoutAgents = 1, kTimeoutFeatures = 2, kTimeoutTile = 3, kTimeoutLoads = 4;

// shared-memory map (bytes from a 1024-byte aligned base)
constexpr int kTileBytes = KT * 128;                    // one swizzled 64 x 64 tile of 16-bit elements
constexpr int OFF_A = 0;                                // resident agents A            [64][128 B] swizzled
constexpr int OFF_VA = OFF_A + kTileBytes;              // resident agent features V_A  [64][128 B] swizzled
constexpr int OFF_W = OFF_VA + kTileBytes;              // filter taps [9][64] fp32
constexpr int OFF_UNION = 19456;                        // 19 KiB: start of the per-task area
// G tasks: ring of STAGES x (K tile | V tile | B1 tile)
constexpr int kStageBytes = 3 * kTileBytes;
constexpr int kGBytes = STAGES * kStageBytes;
// B tasks: fp32 patch | V rows with zero borders | B2 tile
constexpr int PO = DK + 4;                              // patch pitch (floats): row-per-thread 16-byte stores spread over all banks
constexpr int OFF_PATCH = OFF_UNION;
constexpr int kPatchBytes = QT * PO * 4;
constexpr int OFF_HALO = OFF_PATCH + kPatchBytes;
constexpr int kHaloBytes = kHaloTokens * DK * 2;
constexpr int OFF_B2 = OFF_HALO + kHaloBytes;
constexpr int kB2Bytes = QT * RP * 2 + 16;              // + one spare vector: pairs are read as two words
constexpr int kBBytes = kPatchBytes + kHaloBytes + kB2Bytes;
constexpr int OFF_BAR = OFF_UNION + (kGBytes > kBBytes ? kGBytes : kBBytes);   // mbarriers (8 bytes each)
constexpr int kNumBars = STAGES + 4;                    // ring stages, agents, Q tile, MMA completion, V rows + B2 tile
constexpr int kTmemCols = 128;                          // per block: 64 columns of logits + 64 of output
static_assert(kPatchBytes >= 2 * QT * 128, "the Q and P operand tiles alias the patch");
constexpr int kSmemBytes = OFF_BAR + 8 * kNumBars + 1024;   // + slack to align the base to 1024
static_assert(OFF_W + 9 * DK * 4 <= OFF_UNION, "common area overflows");
static_assert(OFF_UNION % 1024 == 0 && kStageBytes % 1024 == 0 && OFF_BAR % 8 == 0, "alignment");

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// The calling thread polls until *ctr >= target; gives up after `limit` polls and records `code`.
__device__ __forceinline__ void poll_counter(const unsigned* ctr, unsigned target, int* status, int code, unsigned limit) {
    unsigned spins = 0;
    while (ld_acquire(ctr) < target) {
        if (++spins > limit) { atomicExch(status, code); break; }
        // once any block has given up, the others stop waiting too
        if ((spins & 255u) == 0 && ld_acquire(reinterpret_cast<const unsigned*>(status)) != 0u) break;
        __nanosleep(40);
    }
}
// Thread 0 polls, then a block barrier passes the result on.
__device__ __forceinline__ void wait_counter(const unsigned* ctr, unsigned target, int* status, int code, unsigned limit) {
    if (threadIdx.x == 0) poll_counter(ctr, target, status, code, limit);
    __syncthreads();
}
// Publish: all of this block's prior global writes become visible before the counter moves.
__device__ __forceinline__ void publish_add(unsigned* ctr) {
    __syncthreads();
    if (threadIdx.x == 0) { __threadfence(); atomicAdd(ctr, 1u); }
}
// Thread 0 waits (bounded, with back-off so that it does not eat issue slots) for a phase of an
// mbarrier; the caller follows with __syncthreads(), which passes the completed copies on to the
// rest of the block.  On expiry the block records `code` and goes on.
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, int* status, int code) {
    if (threadIdx.x == 0) {
        unsigned tries = 0;
        while (!mbar_try_wait(bar, parity)) {
            if (++tries > kBarLimit) { atomicExch(status, code); break; }
            __nanosleep(32);
        }
    }
}
// Every thread waits (bounded) for a phase of an mbarrier itself, parked by the suspended form of try_wait: no
// block barrier is needed to pass the completion on.  On expiry the thread records `code` and goes on.
__device__ __forceinline__ void wait_bar_all(uint32_t bar, uint32_t parity, int* status, int code) {
    if (mbar_try_wait_suspend(bar, parity, 2000u)) return;
    for (unsigned tries = 0; tries < (1u << 20); ++tries)
        if (mbar_try_wait_suspend(bar, parity, 2000u)) return;
    atomicExch(status, code);
}
// Byte offset of element (row, col) in a swizzled [rows][64] tile of 16-bit elements: the 16-byte
// chunk index is XORed with the row index modulo 8 (the TMA 128-byte swizzle).
__device__ __forceinline__ int swz(int row, int col) {
    return row * 128 + ((((col >> 3) ^ row) & 7) << 4) + (col & 7) * 2;
}

// Tile of `box` tokens from token `tok` of slab (b, head): a 2-D map over [slabs * N][d] when the tensor is
// dense (rows past the slab then belong to the next slab: the readers mask them), else the 4-D strided map.
__device__ __forceinline__ void load_tokens(uint32_t dst, const CUtensorMap* map, int dense, int head_first, int tok,
                                            int head, int b, int row0, uint32_t bar) {
    if (dense) tma_load_2d(dst, map, 0, row0 + tok, bar);
    else tma_load_tok(dst, map, head_first, tok, head, b, bar);
}

// Flat global -> shared copy of `bytes` (a multiple of 2) by plain loads: the fallback when a
// bulk copy's alignment rules do not hold.
__device__ __forceinline__ void copy_flat(unsigned char* dst, const unsigned char* src, int bytes, int tid) {
    for (int i = 2 * tid; i < bytes; i += 2 * NT)
        *reinterpret_cast<unsigned short*>(dst + i) = *reinterpret_cast<const unsigned short*>(src + i);
}

// Block-level state that persists across tasks: mbarrier phase parities.
struct BlockState {
    uint32_t bar_base;          // shared address of the first mbarrier
    uint32_t ph;                // parity to wait for next: bit s = ring stage s, then agents, broadcast inputs, MMA
    uint32_t tmem;              // base address of this block's tensor-memory columns
};
constexpr int kBitAgents = STAGES, kBitBin = STAGES + 1, kBitMma = STAGES + 2, kBitVb = STAGES + 3;
__device__ __forceinline__ uint32_t bar_full(const BlockState& st, int s) { return st.bar_base + 8 * s; }
__device__ __forceinline__ uint32_t bar_agents(const BlockState& st) { return st.bar_base + 8 * STAGES; }
__device__ __forceinline__ uint32_t bar_bin(const BlockState& st) { return st.bar_base + 8 * (STAGES + 1); }
__device__ __forceinline__ uint32_t bar_mma(const BlockState& st) { return st.bar_base + 8 * (STAGES + 2); }
__device__ __forceinline__ uint32_t bar_vb(const BlockState& st) { return st.bar_base + 8 * (STAGES + 3); }
// barrier among the 128 threads of warps 0-3 (the threads that own TMEM lanes in the broadcast)
__device__ __forceinline__ void sync_rows() { asm volatile("bar.sync 1, 128;\n" ::: "memory"); }
}  // namespace

// Compile-time shape: a kernel instantiated for one token grid and agent grid (with biases and the
// depthwise term present) folds its index arithmetic and loop bounds; 0 means "read it from the
// arguments".  The generic kernel uses ShapeAny.
template <int H_, int W_, int P_, bool DENSE_ = true> struct FusedShape {
    static constexpr int kH = H_, kW = W_, kP = P_;
    static constexpr bool kFixed = (H_ > 0);
    static constexpr bool kDense = kFixed && DENSE_;     // dense [B][heads][N][d] tensors: constant strides, 2-D maps
};
using ShapeAny = FusedShape<0, 0, 0, false>;

// ---------------------------------------------------------------------------------- G task
template <typename T, typename SH>
__device__ __forceinline__ void run_g_task(const FusedArgs& p, int slab, int sub, unsigned char* smem,
                                           BlockState& st, int* s_flag, int& next_task) {
    constexpr int NWK = 2, KW = KT / NWK;
    constexpr int cpr = DK / 8;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp & 3, wk = warp >> 2;
    const int head = slab % p.heads;
    const int H = SH::kFixed ? SH::kH : p.H, W = SH::kFixed ? SH::kW : p.W, P = SH::kFixed ? SH::kP : p.p;
    const int N = H * W, n = SH::kFixed ? SH::kP * SH::kP : p.n;
    const int win_h = H / P, win_w = W / P;
    const int gr0 = sub * p.plan.rows_per_g, gr1 = min(H, gr0 + p.plan.rows_per_g);
    const int t_begin = gr0 * W, t_end = gr1 * W;
    const int tiles = (t_end - t_begin + KT - 1) / KT;
    const bool has_bias = SH::kFixed ? true : (p.b1 != nullptr);
    const bool bias_tma = has_bias && p.b1_tma;

    unsigned char* sA = smem + OFF_A;
    unsigned char* ring = smem + OFF_UNION;
    const uint32_t ring_u32 = smem_u32(ring);
    // the shape-specialised kernels serve dense tensors only: their strides are compile-time constants
    const T* gQ = static_cast<const T*>(p.q) + (SH::kDense ? (long long)slab * N * DK : tok_offset(p.lin, slab, p.heads, 0));
    const size_t sq = SH::kDense ? (size_t)DK : (size_t)p.lin.st;     // token stride of Q, K and V
    const T* gB = has_bias ? static_cast<const T*>(p.b1) + (size_t)head * n * N : nullptr;
    T* gA = static_cast<T*>(p.a_ws) + (size_t)slab * n * DK;
    const uint32_t tile_tx = 2 * kTileBytes + (bias_tma ? kTileBytes : 0);

    // tile t of this range -> ring stage s: K and V rows, and the B1 columns of the same tokens
    auto issue_tile = [&](int t, int s) {
        const int c0 = t_begin + t * KT;
        if (tid == 0) {
            const uint32_t bar = bar_full(st, s), dst = ring_u32 + s * kStageBytes;
            mbar_arrive_expect_tx(bar, tile_tx);
            load_tokens(dst, &p.tm_k, SH::kDense ? 1 : p.dense_in, p.hf_k, c0, head, slab / p.heads, slab * N, bar);
            load_tokens(dst + kTileBytes, &p.tm_v, SH::kDense ? 1 : p.dense_in, p.hf_v, c0, head, slab / p.heads, slab * N, bar);
            if (bias_tma) tma_load_2d(dst + 2 * kTileBytes, &p.tm_b1, c0, head * n, bar);
        }
        if (has_bias && !bias_tma) {       // B1 rows not 16-byte aligned: plain loads into the same layout
            unsigned char* sB = ring + s * kStageBytes + 2 * kTileBytes;
            for (int e = tid; e < n * KT; e += NT) {
                const int r = e / KT, j = e - r * KT;
                const int key = c0 + j;
                *reinterpret_cast<T*>(sB + swz(r, j)) = key < t_end ? gB[(size_t)r * N + key] : Elem<T>::from_f32(0.f);
            }
        }
    };
    // 1. start the ring
    for (int s = 0; s < STAGES - 1; ++s)
        if (s < tiles) issue_tile(s, s);

    // 2. pool this range of Q: whole windows, i.e. complete rows of A (text under Eq. 6)
    {
        const int ar0 = gr0 / win_h, ar1 = gr1 / win_h;
        const int nwin = (ar1 - ar0) * P;
        const int cnt = win_h * win_w;
        constexpr int tpl = 32 / cpr;
        const int cg = lane % cpr, tsub = lane / cpr;
        const float inv = 1.f / (float)cnt;
        // windows of at most four tokens (one load per lane): eight windows of the warp in flight at once,
        // so that their load latencies overlap instead of adding up
        for (int w0 = warp; cnt <= tpl && w0 < nwin; w0 += 8 * (NT / 32)) {
            uint4 raw[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int wi = w0 + u * (NT / 32);
                raw[u] = make_uint4(0u, 0u, 0u, 0u);
                if (wi < nwin && tsub < cnt) {
                    const int ay = ar0 + wi / P, ax = wi % P;
                    const int wy = tsub / win_w, wx = tsub - wy * win_w;
                    const size_t tok = (size_t)(ay * win_h + wy) * W + (ax * win_w + wx);
                    raw[u] = __ldg(reinterpret_cast<const uint4*>(gQ + tok * sq) + cg);
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int wi = w0 + u * (NT / 32);
                if (wi >= nwin) break;                       // uniform over the warp
                float acc[8];
                unpack16<T>(raw[u], acc);
#pragma unroll
                for (int o = cpr; o < 32; o <<= 1) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], o);
                }
                if (tsub == 0) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] *= inv;
                    *(reinterpret_cast<uint4*>(gA + (size_t)((ar0 + wi / P) * P + wi % P) * DK) + cg) = pack16<T>(acc);
                }
            }
        }
        for (int wi = warp; cnt > tpl && wi < nwin; wi += NT / 32) {
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
                        raw[u] = __ldg(reinterpret_cast<const uint4*>(gQ + tok * sq) + cg);
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
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] *= inv;
                *(reinterpret_cast<uint4*>(gA + (size_t)(ay * P + ax) * DK) + cg) = pack16<T>(acc);
            }
        }
    }
    // 3. publish these agent rows, wait for the slab's other G tasks
    publish_add(p.counters + slab);
    wait_counter(p.counters + slab, (unsigned)p.plan.g_tasks, p.status, kTimeoutAgents, p.poll_limit);
    // 4. all agents of the slab -> shared memory (rows >= n receive foreign rows; they only feed
    //    padded agent rows, which are never merged)
    if (tid == 0) {
        fence_proxy_async_all();       // the siblings' agent rows were written with plain stores
        mbar_arrive_expect_tx(bar_agents(st), kTileBytes);
        tma_load_2d(smem_u32(sA), &p.tm_a, 0, slab * n, bar_agents(st));
    }
    wait_bar(bar_agents(st), (st.ph >> kBitAgents) & 1u, p.status, kTimeoutLoads);
    st.ph ^= 1u << kBitAgents;
    __syncthreads();

    const int g = lane >> 2, t4 = lane & 3, xr = lane & 7;
    const int r0 = wm * 16, kw0 = wk * KW;
    uint32_t af[DK / 16][4];
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks)
        ldmatrix_x4(af[ks][0], af[ks][1], af[ks][2], af[ks][3],
                    sA + (r0 + xr + ((lane >> 3) & 1) * 8) * 128 + (((ks * 2 + (lane >> 4)) ^ xr) << 4));
    // B fragment that is 1 in column 0: one more MMA per key block yields the row sums of P
    const uint32_t ones = (g == 0) ? pack2<T>(1.f, 1.f) : 0u;

    float m0 = -INFINITY, m1 = -INFINITY;            // running row maxima, natural units
    float acc[DK / 8][4], accl[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < DK / 8; ++j) { acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f; }
    // 5. online-softmax aggregation over the range
    for (int it = 0; it < tiles; ++it) {
        const int s = it % STAGES;
        wait_bar(bar_full(st, s), (st.ph >> s) & 1u, p.status, kTimeoutTile);
        st.ph ^= 1u << s;
        __syncthreads();               // tile `it` has landed, and every warp is done with tile it-1
        if (it + STAGES - 1 < tiles) issue_tile(it + STAGES - 1, (it + STAGES - 1) % STAGES);
        const unsigned char* sK = ring + s * kStageBytes;
        const unsigned char* sV = sK + kTileBytes;
        const unsigned char* sB = sV + kTileBytes;
        const int c0 = t_begin + it * KT;
        if (c0 + KT > t_end) {
            // ragged last tile: the rows past the range belong to the next range or slab; their weights are 0, and
            // 0 * NaN is not 0, so the V rows are cleared before the product
            unsigned char* vz = ring + s * kStageBytes + kTileBytes;
            for (int e = tid; e < (c0 + KT - t_end) * 8; e += NT)
                *(reinterpret_cast<uint4*>(vz + (t_end - c0 + (e >> 3)) * 128) + (e & 7)) = make_uint4(0u, 0u, 0u, 0u);
            __syncthreads();
        }

        float sc[KW / 8][4];
#pragma unroll
        for (int j = 0; j < KW / 8; ++j) { sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < DK / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < KW / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3,
                            sK + (kw0 + np * 16 + xr + (lane >> 4) * 8) * 128 + (((ks * 2 + ((lane >> 3) & 1)) ^ xr) << 4));
                mma16816<T>(sc[2 * np], af[ks], b0, b1);
                mma16816<T>(sc[2 * np + 1], af[ks], b2, b3);
            }
        }
        // logits in natural units: t = scale1 * a.k + b1
#pragma unroll
        for (int j = 0; j < KW / 8; ++j) {
            float2 ba = make_float2(0.f, 0.f), bb = make_float2(0.f, 0.f);
            if (has_bias) {
                const int cb = (((kw0 >> 3) + j) ^ g) << 4;      // rows r0+g and r0+g+8 share row % 8 = g
                ba = unpack2<T>(*reinterpret_cast<const uint32_t*>(sB + (r0 + g) * 128 + cb + t4 * 4));
                bb = unpack2<T>(*reinterpret_cast<const uint32_t*>(sB + (r0 + g + 8) * 128 + cb + t4 * 4));
            }
            sc[j][0] = fmaf(sc[j][0], p.scale1, ba.x);
            sc[j][1] = fmaf(sc[j][1], p.scale1, ba.y);
            sc[j][2] = fmaf(sc[j][2], p.scale1, bb.x);
            sc[j][3] = fmaf(sc[j][3], p.scale1, bb.y);
        }
        if (c0 + KT > t_end) {          // ragged last tile of the range: keys beyond it do not belong to it
#pragma unroll
            for (int j = 0; j < KW / 8; ++j) {
                const int key = c0 + kw0 + 8 * j + 2 * t4;
                if (key >= t_end)     { sc[j][0] = -INFINITY; sc[j][2] = -INFINITY; }
                if (key + 1 >= t_end) { sc[j][1] = -INFINITY; sc[j][3] = -INFINITY; }
            }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int j = 0; j < KW / 8; ++j) {
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
        const float nb0 = -base0 * kLog2e, nb1 = -base1 * kLog2e;
        // rescale the running state only when some row of the warp saw a new maximum
        if (__any_sync(0xffffffffu, (mn0 != m0) || (mn1 != m1))) {
            const float corr0 = fast_exp2(fmaf(m0, kLog2e, nb0)), corr1 = fast_exp2(fmaf(m1, kLog2e, nb1));
            accl[0] *= corr0; accl[2] *= corr1;
#pragma unroll
            for (int j = 0; j < DK / 8; ++j) {
                acc[j][0] *= corr0; acc[j][1] *= corr0; acc[j][2] *= corr1; acc[j][3] *= corr1;
            }
        }
        m0 = mn0; m1 = mn1;
        // probabilities rounded to the operand type; their row sums come out of one more MMA
        uint32_t pk[KW / 8][2];
#pragma unroll
        for (int j = 0; j < KW / 8; ++j) {
            pk[j][0] = pack2<T>(fast_exp2(fmaf(sc[j][0], kLog2e, nb0)), fast_exp2(fmaf(sc[j][1], kLog2e, nb0)));
            pk[j][1] = pack2<T>(fast_exp2(fmaf(sc[j][2], kLog2e, nb1)), fast_exp2(fmaf(sc[j][3], kLog2e, nb1)));
        }
#pragma unroll
        for (int kk = 0; kk < KW / 16; ++kk) {
            const uint32_t pa[4] = {pk[2 * kk][0], pk[2 * kk][1], pk[2 * kk + 1][0], pk[2 * kk + 1][1]};
#pragma unroll
            for (int np = 0; np < DK / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(b0, b1, b2, b3,
                                  sV + (kw0 + kk * 16 + xr + ((lane >> 3) & 1) * 8) * 128 + (((np * 2 + (lane >> 4)) ^ xr) << 4));
                mma16816<T>(acc[2 * np], pa, b0, b1);
                mma16816<T>(acc[2 * np + 1], pa, b2, b3);
            }
            mma16816<T>(accl, pa, ones, ones);
        }
    }
    __syncthreads();                   // every warp is done with the ring

    // row sums sit in column 0 of the extra product: lanes with t4 == 0 hold them
    const float l0 = __shfl_sync(0xffffffffu, accl[0], lane & ~3);
    const float l1 = __shfl_sync(0xffffffffu, accl[2], lane & ~3);
    // 6. the two key halves of the block combine through shared memory into one partial state;
    float* sX = reinterpret_cast<float*>(ring);        // [4 row groups][36 values][32 lanes]
    if (wk == 1) {
        float* x = sX + wm * 36 * 32 + lane;
        x[0] = m0; x[32] = m1; x[64] = l0; x[96] = l1;
#pragma unroll
        for (int j = 0; j < DK / 8; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) x[(4 + 4 * j + e) * 32] = acc[j][e];
        }
    }
    __syncthreads();
    const int parts = p.plan.parts;
    const size_t pf = partial_floats(RP, DK);
    float* slab_parts = p.partials + (size_t)slab * parts * pf;
    if (wk == 0) {
        const float* x = sX + wm * 36 * 32 + lane;
        const float om0 = x[0], om1 = x[32];
        const float mm0 = fmaxf(m0, om0), mm1 = fmaxf(m1, om1);
        const float bs0 = (mm0 == -INFINITY) ? 0.f : mm0, bs1 = (mm1 == -INFINITY) ? 0.f : mm1;
        const float wa0 = fast_exp2((m0 - bs0) * kLog2e), wb0 = fast_exp2((om0 - bs0) * kLog2e);
        const float wa1 = fast_exp2((m1 - bs1) * kLog2e), wb1 = fast_exp2((om1 - bs1) * kLog2e);
        float* part = slab_parts + (size_t)sub * pf;
        if (t4 == 0) {
            part[r0 + g] = mm0 * kLog2e; part[r0 + g + 8] = mm1 * kLog2e;     // the merge works in log2 units
            part[RP + r0 + g] = l0 * wa0 + x[64] * wb0;
            part[RP + r0 + g + 8] = l1 * wa1 + x[96] * wb1;
        }
        float* pacc = part + 2 * RP;
#pragma unroll
        for (int j = 0; j < DK / 8; ++j) {
            const int col = 8 * j + 2 * t4;
            *reinterpret_cast<float2*>(pacc + (size_t)(r0 + g) * DK + col) =
                make_float2(acc[j][0] * wa0 + x[(4 + 4 * j) * 32] * wb0, acc[j][1] * wa0 + x[(5 + 4 * j) * 32] * wb0);
            *reinterpret_cast<float2*>(pacc + (size_t)(r0 + g + 8) * DK + col) =
                make_float2(acc[j][2] * wa1 + x[(6 + 4 * j) * 32] * wb1, acc[j][3] * wa1 + x[(7 + 4 * j) * 32] * wb1);
        }
    }
    // 7. when all of the slab's partial states are written, every G task merges its share of the
    //    agent rows (fixed order of the parts: bit-reproducible) and counts itself done
    unsigned* arrived = p.counters + p.slabs + slab;
    publish_add(arrived);
    wait_counter(arrived, (unsigned)p.plan.g_tasks, p.status, kTimeoutAgents, p.poll_limit);
    // no wait lies ahead in this task: take the next ticket now, so that the queue's round trip runs under the merge
    if (tid == 0) next_task = (int)atomicAdd(p.counters + 3 * (size_t)p.slabs, 1u);
    {
        const int rows_per = (n + p.plan.g_tasks - 1) / p.plan.g_tasks;
        const int rb = sub * rows_per, re = min(n, rb + rows_per);
        T* va = static_cast<T*>(p.va_ws) + (size_t)slab * n * DK;
        for (int e = tid; e < (re - rb) * (DK / 4); e += NT) {
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
    }
    publish_add(p.counters + 2 * p.slabs + slab);
    // (the caller closes the task: proxy fence and block barrier, after which the ring is free)
}

// ---------------------------------------------------------------------------------- B task
// One tile = R whole grid rows (R*W <= 128 tokens).  Warps own 16 query rows each for the attention
// part and leave their fp32 result in the patch; then all threads switch to a (row, 4-channel
// group, x-segment) mapping and slide a 3x3 window along x over the V rows held in shared memory
// (with explicit zero columns at x = -1 and x = W and zero rows outside the grid), add the
// depthwise term (Eq. 6), round once and store.
template <typename T, typename SH>
__device__ __forceinline__ void run_b_task(const FusedArgs& p, int slab, int tile, unsigned char* smem,
                                           BlockState& st, int* s_whead, float (*s_red)[128], int& next_task) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int head = slab % p.heads;
    const int H = SH::kFixed ? SH::kH : p.H, W = SH::kFixed ? SH::kW : p.W;
    const int N = H * W, n = SH::kFixed ? SH::kP * SH::kP : p.n;
    const int n16 = (n + 15) >> 4;
    const int R = SH::kFixed ? (QT / SH::kW > 16 ? 16 : (QT / SH::kW > SH::kH ? SH::kH : QT / SH::kW)) : p.plan.rows_per_b;
    const int y0 = tile * R;
    const int rows = min(R, H - y0);
    const int q0 = y0 * W, TQ = rows * W;            // tokens of this tile
    const bool has_dwc = SH::kFixed ? true : (p.dwc_w != nullptr);
    const bool has_b2 = SH::kFixed ? true : (p.b2 != nullptr);
    const int HP = W + 2;                             // V-row pitch in tokens (zero columns at both ends)
    unsigned char* sA = smem + OFF_A;
    unsigned char* sVA = smem + OFF_VA;
    float* sW = reinterpret_cast<float*>(smem + OFF_W);
    float* sPatchAll = reinterpret_cast<float*>(smem + OFF_PATCH);   // [128][PO] fp32
    T* sH = reinterpret_cast<T*>(smem + OFF_HALO);                   // [(rows+2)][W+2][DK]
    T* sB2 = reinterpret_cast<T*>(smem + OFF_B2);                    // [TQ][n] flat

    const unsigned* va_flag = p.counters + 2 * p.slabs + slab;
    const unsigned va_target = (unsigned)p.plan.g_tasks;   // every G task of the slab merged its rows
    const bool early = ld_acquire(va_flag) >= va_target;      // usual case: the slab's aggregation is long done
    auto issue_agents = [&]() {
        if (tid == 0) {
            fence_proxy_async_all();   // A and V_A were written by other blocks with plain stores
            mbar_arrive_expect_tx(bar_agents(st), kTileBytes + (uint32_t)n * 128u);     // A: 64-row box, V_A: n-row box
            tma_load_2d(smem_u32(sA), &p.tm_a, 0, slab * n, bar_agents(st));
            tma_load_2d(smem_u32(sVA), &p.tm_va, 0, slab * n, bar_agents(st));
        }
    };
    // 1. bulk copies that do not depend on the aggregation: V rows y0-1 .. y0+rows, the B2 tile
    const T* b2src = has_b2 ? static_cast<const T*>(p.b2) + ((size_t)head * N + q0) * n : nullptr;
    const int b2bytes = TQ * n * 2;
    const bool b2_bulk = has_b2 && ((reinterpret_cast<uintptr_t>(b2src) & 15u) == 0) && ((b2bytes & 15) == 0);
    int vrows = 0;
    if (has_dwc) vrows = min(H, y0 + rows + 1) - max(0, y0 - 1);
    // Two threads share the issue work, each with a barrier of its own: thread 0 brings the Q tile (and A, V_A below),
    // lane 0 of warp 1 the V rows and the B2 tile, so that neither instruction stream waits for the other.
    const uint32_t vb_bytes = (uint32_t)vrows * W * DK * 2 + (b2_bulk ? b2bytes : 0);
    if (tid == 0) {
        const uint32_t bar = bar_bin(st);
        mbar_arrive_expect_tx(bar, (uint32_t)QT * DK * 2);
        // Q tile: 128 rows from the tile's first token (rows past the tile feed rows that are never stored)
        load_tokens(smem_u32(smem + OFF_PATCH), &p.tm_q, SH::kDense ? 1 : p.dense_in, p.hf_q, q0, head, slab / p.heads, slab * N, bar);
    }
    if (tid == 32 && vb_bytes) {
        const uint32_t bar = bar_vb(st);
        mbar_arrive_expect_tx(bar, vb_bytes);
        if (has_dwc) {
            for (int hr = 0; hr < rows + 2; ++hr) {
                const int y = y0 - 1 + hr;
                if (y >= 0 && y < H)
                    if (SH::kDense)              // dense: one copy of W * 128 contiguous bytes
                        bulk_load_1d(smem_u32(sH + ((size_t)hr * HP + 1) * DK),
                                     static_cast<const T*>(p.v) + ((size_t)slab * N + (size_t)y * W) * DK, W * DK * 2, bar);
                    else if (p.v_rows_contiguous)
                        bulk_load_1d(smem_u32(sH + ((size_t)hr * HP + 1) * DK),
                                     static_cast<const T*>(p.v) + tok_offset(p.lin, slab, p.heads, (long long)y * W), W * DK * 2, bar);
                    else
                        tma_load_tok(smem_u32(sH + ((size_t)hr * HP + 1) * DK), &p.tm_vrow, p.hf_vrow, y * W, head, slab / p.heads, bar);
            }
        }
        if (b2_bulk) bulk_load_1d(smem_u32(sB2), b2src, b2bytes, bar);
    }
    if (early) issue_agents();
    if (has_dwc) {
        // zero borders: columns x = -1 and x = W of every row, and rows that fall outside the grid
        for (int e = tid; e < (rows + 2) * 2 * (DK / 8); e += NT) {
            const int hr = e / (2 * (DK / 8)), rest = e - hr * 2 * (DK / 8);
            const int side = rest / (DK / 8), c = rest - side * (DK / 8);
            *(reinterpret_cast<uint4*>(sH + ((size_t)hr * HP + (side ? W + 1 : 0)) * DK) + c) = make_uint4(0, 0, 0, 0);
        }
        if (y0 == 0)
            for (int e = tid; e < W * (DK / 8); e += NT) *(reinterpret_cast<uint4*>(sH + DK) + e) = make_uint4(0, 0, 0, 0);
        if (y0 + rows >= H)
            for (int e = tid; e < W * (DK / 8); e += NT)
                *(reinterpret_cast<uint4*>(sH + ((size_t)(rows + 1) * HP + 1) * DK) + e) = make_uint4(0, 0, 0, 0);
        if (*s_whead != head) {       // filter taps change only with the head
            const T* w = static_cast<const T*>(p.dwc_w) + (size_t)head * DK * 9;
            for (int e = tid; e < 9 * DK; e += NT) {
                const int c = e / 9, tap = e - c * 9;
                sW[tap * DK + c] = Elem<T>::to_f32(w[e]);
            }
        }
    }
    if (has_b2 && !b2_bulk)
        copy_flat(reinterpret_cast<unsigned char*>(sB2), reinterpret_cast<const unsigned char*>(b2src), b2bytes, tid);
    // 2. wait for the slab's agent features, then fetch A and V_A (L2)
    //    (thread 0 alone: the barrier below passes everything on; a flag already seen set is not read again)
    if (tid == 0 && !early) poll_counter(va_flag, va_target, p.status, kTimeoutFeatures, p.poll_limit);
    if (!early) issue_agents();
    wait_bar(bar_agents(st), (st.ph >> kBitAgents) & 1u, p.status, kTimeoutLoads);
    st.ph ^= 1u << kBitAgents;
    wait_bar(bar_bin(st), (st.ph >> kBitBin) & 1u, p.status, kTimeoutLoads);
    st.ph ^= 1u << kBitBin;
    if (vb_bytes) {
        wait_bar(bar_vb(st), (st.ph >> kBitVb) & 1u, p.status, kTimeoutLoads);
        st.ph ^= 1u << kBitVb;
    }
    __syncthreads();
    if (tid == 0 && has_dwc) *s_whead = head;      // every thread has compared the old value before the barrier
    // (rows >= n of the V_A tile are zero: the copy brings n rows and the kernel cleared the rest at its start)
    // 3. attention part on the 5th-generation tensor cores: logits S = Q A^T accumulate in tensor
    //    memory; two threads share each query row (32 logit columns each: warps w and w+4 own the same
    //    tensor-memory lanes), exchange their partial maxima and sums through shared memory, write the
    //    probabilities back as the A operand of O = P V_A, and put the normalised row into the patch
    {
        unsigned char* sQt = smem + OFF_PATCH;                 // [128][128 B] swizzled Q tile (TMA)
        unsigned char* sPt = smem + OFF_PATCH + QT * 128;      // [128][128 B] swizzled P tile
        constexpr int fmt = Elem<T>::kIsBf16 ? 1 : 0;
        const uint32_t tS = st.tmem, tO = st.tmem + 64;
        const int half = warp >> 2, row = tid & 127, c0 = 32 * half;
        const uint32_t lane_base = ((uint32_t)(32 * (warp & 3))) << 16;     // this warp's 32 rows
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t idesc = umma_idesc(fmt, 128, 64, 0);
#pragma unroll
            for (int kk = 0; kk < DK / 16; ++kk)
                umma_f16(tS, umma_desc_sw128(smem_u32(sQt) + kk * 32), umma_desc_sw128(smem_u32(sA) + kk * 32), idesc, kk > 0);
            umma_commit(bar_mma(st));
        }
        wait_bar_all(bar_mma(st), (st.ph >> kBitMma) & 1u, p.status, kTimeoutLoads);
        st.ph ^= 1u << kBitMma;
        tc_fence_after_sync();
        float s[32];
        {
            uint32_t r[32];
            tmem_ld32(tS + lane_base + c0, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) s[i] = __uint_as_float(r[i]);
        }
        // logits in natural units: t = scale2 * q.a + b2; columns >= n are not agents
        const uint32_t* w32 = reinterpret_cast<const uint32_t*>(sB2) + ((row * n) >> 1) + 16 * half;
        const int sh = ((row * n) & 1) * 16;     // rows are n (possibly odd) elements long
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if (c0 + 2 * j < n) {
                float2 b = make_float2(0.f, 0.f);
                if (has_b2) b = unpack2<T>(__funnelshift_r(w32[j], w32[j + 1], sh));
                s[2 * j] = fmaf(s[2 * j], p.scale2, b.x);
                s[2 * j + 1] = (c0 + 2 * j + 1 < n) ? fmaf(s[2 * j + 1], p.scale2, b.y) : -INFINITY;
                mx = fmaxf(mx, fmaxf(s[2 * j], s[2 * j + 1]));
            }
        }
        s_red[half][row] = mx;
        __syncthreads();
        mx = fmaxf(mx, s_red[half ^ 1][row]);
        const float nm = -mx * kLog2e;
        float l = 0.f;
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if (c0 + 2 * j < n) {
                const float p0 = fast_exp2(fmaf(s[2 * j], kLog2e, nm));
                const float p1 = fast_exp2(fmaf(s[2 * j + 1], kLog2e, nm));      // exp2(-inf) = 0 past the last agent
                pk[j] = pack2<T>(p0, p1);
                const float2 q = unpack2<T>(pk[j]);    // the normaliser sums the rounded weights
                l += q.x + q.y;
            } else {
                pk[j] = 0u;
            }
        }
        s_red[2 + half][row] = l;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4*>(sPt + row * 128 + (((4 * half + c) ^ (row & 7)) << 4)) =
                make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
        fence_proxy_async();              // the tensor core reads P through the async proxy
        tc_fence_before_sync();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t idesc = umma_idesc(fmt, 128, 64, 1);       // V_A is [agents][d]: MN-major B operand
            for (int kk = 0; kk < n16; ++kk)
                umma_f16(tO, umma_desc_sw128(smem_u32(sPt) + kk * 32), umma_desc_sw128(smem_u32(sVA) + kk * 2048), idesc, kk > 0);
            umma_commit(bar_mma(st));
        }
        wait_bar_all(bar_mma(st), (st.ph >> kBitMma) & 1u, p.status, kTimeoutLoads);
        st.ph ^= 1u << kBitMma;
        tc_fence_after_sync();
        const float inv = 1.f / (s_red[2][row] + s_red[3][row]);
        float* prow = sPatchAll + row * PO + c0;
        {
            uint32_t r[32];
            tmem_ld32(tO + lane_base + c0, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 8; ++i)
                *reinterpret_cast<float4*>(prow + 4 * i) =
                    make_float4(__uint_as_float(r[4 * i]) * inv, __uint_as_float(r[4 * i + 1]) * inv,
                                __uint_as_float(r[4 * i + 2]) * inv, __uint_as_float(r[4 * i + 3]) * inv);
        }
        tc_fence_before_sync();
    }
    __syncthreads();
    // the rest of the task waits for nothing: take the next ticket now, so that the queue's round trip runs under it
    if (tid == 0) next_task = (int)atomicAdd(p.counters + 3 * (size_t)p.slabs, 1u);

    // 4. depthwise 3x3 term + store: thread = (tile row r, 4-channel group cq, x-segment)
    {
        constexpr int NCQ = DK / 4;
        const int npairs = rows * NCQ;
        int nseg = NT / npairs;
        if (nseg < 1) nseg = 1;
        if (nseg > W) nseg = W;
        const int seg_len = (W + nseg - 1) / nseg;
        T* gO = static_cast<T*>(p.out) + (SH::kDense ? ((long long)slab * N + q0) * DK : tok_offset(p.lout, slab, p.heads, q0));
        const size_t so = SH::kDense ? (size_t)DK : (size_t)p.lout.st;    // token stride of out
        for (int item = tid; item < npairs * nseg; item += NT) {
            const int pair = item % npairs, seg = item / npairs;
            const int r = pair / NCQ, cq = pair - r * NCQ;
            const int x0 = seg * seg_len, x1 = min(W, x0 + seg_len);
            if (x0 >= x1) continue;
            const float* pp = sPatchAll + (r * W) * PO + cq * 4;
            T* op = gO + (size_t)(r * W) * so + cq * 4;
            if (has_dwc) {
                float2 w[9][2];                 // taps x two channel pairs
#pragma unroll
                for (int tap = 0; tap < 9; ++tap) {
                    const float4 t = *reinterpret_cast<const float4*>(sW + tap * DK + cq * 4);
                    w[tap][0] = make_float2(t.x, t.y);
                    w[tap][1] = make_float2(t.z, t.w);
                }
                // buffer rows r, r+1, r+2 are grid rows y-1, y, y+1; buffer column x+1 is grid column x
                const T* hp = sH + (r * HP) * DK + cq * 4;
                float2 ca[3][2], cb[3][2], cc[3][2];
                auto load_col = [&](int hx, float2 (&c)[3][2]) {
#pragma unroll
                    for (int u = 0; u < 3; ++u) {
                        const uint2 raw = *reinterpret_cast<const uint2*>(hp + (u * HP + hx) * DK);
                        c[u][0] = unpack2<T>(raw.x);
                        c[u][1] = unpack2<T>(raw.y);
                    }
                };
                auto emit = [&](int x, const float2 (&l)[3][2], const float2 (&c)[3][2], const float2 (&rr)[3][2]) {
                    const float4 a4 = *reinterpret_cast<const float4*>(pp + x * PO);
                    float2 o0 = make_float2(a4.x, a4.y), o1 = make_float2(a4.z, a4.w);
#pragma unroll
                    for (int u = 0; u < 3; ++u) {
                        o0 = ffma2(w[u * 3 + 0][0], l[u][0], o0);  o1 = ffma2(w[u * 3 + 0][1], l[u][1], o1);
                        o0 = ffma2(w[u * 3 + 1][0], c[u][0], o0);  o1 = ffma2(w[u * 3 + 1][1], c[u][1], o1);
                        o0 = ffma2(w[u * 3 + 2][0], rr[u][0], o0); o1 = ffma2(w[u * 3 + 2][1], rr[u][1], o1);
                    }
                    uint2 outw;
                    outw.x = pack2<T>(o0.x, o0.y);
                    outw.y = pack2<T>(o1.x, o1.y);
                    *reinterpret_cast<uint2*>(op + x * so) = outw;
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
                    *reinterpret_cast<uint2*>(op + x * so) = outw;
                }
            }
        }
    }
    // (the caller closes the task: proxy fence and block barrier, after which shared memory is free)
}

// ---------------------------------------------------------------------------------- kernel
template <typename T, typename SH>
__global__ void __launch_bounds__(NT, 2) fused_kernel(const __grid_constant__ FusedArgs p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ int s_task[2], s_flag, s_whead;
    __shared__ uint32_t s_tmem;
    __shared__ float s_red[4][128];     // per query row: partial maxima and partial sums of the two column halves
    // TMA tiles with the 128-byte swizzle want a 1024-byte aligned base
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x;
    BlockState st;
    st.bar_base = smem_u32(smem + OFF_BAR);
    st.ph = 0u;
    if (tid == 0) {
        s_whead = -1;
        for (int i = 0; i < kNumBars; ++i) mbar_init(st.bar_base + 8 * i, 1);
        mbar_fence_init();
    }
    // rows >= n of the V_A tile never receive data (its copies bring n rows): zero, since 0 * NaN is not 0
    for (int e = tid; e < (RP - p.n) * 8; e += NT)
        *(reinterpret_cast<uint4*>(smem + OFF_VA + (p.n + e / 8) * 128) + (e & 7)) = make_uint4(0, 0, 0, 0);
    fence_proxy_async();          // the tensor core reads V_A through the async proxy
    // tensor memory for the broadcast MMAs: warp 0 allocates (and frees at the end)
    if (tid < 32) tmem_alloc<kTmemCols>(smem_u32(&s_tmem));
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    st.tmem = s_tmem;
    const int G = p.plan.g_tasks, B = p.plan.b_tasks, Lg = p.plan.lag, S = p.slabs;
    const int count0 = Lg * G, count1 = (S - Lg) * (G + B);
    const int total = S * (G + B);
    unsigned* queue = p.counters + 3 * (size_t)S;
    // Every task takes the ticket of the block's next task at the start of its wait-free tail (thread 0) and
    // the ticket is handed to the block through s_task[] before the task's closing barrier, so no barrier of
    // its own is spent on the queue.  Two slots: a slot is rewritten two tasks after it was read.
    if (tid == 0) s_task[0] = (int)atomicAdd(queue, 1u);
    __syncthreads();
    for (int par = 0;; par ^= 1) {
        const int task = s_task[par];
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
        int next_task = total;          // thread 0: set by the task
        if (is_g) run_g_task<T, SH>(p, slab, sub, smem, st, &s_flag, next_task);
        else      run_b_task<T, SH>(p, slab, sub, smem, st, &s_whead, s_red, next_task);
        if (tid == 0) s_task[par ^ 1] = next_task;
        fence_proxy_async();   // this task's plain shared-memory writes precede the next task's TMA writes
        __syncthreads();       // shared memory is free for the next task, and its ticket is visible
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid < 32) tmem_dealloc<kTmemCols>(st.tmem);
}


// Per-instantiation host helpers: occupancy query and launch.
template <typename T, typename SH>
static int fused_occupancy_of() {
    int occ = 0;
    auto kern = fused_kernel<T, SH>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, NT, kSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return occ;
}
template <typename SH>
static int fused_occupancy_dt(int dtype) {
    return dtype == kBF16 ? fused_occupancy_of<__nv_bfloat16, SH>() : fused_occupancy_of<__half, SH>();
}
template <typename SH>
static cudaError_t fused_launch_dt(int dtype, const FusedArgs& a, cudaStream_t st) {
    if (dtype == kBF16) fused_kernel<__nv_bfloat16, SH><<<a.plan.grid, NT, kSmemBytes, st>>>(a);
    else if (dtype == kF16) fused_kernel<__half, SH><<<a.plan.grid, NT, kSmemBytes, st>>>(a);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace aa
