// Helpers of the streaming kernels for small agent counts (stream_prep.cu, stream_aggregate.cu,
// stream_broadcast.cu): tcgen05.mma with the A operand in tensor memory, packed 16-bit conversions and
// exponentials, bounded mbarrier waits with an explicit phase parity.
#pragma once
#include "common.cuh"
#include "kernels.h"
#include "pipe.cuh"

namespace aa {

// One fp32 column of this thread's tensor-memory row.
__device__ __forceinline__ uint32_t tmem_ld1(uint32_t taddr) {
    uint32_t r;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];\n" : "=r"(r) : "r"(taddr) : "memory");
    return r;
}

// 16 consecutive fp32 columns of this thread's tensor-memory row <- registers
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// Packed 16-bit arithmetic of the element type: two fp32 -> one pair (low half = first value), and the
// base-2 exponential of a pair in one instruction (its result is the pair of probabilities, already in the
// operand type of the next product).
template <typename T> struct Pair;
template <> struct Pair<__nv_bfloat16> {
    static constexpr uint32_t kOne = 0x3F80u;            // 1.0
    static constexpr float kBig = 30000.f;               // biases are clamped to +-kBig: low enough to remove a key, small
                                                         // enough that logit arithmetic in fp32 stays exact to 0.01
    static constexpr float kPad = 60000.f;               // minus this: bias of the agent columns past n
    __device__ static __forceinline__ uint32_t cvt(float lo, float hi) {
        uint32_t d;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
        return d;
    }
    __device__ static __forceinline__ uint32_t ex2(uint32_t x) {
        uint32_t d;
        asm("ex2.approx.ftz.bf16x2 %0, %1;" : "=r"(d) : "r"(x));
        return d;
    }
};
template <> struct Pair<__half> {
    static constexpr uint32_t kOne = 0x3C00u;
    static constexpr float kBig = 30000.f;
    static constexpr float kPad = 60000.f;
    __device__ static __forceinline__ uint32_t cvt(float lo, float hi) {
        uint32_t d;
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
        return d;
    }
    __device__ static __forceinline__ uint32_t ex2(uint32_t x) {
        uint32_t d;
        asm("ex2.approx.f16x2 %0, %1;" : "=r"(d) : "r"(x));
        return d;
    }
};
// A pair holds a value >= 2 (or a NaN) in either half: bit 14 of a half is the top exponent bit of both
// 16-bit formats, and probabilities are never negative.
constexpr uint32_t kPairGe2 = 0x40004000u;

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Bounded wait for the phase of mbarrier i with the given parity (the caller derives the parity from its
// loop counter).  On expiry the block's `dead` flag is set, every later wait of the block returns at once,
// and `code` goes to the device status word: a logic error ends as a status code, never as a hang.
__device__ __forceinline__ void wait_par(Pipe& pp, int i, uint32_t parity, int code) {
    const uint32_t bar = pipe_bar(pp, i);
    if (mbar_try_wait_suspend(bar, parity & 1u, kPipeSuspendNs)) return;
    for (unsigned tries = 0; tries < kPipeBarLimit; ++tries) {
        if (mbar_try_wait_suspend(bar, parity & 1u, kPipeSuspendNs)) return;
        __nanosleep(64);                                   // a waiting warp must not take issue slots from working ones
        if ((tries & 63u) == 63u && pipe_dead(pp)) return;
    }
    *reinterpret_cast<volatile int*>(pp.dead) = 1;
    if (pp.status) atomicCAS(pp.status, 0, code);
}

// Wait of an issuing role (producer, MMA issuers).  The thread is parked by the suspended form of try_wait and
// woken by the phase completion: a tight polling loop here would take issue slots from the compute warp that
// shares the scheduler.  Bounded like every other wait.
__device__ __forceinline__ void wait_spin(Pipe& pp, int i, uint32_t parity, int code) {
    const uint32_t bar = pipe_bar(pp, i);
    if (mbar_try_wait(bar, parity & 1u)) return;
    for (unsigned tries = 0; tries < (1u << 22); ++tries) {
        if (mbar_try_wait_suspend(bar, parity & 1u, 4000u)) return;
        if ((tries & 63u) == 63u && pipe_dead(pp)) return;
    }
    *reinterpret_cast<volatile int*>(pp.dead) = 1;
    if (pp.status) atomicCAS(pp.status, 0, code);
}

// End of an MMA-issuing warp: commit to a barrier of its own and wait (bounded, whatever the block's state) until
// every instruction it has issued is complete, so that the block never frees its tensor memory under a running one.
__device__ __forceinline__ void umma_drain_w(Pipe& pp, int i) {
    umma_commit_w(pipe_bar(pp, i));
    const uint32_t bar = pipe_bar(pp, i);
    for (unsigned tries = 0; tries < (1u << 16); ++tries)
        if (mbar_try_wait_suspend(bar, 0u, 4000u)) return;
}

// 3-D tiled load: box at (0, row, z) of a map whose dimensions are (64 channels or columns, rows, slabs or
// heads).  Rows outside [0, rows) are zero-filled, so a tile never runs into the next slab.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

// 4-D tiled load of a [slab][y][x][64] view: box at (0, x, y, slab); coordinates outside the grid (x = -1, x = W,
// y = -1, y = H) are zero-filled, which is the zero padding of the depthwise window.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

// Programmatic dependent launch: a kernel launched with the attribute may start before its predecessor in
// the stream has finished; it must pass pdl_wait() before it touches anything the predecessor writes.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// Host: map of a [z][rows][64] tensor of 16-bit elements (row pitch 128 bytes, z pitch rows * 128 bytes) with a
// box of 64 x box_rows x 1, 128-byte swizzle or none.
inline bool make_map_rows3d_u16(CUtensorMap* out, const void* base, uint64_t zs, uint64_t rows, uint32_t box_rows, bool swizzle) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || box_rows > 256 || box_rows < 1) return false;
    const cuuint64_t dims[3] = {64, rows, zs};
    const cuuint64_t strides[2] = {128, rows * 128};
    const cuuint32_t box[3] = {64, box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Host: map of a dense [z][H][W][64] tensor of 16-bit elements with a box of 64 x box_w x box_h x 1, 128-byte swizzle or none.
inline bool make_map_grid4d_u16(CUtensorMap* out, const void* base, uint64_t zs, uint64_t H, uint64_t W, uint32_t box_h, uint32_t box_w, bool swizzle) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || box_h > 256 || box_w > 256 || box_h < 1 || box_w < 1) return false;
    const cuuint64_t dims[4] = {64, W, H, zs};
    const cuuint64_t strides[3] = {128, W * 128, H * W * 128};
    const cuuint32_t box[4] = {64, box_w, box_h, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace aa
