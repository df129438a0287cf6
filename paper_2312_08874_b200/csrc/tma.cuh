// Tensor Memory Accelerator and mbarrier helpers (sm_90+/sm_100 PTX), plus the host-side encoder
// of 2-D tensor maps.  No cluster multicast is used anywhere: every block fetches its own tiles.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.h"

namespace aa {

// ------------------------------------------------------------------------------------ device
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}
// One arrival that also announces `bytes` of asynchronous copies to come.
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// try_wait with a suspend-time hint (nanoseconds): the thread stays parked until the phase completes
// or the time is up, instead of spinning.
__device__ __forceinline__ bool mbar_try_wait_suspend(uint32_t bar, uint32_t parity, uint32_t ns = 2000u) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// Bounded wait: returns false (and the caller records a timeout) if the phase never completes.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Orders this thread's earlier generic-proxy accesses to shared memory before later async-proxy
// (TMA) accesses to it.
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
}
// Orders this thread's earlier generic-proxy accesses (here: the acquire that observed other blocks' plain global
// stores) before its later async-proxy accesses (TMA reads of that global memory).
__device__ __forceinline__ void fence_proxy_async_all() {
    asm volatile("fence.proxy.async;\n" ::: "memory");
}
// 2-D tiled load: box at (x = innermost coordinate, y) of the tensor map -> shared memory.
// x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
// 4-D tiled load of a [batch, head, token, d] tensor with arbitrary (batch, head, token) strides: the map's
// dimensions are (d, then head and token in the order of their strides, then batch); `head_first` says
// which of the two comes second.  The box is 64 channels x `box tokens` of one head of one batch item;
// tokens past the grid are zero-filled.
__device__ __forceinline__ void tma_load_tok(uint32_t dst, const CUtensorMap* map, int head_first, int tok, int head,
                                             int b, uint32_t bar) {
    const int c1 = head_first ? head : tok, c2 = head_first ? tok : head;
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(c1), "r"(c2), "r"(b), "r"(bar) : "memory");
}
// 1-D bulk copy global -> shared: both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Driver entry point looked up through the runtime (the library does not link libcuda).
inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Map of a dense row-major matrix of 16-bit elements [rows][cols] (row pitch = cols * 2 bytes, a
// multiple of 16) with a box of box_rows x box_cols and the 128-byte swizzle (box_cols * 2 = 128).
inline bool make_map_2d_u16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                            uint32_t box_rows, uint32_t box_cols) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((cols * 2) & 15u) || box_cols * 2 != 128 || box_rows > 256)
        return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Map of such a tensor of 16-bit elements for tma_load_tok: box = 64 channels (d <= 64: the rest is
// zero-filled) x box_tokens, with the 128-byte swizzle or none.  *head_first receives the order.
// False if the strides cannot be expressed (not multiples of 16 bytes, or not nested).
inline bool make_map_tok_u16(CUtensorMap* out, int* head_first, const void* base, const TokLayout& l, int batch,
                             int heads, long long n_tokens, int d, uint32_t box_tokens, bool swizzle) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || box_tokens > 256 || d > 64 || d % 8 != 0) return false;
    if ((l.sb & 7) || (l.sh & 7) || (l.st & 7) || l.st < d) return false;
    const int hf = (heads > 1 && l.sh < l.st) ? 1 : 0;
    *head_first = hf;
    const cuuint64_t n1 = hf ? (cuuint64_t)heads : (cuuint64_t)n_tokens, n2 = hf ? (cuuint64_t)n_tokens : (cuuint64_t)heads;
    const cuuint64_t s1 = (cuuint64_t)(hf ? l.sh : l.st) * 2;
    cuuint64_t s2 = (cuuint64_t)(hf ? l.st : l.sh) * 2;
    if (heads == 1 && s2 < s1 * n1) s2 = s1 * n1;          // a single head: its stride is never used
    cuuint64_t s3 = (cuuint64_t)l.sb * 2;
    if (batch == 1 && s3 < s2 * n2) s3 = s2 * n2;          // a single batch item: its stride is never used
    const cuuint64_t dims[4] = {(cuuint64_t)d, n1, n2, (cuuint64_t)batch};
    const cuuint64_t strides[3] = {s1, s2, s3};
    if (strides[1] < strides[0] || strides[2] < strides[1]) return false;
    const cuuint32_t box[4] = {64u, hf ? 1u : box_tokens, hf ? box_tokens : 1u, 1u};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace aa
