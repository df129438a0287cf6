// Building blocks of the warp-specialised tensor-memory kernels (aggregate_umma.cu, broadcast_umma.cu):
// bounded mbarrier waits with per-thread phase tracking, group arrivals, tensor-memory stores.
#pragma once
#include "tma.cuh"
#include "umma.cuh"

namespace aa {

constexpr unsigned kPipeBarLimit = 1u << 20;      // mbarrier try_wait attempts before a wait gives up
constexpr unsigned kPipeSuspendNs = 2000;         // a try_wait may keep its thread suspended this long

// Per-thread view of a block's mbarriers.  Every wait is bounded: on expiry the thread sets the
// block-wide `dead` flag (every later wait of the block then returns at once) and records `code` in the
// device status word, so a logic error ends as a status code instead of a hang.
struct Pipe {
    int* status;          // device status word (global)
    int* dead;            // shared flag
    uint32_t bars;        // shared address of mbarrier 0
    uint32_t ph;          // parity to wait for next, one bit per mbarrier this thread waits on (at most 32 barriers)
    uint32_t tmem;        // base of the block's tensor-memory columns
};
__device__ __forceinline__ uint32_t pipe_bar(const Pipe& pp, int i) { return pp.bars + 8u * (uint32_t)i; }
__device__ __forceinline__ int pipe_dead(const Pipe& pp) { return *reinterpret_cast<const volatile int*>(pp.dead); }

// One thread waits for the next phase of mbarrier i (its parity bit flips either way).  The first
// attempt is the fast path; the bounded loop and the look at the block's flag come only after it fails.
__device__ __forceinline__ void pipe_wait_one(Pipe& pp, int i, int code) {
    const uint32_t parity = (pp.ph >> i) & 1u;
    pp.ph ^= 1u << i;
    const uint32_t bar = pipe_bar(pp, i);
    if (mbar_try_wait_suspend(bar, parity, kPipeSuspendNs)) return;
    for (unsigned tries = 0; tries < kPipeBarLimit; ++tries) {
        if (pipe_dead(pp)) return;
        if (mbar_try_wait_suspend(bar, parity, kPipeSuspendNs)) return;
    }
    *reinterpret_cast<volatile int*>(pp.dead) = 1;
    if (pp.status) atomicCAS(pp.status, 0, code);
}
__device__ __forceinline__ void pipe_arrive(const Pipe& pp, int i) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(pipe_bar(pp, i)) : "memory");
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

}  // namespace aa
