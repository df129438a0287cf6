// Merge of split online-softmax partial states into V_A (Eq. 3, agent aggregation).
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace aa {

// Arrival counter: returns true in every thread of the block that arrives last for its slab.
// Each block calls this after its partial state is written; `expected` blocks arrive per slab.
// The last block resets the counter, so it is zero again when the kernel ends.  Nothing waits.
__device__ __forceinline__ bool arrive_is_last(unsigned* ticket, unsigned expected, int* s_flag) {
    __threadfence();                       // this block's partial is visible device-wide ...
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned t = atomicAdd(ticket, 1u);  // ... before its arrival is counted
        const int last = (t == expected - 1u);
        if (last) *ticket = 0u;
        *s_flag = last;
    }
    __syncthreads();
    const bool last = (*s_flag != 0);
    if (last) __threadfence();             // order the partial reads after the last arrival
    return last;
}

// parts_base: first partial of the slab; every partial is m[rows_pad], l[rows_pad],
// acc[rows_pad][dpad] (fp32, m in log2 units).  With m = max_j m_j:
//   V_A[r][c] = sum_j acc_j[r][c] 2^(m_j - m)  /  sum_j l_j 2^(m_j - m),
// summed in the fixed order j = 0..parts-1, so the result does not depend on arrival order.
template <typename T>
__device__ __forceinline__ void merge_partials(const float* parts_base, int parts, int rows_pad,
                                               int dpad, int rows, int d, T* out) {
    const size_t pf = partial_floats(rows_pad, dpad);
    for (int e = threadIdx.x; e < rows * d; e += blockDim.x) {
        const int r = e / d, c = e - r * d;
        float m = -INFINITY;
        for (int j = 0; j < parts; ++j) m = fmaxf(m, __ldcg(parts_base + j * pf + r));
        float num = 0.f, den = 0.f;
        for (int j = 0; j < parts; ++j) {
            const float* pj = parts_base + j * pf;
            const float mj = __ldcg(pj + r);
            const float w = (mj == -INFINITY) ? 0.f : exp2f(mj - m);
            den += w * __ldcg(pj + rows_pad + r);
            num += w * __ldcg(pj + 2 * (size_t)rows_pad + (size_t)r * dpad + c);
        }
        out[e] = Elem<T>::from_f32(num / den);
    }
}

}  // namespace aa
