// The original error feedback method (Algorithm 4), the parts that differ from Algorithm 2.  The
// worker state is the error e_i (kept where Algorithm 2 keeps g_i).  One iteration from (x, e_i):
//   p_i = e_i + gamma grad f_i(x)           the vector worker i would like to send
//   w_i = C(p_i)                            the message (Top-k kernels, no subtrahend)
//   x   <- x - (1/n) sum_i w_i              (aggregation kernels, target x, factor -1/n)
//   e_i <- p_i - w_i                        the error carried to the next iteration
// Each of gamma * grad, e + a, p - w is one rounded fp32 operation.
#pragma once
#include "common.cuh"

namespace ef21 {

// e_i <- e_i + gamma * grad_i, all n rows (grad has leading dimension pitch, e has ld).
__global__ void ef_compose_kernel(const float* __restrict__ grad, i64 pitch, float* __restrict__ e, i64 ld,
                                  int n, i64 d, float gamma) {
    const i64 total = (i64)n * d;
    for (i64 t = blockIdx.x * (i64)blockDim.x + threadIdx.x; t < total; t += (i64)gridDim.x * blockDim.x) {
        const i64 i = t / d, j = t - i * d;
        float* p = e + i * ld + j;
        *p = __fadd_rn(*p, __fmul_rn(gamma, grad[i * pitch + j]));
    }
}

// e_i[idx] <- p_i[idx] - w_i[idx] on the n*k sent coordinates (the others keep p_i - 0 = p_i).
__global__ void ef_subtract_sent_kernel(const int* __restrict__ idx, const float* __restrict__ val, i64 total, int k,
                                        i64 ld, float* __restrict__ e) {
    const i64 t = blockIdx.x * (i64)blockDim.x + threadIdx.x;
    if (t >= total) return;
    const i64 i = t / k;
    float* p = e + i * ld + idx[t];
    *p = __fsub_rn(*p, val[t]);
}

}  // namespace ef21
