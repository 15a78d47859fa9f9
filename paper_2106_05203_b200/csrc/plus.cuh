// EF21+ (Algorithm 3): every worker keeps the better of the plain compressor b_i = C(grad_i) and the
// Markov compressor m_i = g_i + C(grad_i - g_i), judged by the distortions
//     B_i = ||b_i - grad_i||^2,   M_i = ||m_i - grad_i||^2      (fp64 sums of fp32 terms),
// g_i <- m_i if M_i <= B_i else b_i; the master recomputes g = (1/n) sum_i g_i.
#pragma once
#include "common.cuh"

namespace ef21 {

constexpr int PLUS_BLOCK = 256;

// Deterministic block sum of doubles (fixed tree): result valid in thread 0.
__device__ __forceinline__ double block_sum_f64(double v, double* scratch /* [PLUS_BLOCK/32] */) {
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double s = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < PLUS_BLOCK / 32; ++w) s += scratch[w];
    __syncthreads();
    return s;
}

// One block per worker.  a: local gradients (pitch_a), gi: worker states (pitch ld).
// (idx_m, val_m): C(grad_i - g_i); (idx_b, val_b): C(grad_i).  On exit g_i holds the chosen vector,
// (idx_m, val_m) holds the compressed vector that was used and choice[i] is 0 (Markov) or 1 (plain).
__global__ void __launch_bounds__(PLUS_BLOCK)
plus_choose_kernel(const float* __restrict__ a, i64 pitch_a, float* gi, i64 ld, i64 d, int k,
                   int* __restrict__ idx_m, float* __restrict__ val_m,
                   const int* __restrict__ idx_b, const float* __restrict__ val_b,
                   float* __restrict__ old_vals, unsigned* __restrict__ bitmap, int* __restrict__ choice) {
    __shared__ double scratch[PLUS_BLOCK / 32];
    __shared__ int take_plain;
    const int i = blockIdx.x;
    const float* __restrict__ grad = a + (i64)i * pitch_a;
    float* g = gi + (i64)i * ld;
    int* im = idx_m + (i64)i * k;
    float* vm = val_m + (i64)i * k;
    const int* ib = idx_b + (i64)i * k;
    const float* vb = val_b + (i64)i * k;
    float* old = old_vals + (i64)i * k;

    // mark the entries kept by the plain compressor (bitmap row of this worker)
    const i64 words = (d + 31) >> 5;
    unsigned* bm = bitmap + (i64)i * words;
    for (i64 w = threadIdx.x; w < words; w += PLUS_BLOCK) bm[w] = 0u;
    __syncthreads();
    for (int t = threadIdx.x; t < k; t += PLUS_BLOCK) atomicOr(&bm[ib[t] >> 5], 1u << (ib[t] & 31));
    // tentatively g_i <- m_i, remembering the k overwritten entries
    for (int t = threadIdx.x; t < k; t += PLUS_BLOCK) {
        const int j = im[t];
        const float o = g[j];
        old[t] = o;
        g[j] = __fadd_rn(o, vm[t]);
    }
    __syncthreads();
    // M = sum_j (m_j - grad_j)^2 and B = sum_j (b_j - grad_j)^2 over the same coordinates in the same order,
    // so that the two sums are bit-identical whenever the two candidates coincide (e.g. g_i = 0)
    double m_part = 0.0, b_part = 0.0;
    for (i64 j = threadIdx.x; j < d; j += PLUS_BLOCK) {
        const double gr = (double)grad[j];
        const double e = (double)g[j] - gr;
        m_part += e * e;
        const bool kept = (bm[j >> 5] >> (j & 31)) & 1u;
        b_part += kept ? 0.0 : gr * gr;
    }
    const double M = block_sum_f64(m_part, scratch);
    const double B = block_sum_f64(b_part, scratch);
    if (threadIdx.x == 0) {
        take_plain = (M <= B) ? 0 : 1;
        choice[i] = take_plain;
    }
    __syncthreads();
    if (take_plain) {
        for (i64 j = threadIdx.x; j < d; j += PLUS_BLOCK) g[j] = 0.f;
        __syncthreads();
        for (int t = threadIdx.x; t < k; t += PLUS_BLOCK) {
            g[ib[t]] = vb[t];
            im[t] = ib[t];
            vm[t] = vb[t];
        }
    }
}

// g_j = (sum over workers, ascending, of g_ij) * (1/n).
__global__ void dense_mean_kernel(const float* __restrict__ gi, i64 ld, int n, i64 d, float inv_n,
                                  float* __restrict__ g) {
    for (i64 j = blockIdx.x * (i64)blockDim.x + threadIdx.x; j < d; j += (i64)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int i = 0; i < n; ++i) s = __fadd_rn(s, gi[(i64)i * ld + j]);
        g[j] = __fmul_rn(s, inv_n);
    }
}

}  // namespace ef21
