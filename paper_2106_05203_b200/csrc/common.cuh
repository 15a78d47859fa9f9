// Shared device helpers of libef21 (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ef21 {

typedef long long i64;

// Status word layout in the workspace (one 256-byte slot): word 0 = first error code seen.
__device__ __forceinline__ void record_error(unsigned* status, unsigned code) {
    atomicCAS(status, 0u, code);
}

// Magnitude key of Top-k: the bit pattern of |v|.  For finite values the order of keys is the
// order of magnitudes; +0 and -0 share key 0.
__device__ __forceinline__ unsigned mag_key(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// Non-finite inputs of the compressor: a NaN or Inf has a key above every finite value's, so it is always
// among the k selected entries -- checking the selected values is enough to notice one anywhere in the vector.
// Records EF21_ERR_NONFINITE in the status word (status may be null: standalone calls have none).
__device__ __forceinline__ void flag_nonfinite(unsigned* status, float selected) {
    if (status != nullptr && mag_key(selected) > 0x7f7fffffu) record_error(status, 6u /* EF21_ERR_NONFINITE */);
}

// v = a - b as one rounded fp32 subtraction (b == nullptr: v = a).
__device__ __forceinline__ float diff_at(const float* __restrict__ a, const float* __restrict__ b, i64 j) {
    float av = a[j];
    return b ? __fsub_rn(av, b[j]) : av;
}

__device__ __forceinline__ unsigned warp_incl_scan(unsigned v) {
    const unsigned lane = threadIdx.x & 31u;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= (unsigned)o) v += t;
    }
    return v;
}

// Exclusive prefix sum over the threads of a block (blockDim.x a multiple of 32, <= 1024).
// scratch: 33 unsigned words of shared memory.  Returns the exclusive prefix; total = block sum.
__device__ __forceinline__ unsigned block_excl_scan(unsigned v, unsigned* scratch, unsigned& total) {
    const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    __syncthreads();
    unsigned inc = warp_incl_scan(v);
    if (lane == 31u) scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned w = lane < nwarps ? scratch[lane] : 0u;
        unsigned wi = warp_incl_scan(w);
        scratch[lane] = wi - w;
        if (lane == 31u) scratch[32] = wi;
    }
    __syncthreads();
    total = scratch[32];
    return inc - v + scratch[warp];
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum of v[r] over the 32 lanes for RB rows at once: after the call lane L holds the total of
// row L / (32/RB).  RB-1 shuffles for the halving steps plus log2(32/RB) butterfly steps.
template <int RB>
__device__ __forceinline__ float reduce_rows(float (&v)[RB], int lane) {
#pragma unroll
    for (int half = RB / 2, off = 16; half >= 1; half >>= 1, off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int r = 0; r < half; ++r) {
            const float keep = upper ? v[r + half] : v[r];
            const float send = upper ? v[r] : v[r + half];
            v[r] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    float s = v[0];
#pragma unroll
    for (int off = (32 / RB) / 2; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    return s;
}

__device__ __forceinline__ float4 fma4(float s, float4 a, float4 c) {
    c.x = fmaf(s, a.x, c.x); c.y = fmaf(s, a.y, c.y); c.z = fmaf(s, a.z, c.z); c.w = fmaf(s, a.w, c.w);
    return c;
}
__device__ __forceinline__ float dot4(float4 a, float4 b, float z) {
    z = fmaf(a.x, b.x, z); z = fmaf(a.y, b.y, z); z = fmaf(a.z, b.z, z); z = fmaf(a.w, b.w, z);
    return z;
}
// -y / (1 + exp(y z)): derivative of log(1 + exp(-y z)) with respect to z, overflow-safe.
__device__ __forceinline__ float logistic_residual(float y, float z) {
    float t = y * z;
    float e = expf(-fabsf(t));                 // in (0, 1]
    float num = t >= 0.f ? e : 1.f;
    return __fdiv_rn(-y * num, 1.f + e);
}

// Residual rho_r = d loss / d margin for the two built-in objectives:
//   objective 0: logistic loss log(1 + exp(-y z))      (Section 5, Eq. 19)
//   objective 1: least squares (z - y)^2               (Appendix A.2)
__device__ __forceinline__ float loss_residual(int objective, float y, float z) {
    return objective == 0 ? logistic_residual(y, z) : 2.f * (z - y);
}

// a / b, correctly rounded, for four numerators at once, given rc = the correctly rounded reciprocal of b
// (__frcp_rn(b)): q = a*rc followed by two refinement steps q <- fma(fma(-q, b, a), rc, q).  The residual
// a - q*b is exact in an fma, and with rc correctly rounded and q already within an ulp the last step yields
// the correctly rounded quotient (Markstein's theorem on division by reciprocal and fused correction), as long as
// nothing over- or underflows on the way: |a| in [2^-100, 2^100], or a = 0 (which keeps its sign by a select);
// otherwise the IEEE division instruction sequence is used.  Four independent chains of five operations replace
// four division subroutines that would run one after the other (36 against 228 cycles in one warp, measured).
__device__ __forceinline__ float4 div4_rn(float4 a, float b, float rc) {
    const float lo = 7.888609e-31f, hi = 1.2676506e30f;      // 2^-100, 2^100
    const float m0 = fabsf(a.x), m1 = fabsf(a.y), m2 = fabsf(a.z), m3 = fabsf(a.w);
    const bool plain = (m0 >= lo || m0 == 0.f) && (m1 >= lo || m1 == 0.f) && (m2 >= lo || m2 == 0.f) && (m3 >= lo || m3 == 0.f) &&
                       fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) <= hi;
    float4 q;
    if (plain) {
        q.x = a.x * rc; q.y = a.y * rc; q.z = a.z * rc; q.w = a.w * rc;
#pragma unroll
        for (int step = 0; step < 2; ++step) {
            q.x = fmaf(fmaf(-q.x, b, a.x), rc, q.x); q.y = fmaf(fmaf(-q.y, b, a.y), rc, q.y);
            q.z = fmaf(fmaf(-q.z, b, a.z), rc, q.z); q.w = fmaf(fmaf(-q.w, b, a.w), rc, q.w);
        }
        q.x = m0 == 0.f ? a.x : q.x; q.y = m1 == 0.f ? a.y : q.y;       // (+-0) / b = +-0
        q.z = m2 == 0.f ? a.z : q.z; q.w = m3 == 0.f ? a.w : q.w;
    } else {
        q.x = __fdiv_rn(a.x, b); q.y = __fdiv_rn(a.y, b); q.z = __fdiv_rn(a.z, b); q.w = __fdiv_rn(a.w, b);
    }
    return q;
}

// d/dx of lambda x^2/(1+x^2) = 2 lambda x / (1+x^2)^2.
__device__ __forceinline__ float regulariser_grad(float lambda, float x) {
    float q = fmaf(x, x, 1.f);
    return __fdiv_rn(2.f * lambda * x, q * q);
}

}  // namespace ef21
