// State updates of Algorithm 2 after the messages c_i = (idx, val)[k] are known:
//   g_i <- g_i + c_i                      (worker state, node loop)
//   g   <- g + (1/n) sum_i c_i            (master, last line of the loop)
//   x   <- x - gamma g                    (master, first line of the loop)
// The per-coordinate sum over workers runs in ascending worker index starting from 0, each
// operation a single rounded fp32 add / multiply, so the result does not depend on scheduling.
#pragma once
#include "common.cuh"

namespace ef21 {

constexpr int AGG_TILE = 2048;     // coordinates per block in the aggregation
constexpr int AGG_BLOCK = 256;

// g_i[idx] += val for all n*k message entries (indices within a worker are distinct).
__global__ void apply_messages_kernel(const int* __restrict__ idx, const float* __restrict__ val,
                                      i64 total, int k, i64 ld, float* __restrict__ gi) {
    const i64 e = blockIdx.x * (i64)blockDim.x + threadIdx.x;
    if (e >= total) return;
    const i64 i = e / k;
    float* p = gi + i * ld + idx[e];
    *p = __fadd_rn(*p, val[e]);
}

// Scaled Rand-k (Appendix, Lemma 8 and Example 2: Rand-k times 1/(1 + omega) keeps the k sampled entries as they
// are): message entry t of worker i is (S, a[S] - g_i[S]) with S = sets[i][t], and g_i[S] takes the sum.  The sets are
// an input: k distinct indices in ascending order per worker.  An index outside [0, d), or one that does not exceed
// its predecessor, is reported through the status word and replaced by position t (never dereferenced as given).
__global__ void randk_select_kernel(const float* __restrict__ a, i64 pitch_a, float* __restrict__ gi, i64 ld,
                                    const int* __restrict__ sets, i64 total, int k, i64 d,
                                    int* __restrict__ idx_out, float* __restrict__ val_out, unsigned* status) {
    const i64 e = blockIdx.x * (i64)blockDim.x + threadIdx.x;
    if (e >= total) return;
    const i64 i = e / k;
    const int t = (int)(e - i * k);
    int j = sets[e];
    const bool bad = j < 0 || (i64)j >= d || (t > 0 && sets[e - 1] >= j);
    if (bad) { record_error(status, 1u /* EF21_ERR_INVALID_ARG */); j = t; }
    float* p = gi + i * ld + j;
    const float v = __fsub_rn(a[i * pitch_a + j], *p);
    idx_out[e] = j; val_out[e] = v;
    flag_nonfinite(status, v);
    *p = __fadd_rn(*p, v);
}

// off[i][b] = first position in worker i's ascending index list with idx >= b * AGG_TILE,
// for b = 0 .. ntiles (so tile b owns entries [off[i][b], off[i][b+1])).
__global__ void agg_offsets_kernel(const int* __restrict__ idx, int n, int k, int ntiles,
                                   int* __restrict__ off) {
    const i64 e = blockIdx.x * (i64)blockDim.x + threadIdx.x;
    const i64 total = (i64)n * (ntiles + 1);
    if (e >= total) return;
    const int i = (int)(e / (ntiles + 1));
    const int b = (int)(e - (i64)i * (ntiles + 1));
    const i64 bound = (i64)b * AGG_TILE;
    const int* __restrict__ ix = idx + (i64)i * k;
    int lo = 0, hi = k;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((i64)ix[mid] < bound) lo = mid + 1; else hi = mid;
    }
    off[e] = lo;
}

// One block per tile of AGG_TILE coordinates.  UPDATE_X: also perform x <- fma(-gamma, g_old, x)
// on the tile before g changes (Algorithm 2 updates x from g^t, then g^{t+1} from the messages).
template <bool UPDATE_X>
__global__ void __launch_bounds__(AGG_BLOCK)
aggregate_kernel(const int* __restrict__ idx, const float* __restrict__ val, const int* __restrict__ off,
                 int n, int k, int ntiles, i64 d, float inv_n, float gamma,
                 float* __restrict__ g, float* __restrict__ x) {
    __shared__ float s[AGG_TILE];
    __shared__ unsigned char touched[AGG_TILE];
    const int b = blockIdx.x;
    const i64 j0 = (i64)b * AGG_TILE;
    for (int t = threadIdx.x; t < AGG_TILE; t += AGG_BLOCK) { s[t] = 0.f; touched[t] = 0; }
    __syncthreads();
    for (int i = 0; i < n; ++i) {
        const int lo = off[(i64)i * (ntiles + 1) + b], hi = off[(i64)i * (ntiles + 1) + b + 1];
        for (int e = lo + threadIdx.x; e < hi; e += AGG_BLOCK) {
            const int t = (int)((i64)idx[(i64)i * k + e] - j0);
            s[t] = __fadd_rn(s[t], val[(i64)i * k + e]);
            touched[t] = 1;
        }
        __syncthreads();
    }
    for (int t = threadIdx.x; t < AGG_TILE; t += AGG_BLOCK) {
        const i64 j = j0 + t;
        if (j >= d) break;
        if (UPDATE_X) {
            const float gj = g[j];
            x[j] = fmaf(-gamma, gj, x[j]);
            if (touched[t]) g[j] = __fadd_rn(gj, __fmul_rn(s[t], inv_n));
        } else if (touched[t]) {
            g[j] = __fadd_rn(g[j], __fmul_rn(s[t], inv_n));
        }
    }
}

// The same aggregation with the tile's message entries first staged in shared memory (one
// parallel gather), so that the ordered pass over the workers touches shared memory only.
// Needs n <= AGG_STAGE_MAX_N; a tile with more than AGG_STAGE_CAP entries takes the direct loop.
constexpr int AGG_STAGE_MAX_N = 1024;
constexpr int AGG_STAGE_CAP = 3072;
constexpr int AGG_OWNER_SCAN_MAX = 512;   // tiles with at most this many entries skip the per-worker loop

template <bool UPDATE_X>
__global__ void __launch_bounds__(AGG_BLOCK)
aggregate_staged_kernel(const int* __restrict__ idx, const float* __restrict__ val, const int* __restrict__ off,
                        int n, int k, int ntiles, i64 d, float inv_n, float gamma,
                        float* __restrict__ g, float* __restrict__ x) {
    __shared__ float s[AGG_TILE];
    __shared__ __align__(4) unsigned short touched[AGG_TILE];   // staged entries per coordinate
    __shared__ int w_start[AGG_STAGE_MAX_N + 1];
    __shared__ int w_lo[AGG_STAGE_MAX_N];
    __shared__ unsigned short e_idx[AGG_STAGE_CAP];
    __shared__ float e_val[AGG_STAGE_CAP];
    __shared__ unsigned scratch[33];
    __shared__ unsigned short multi[AGG_OWNER_SCAN_MAX];
    __shared__ unsigned n_multi;
    const int b = blockIdx.x;
    const i64 j0 = (i64)b * AGG_TILE;
    for (int t = threadIdx.x; t < AGG_TILE; t += AGG_BLOCK) { s[t] = 0.f; touched[t] = 0; }
    if (threadIdx.x == 0) n_multi = 0u;
    unsigned base = 0u;
    for (int c0 = 0; c0 < n; c0 += AGG_BLOCK) {
        const int i = c0 + threadIdx.x;
        int lo = 0, hi = 0;
        if (i < n) { lo = off[(i64)i * (ntiles + 1) + b]; hi = off[(i64)i * (ntiles + 1) + b + 1]; }
        unsigned tot;
        const unsigned pre = block_excl_scan((unsigned)(hi - lo), scratch, tot);
        if (i < n) { w_start[i] = (int)(base + pre); w_lo[i] = lo; }
        base += tot;
    }
    if (threadIdx.x == 0) w_start[n] = (int)base;
    __syncthreads();
    const int total = (int)base;
    if (total <= AGG_STAGE_CAP) {
        for (int e = threadIdx.x; e < total; e += AGG_BLOCK) {
            int lo = 0, hi = n;                      // last worker i with w_start[i] <= e
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (w_start[mid] <= e) lo = mid; else hi = mid;
            }
            const i64 src = (i64)lo * k + w_lo[lo] + (e - w_start[lo]);
            e_idx[e] = (unsigned short)((i64)idx[src] - j0);
            e_val[e] = val[src];
        }
        __syncthreads();
        if (total <= AGG_OWNER_SCAN_MAX) {
            // Few entries: count the entries per coordinate (16-bit counters, two per word).
            unsigned* cnt32 = reinterpret_cast<unsigned*>(touched);
            for (int e = threadIdx.x; e < total; e += AGG_BLOCK) {
                const int t = e_idx[e];
                atomicAdd(&cnt32[t >> 1], (t & 1) ? 0x10000u : 1u);
            }
            __syncthreads();
            // coordinates hit once: the entry is the sum; entries of coordinates hit several times go
            // to a short list and are resolved by whole warps below, in staged (= worker) order
            for (int e = threadIdx.x; e < total; e += AGG_BLOCK) {
                const int t = e_idx[e];
                if (touched[t] == 1) s[t] = __fadd_rn(0.f, e_val[e]);
                else { const unsigned q = atomicAdd(&n_multi, 1u); multi[q] = (unsigned short)e; }
            }
            __syncthreads();
            const int nm = (int)n_multi;                 // <= total <= AGG_OWNER_SCAN_MAX
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            for (int q = warp; q < nm; q += AGG_BLOCK / 32) {
                const int e = multi[q];
                const int t = e_idx[e];
                float acc = 0.f; bool owner = true, seen = false;
                for (int base2 = 0; base2 < total; base2 += 32) {
                    const int p = base2 + lane;
                    unsigned m = __ballot_sync(0xffffffffu, p < total && e_idx[p] == t);
                    if (m && !seen) { owner = (base2 + __ffs(m) - 1) == e; seen = true; }
                    if (!owner) break;                       // warp-uniform
                    while (m) { const int bit = __ffs(m) - 1; acc = __fadd_rn(acc, e_val[base2 + bit]); m &= m - 1; }
                }
                if (owner && lane == 0) s[t] = acc;
            }
            __syncthreads();
        } else
        for (int i = 0; i < n; ++i) {
            const int lo = w_start[i], hi = w_start[i + 1];
            if (lo == hi) continue;                  // uniform: read from shared memory
            for (int e = lo + threadIdx.x; e < hi; e += AGG_BLOCK) {
                const int t = e_idx[e];
                s[t] = __fadd_rn(s[t], e_val[e]);
                touched[t] = 1;
            }
            __syncthreads();
        }
    } else {
        for (int i = 0; i < n; ++i) {
            const int lo = w_lo[i], hi = lo + (w_start[i + 1] - w_start[i]);
            for (int e = lo + threadIdx.x; e < hi; e += AGG_BLOCK) {
                const int t = (int)((i64)idx[(i64)i * k + e] - j0);
                s[t] = __fadd_rn(s[t], val[(i64)i * k + e]);
                touched[t] = 1;
            }
            __syncthreads();
        }
    }
    // dense part of the tile: all loads first, then the updates
    constexpr int PER = AGG_TILE / AGG_BLOCK;
    float gv[PER], xv[PER];
#pragma unroll
    for (int u = 0; u < PER; ++u) {
        const int t = u * AGG_BLOCK + threadIdx.x;
        const i64 j = j0 + t;
        gv[u] = 0.f; xv[u] = 0.f;
        if (j < d && (UPDATE_X || touched[t])) gv[u] = g[j];
        if (UPDATE_X && j < d) xv[u] = x[j];
    }
#pragma unroll
    for (int u = 0; u < PER; ++u) {
        const int t = u * AGG_BLOCK + threadIdx.x;
        const i64 j = j0 + t;
        if (j >= d) continue;
        if (UPDATE_X) x[j] = fmaf(-gamma, gv[u], xv[u]);
        if (touched[t]) g[j] = __fadd_rn(gv[u], __fmul_rn(s[t], inv_n));
    }
}

// x <- fma(-gamma, g, x), elementwise.
__global__ void x_update_kernel(const float* __restrict__ g, float* __restrict__ x, i64 d, float gamma) {
    for (i64 j = blockIdx.x * (i64)blockDim.x + threadIdx.x; j < d; j += (i64)gridDim.x * blockDim.x)
        x[j] = fmaf(-gamma, g[j], x[j]);
}

// Dense initial state g_i^0 = V_i, g^0_j = ((0 + V_0j) + V_1j + ...) * (1/n): the k = d message
// round applied to zero state.
__global__ void dense_init_kernel(const float* __restrict__ V, i64 pitch_v, int n, i64 d, i64 ld,
                                  float inv_n, float* __restrict__ gi, float* __restrict__ g) {
    for (i64 j = blockIdx.x * (i64)blockDim.x + threadIdx.x; j < d; j += (i64)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int i = 0; i < n; ++i) {
            const float v = V[(i64)i * pitch_v + j];
            gi[(i64)i * ld + j] = __fadd_rn(0.f, v);
            s = __fadd_rn(s, v);
        }
        g[j] = __fadd_rn(0.f, __fmul_rn(s, inv_n));
    }
}

}  // namespace ef21
