// Top-k compressor (Section 2.1): exact selection of the k entries of largest |v_j|, ties to the
// lower index, on the difference v = a - b formed on the fly (b may be absent).
//
// General multi-block path, any d < 2^31 and any 1 <= k <= d:
//   1. radix select on the 31-bit magnitude key, most significant digit first (11 + 10 + 10
//      bits): a histogram pass over the elements that still match the prefix, then a one-block
//      "find" step that locates the digit holding the k-th largest key.  The search stops as soon
//      as a whole digit bucket is needed.
//   2. the result is a triple (lo_ge, T, need_ties): an element is selected iff key >= lo_ge, or
//      key == T and fewer than need_ties earlier elements (in index order) have key == T.
//   3. ordered compaction (count per chunk, scan over chunks, write) emits the pairs in ascending
//      index order without any sort.
// Only integer compares decide membership; values are copied bit for bit.
#pragma once
#include "common.cuh"

namespace ef21 {

struct TkState {
    unsigned prefix;     // digits fixed so far (top bits of the threshold key)
    unsigned need;       // how many more elements must come from the current bucket
    unsigned lo_ge;      // every key >= lo_ge is selected
    unsigned T;          // tie key (valid when need_ties > 0)
    unsigned need_ties;  // number of key == T elements selected, lowest indices first
    unsigned done;       // search finished
    unsigned pad0, pad1;
};

constexpr int TK_BINS = 2048;
constexpr int TK_CHUNK = 4096;       // elements per block in the streaming passes
constexpr int TK_BLOCK = 256;

__host__ __device__ inline int tk_level_shift(int level) { return level == 0 ? 20 : (level == 1 ? 10 : 0); }
__host__ __device__ inline int tk_level_bits(int level) { return level == 0 ? 11 : 10; }

__global__ void tk_reset_kernel(TkState* __restrict__ st, unsigned* __restrict__ hist, int batch, unsigned k) {
    const int v = blockIdx.x;
    if (v >= batch) return;
    for (int b = threadIdx.x; b < TK_BINS; b += blockDim.x) hist[(i64)v * TK_BINS + b] = 0u;
    if (threadIdx.x == 0) {
        TkState s;
        s.prefix = 0u; s.need = k; s.lo_ge = 0u; s.T = 0u; s.need_ties = 0u; s.done = 0u; s.pad0 = s.pad1 = 0u;
        st[v] = s;
    }
}

// Histogram of the current digit over the elements whose higher digits equal the prefix.
__global__ void __launch_bounds__(TK_BLOCK)
tk_hist_kernel(const float* __restrict__ a, i64 pitch_a, const float* __restrict__ b, i64 pitch_b, i64 d,
               int level, const TkState* __restrict__ st, unsigned* __restrict__ hist) {
    __shared__ unsigned sh[TK_BINS];
    const int v = blockIdx.y;
    const TkState s = st[v];
    if (s.done) return;
    for (int t = threadIdx.x; t < TK_BINS; t += TK_BLOCK) sh[t] = 0u;
    __syncthreads();
    const float* __restrict__ av = a + (i64)v * pitch_a;
    const float* __restrict__ bv = b ? b + (i64)v * pitch_b : nullptr;
    const int shift = tk_level_shift(level);
    const unsigned mask = (1u << tk_level_bits(level)) - 1u;
    const int hi_shift = shift + tk_level_bits(level);   // bits above the current digit
    const i64 j0 = (i64)blockIdx.x * TK_CHUNK;
    const i64 j1 = min(j0 + (i64)TK_CHUNK, d);
    for (i64 j = j0 + threadIdx.x; j < j1; j += TK_BLOCK) {
        const unsigned key = mag_key(diff_at(av, bv, j));
        const bool match = level == 0 ? true : ((key >> hi_shift) == s.prefix);
        if (match) atomicAdd(&sh[(key >> shift) & mask], 1u);
    }
    __syncthreads();
    unsigned* __restrict__ gh = hist + (i64)v * TK_BINS;
    for (int t = threadIdx.x; t < TK_BINS; t += TK_BLOCK) {
        const unsigned c = sh[t];
        if (c) atomicAdd(&gh[t], c);
    }
}

// One block of 1024 threads per vector: walk the digit buckets from the top, find the one that
// holds the need-th largest remaining key, extend the prefix, decide whether the search is over,
// and clear the histogram for the next level.
__global__ void __launch_bounds__(1024)
tk_find_kernel(TkState* __restrict__ st, unsigned* __restrict__ hist, int level) {
    __shared__ unsigned scratch[33];
    const int v = blockIdx.x;
    TkState s = st[v];
    unsigned* __restrict__ gh = hist + (i64)v * TK_BINS;
    if (s.done) return;
    const int p = threadIdx.x;                 // position from the top: buckets 2047-2p and 2046-2p
    const int b_hi = TK_BINS - 1 - 2 * p, b_lo = b_hi - 1;
    const unsigned c_hi = gh[b_hi], c_lo = gh[b_lo];
    unsigned total;
    const unsigned above = block_excl_scan(c_hi + c_lo, scratch, total);
    int found = -1; unsigned above_found = 0u, pop = 0u;
    if (above < s.need && s.need <= above + c_hi) { found = b_hi; above_found = above; pop = c_hi; }
    else if (above + c_hi < s.need && s.need <= above + c_hi + c_lo) { found = b_lo; above_found = above + c_hi; pop = c_lo; }
    gh[b_hi] = 0u; gh[b_lo] = 0u;
    if (found >= 0) {
        const int bits = tk_level_bits(level), shift = tk_level_shift(level);
        s.prefix = (s.prefix << bits) | (unsigned)found;
        s.need -= above_found;
        if (s.need == pop) {               // the whole bucket is selected: nothing left to refine
            s.lo_ge = s.prefix << shift; s.T = 0u; s.need_ties = 0u; s.done = 1u;
        } else if (level == 2) {           // prefix is the exact key of the k-th element; ties remain
            s.T = s.prefix; s.lo_ge = s.prefix + 1u; s.need_ties = s.need; s.done = 1u;
        }
        st[v] = s;
    }
}

// Per chunk: number of keys >= lo_ge and number of keys == T (only when need_ties > 0).
__global__ void __launch_bounds__(TK_BLOCK)
tk_count_kernel(const float* __restrict__ a, i64 pitch_a, const float* __restrict__ b, i64 pitch_b, i64 d,
                const TkState* __restrict__ st, uint2* __restrict__ chunk_counts, int nchunks) {
    __shared__ unsigned wsum[2][TK_BLOCK / 32];
    const int v = blockIdx.y;
    const TkState s = st[v];
    const float* __restrict__ av = a + (i64)v * pitch_a;
    const float* __restrict__ bv = b ? b + (i64)v * pitch_b : nullptr;
    const i64 j0 = (i64)blockIdx.x * TK_CHUNK;
    const i64 j1 = min(j0 + (i64)TK_CHUNK, d);
    unsigned ge = 0u, tie = 0u;
    for (i64 j = j0 + threadIdx.x; j < j1; j += TK_BLOCK) {
        const unsigned key = mag_key(diff_at(av, bv, j));
        ge += key >= s.lo_ge ? 1u : 0u;
        tie += (s.need_ties && key == s.T) ? 1u : 0u;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ge += __shfl_xor_sync(0xffffffffu, ge, o);
        tie += __shfl_xor_sync(0xffffffffu, tie, o);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { wsum[0][warp] = ge; wsum[1][warp] = tie; }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned g2 = 0u, t2 = 0u;
        for (int w = 0; w < TK_BLOCK / 32; ++w) { g2 += wsum[0][w]; t2 += wsum[1][w]; }
        chunk_counts[(i64)v * nchunks + blockIdx.x] = make_uint2(g2, t2);
    }
}

// Exclusive scan of the chunk counts of one vector (one block per vector), in place.
__global__ void __launch_bounds__(1024)
tk_scan_kernel(uint2* __restrict__ chunk_counts, int nchunks) {
    __shared__ unsigned scratch[33];
    uint2* __restrict__ cc = chunk_counts + (i64)blockIdx.x * nchunks;
    unsigned base_ge = 0u, base_tie = 0u;
    for (int c0 = 0; c0 < nchunks; c0 += 1024) {
        const int c = c0 + threadIdx.x;
        uint2 val = c < nchunks ? cc[c] : make_uint2(0u, 0u);
        unsigned tot_ge, tot_tie;
        const unsigned e_ge = block_excl_scan(val.x, scratch, tot_ge);
        const unsigned e_tie = block_excl_scan(val.y, scratch, tot_tie);
        if (c < nchunks) cc[c] = make_uint2(base_ge + e_ge, base_tie + e_tie);
        base_ge += tot_ge; base_tie += tot_tie;
    }
}

// Ordered compaction of one chunk: elements are visited in index order, 256 at a time.
__global__ void __launch_bounds__(TK_BLOCK)
tk_write_kernel(const float* __restrict__ a, i64 pitch_a, const float* __restrict__ b, i64 pitch_b, i64 d,
                const TkState* __restrict__ st, const uint2* __restrict__ chunk_prefix, int nchunks,
                int k, int* __restrict__ idx_out, float* __restrict__ val_out, unsigned* status) {
    __shared__ unsigned scratch[33];
    const int v = blockIdx.y;
    const TkState s = st[v];
    const float* __restrict__ av = a + (i64)v * pitch_a;
    const float* __restrict__ bv = b ? b + (i64)v * pitch_b : nullptr;
    const uint2 pre = chunk_prefix[(i64)v * nchunks + blockIdx.x];
    unsigned ge_before = pre.x, tie_before = pre.y;
    int* __restrict__ io = idx_out + (i64)v * k;
    float* __restrict__ vo = val_out + (i64)v * k;
    const i64 j0 = (i64)blockIdx.x * TK_CHUNK;
    const i64 j1 = min(j0 + (i64)TK_CHUNK, d);
    for (i64 base = j0; base < j1; base += TK_BLOCK) {
        const i64 j = base + threadIdx.x;
        float val = 0.f; unsigned is_ge = 0u, is_tie = 0u;
        if (j < j1) {
            val = diff_at(av, bv, j);
            const unsigned key = mag_key(val);
            is_ge = key >= s.lo_ge ? 1u : 0u;
            is_tie = (s.need_ties && key == s.T) ? 1u : 0u;
        }
        unsigned tot;
        const unsigned packed = block_excl_scan(is_ge | (is_tie << 16), scratch, tot);
        const unsigned my_ge = ge_before + (packed & 0xffffu);
        const unsigned my_tie = tie_before + (packed >> 16);
        if (is_ge) {
            const unsigned pos = my_ge + min(my_tie, s.need_ties);
            if (pos < (unsigned)k) { io[pos] = (int)j; vo[pos] = val; flag_nonfinite(status, val); }
        } else if (is_tie && my_tie < s.need_ties) {
            const unsigned pos = my_ge + my_tie;
            if (pos < (unsigned)k) { io[pos] = (int)j; vo[pos] = val; flag_nonfinite(status, val); }
        }
        ge_before += tot & 0xffffu;
        tie_before += tot >> 16;
    }
}

// ---------------------------------------------------------------------------------------------
// Short vectors (d <= TKS_MAX_D): the whole selection in ONE launch, one block per vector.
//   v = a - b is formed once into shared memory; radix select on the 31-bit key with digits of
//   8 + 8 + 8 + 7 bits (shared-memory histogram over the entries that match the prefix, warp 0
//   locates the digit that holds the k-th largest key); every thread then owns a contiguous piece of
//   the vector, counts its entries above the threshold key T and equal to it, one block scan turns
//   the counts into output positions (ties are taken in index order until need_ties are used up),
//   and the pairs are written in ascending index order.  apply_to (optional): the vector that receives
//   g_i + c_i on the selected coordinates in the same launch.
// ---------------------------------------------------------------------------------------------
constexpr int TKS_MAX_D = 8192;
constexpr int TKS_BLOCK = 512;

__global__ void __launch_bounds__(TKS_BLOCK)
tk_small_kernel(const float* __restrict__ a, i64 pitch_a, const float* b, i64 pitch_b,
                int d, int k, int* __restrict__ idx_out, float* __restrict__ val_out, float* apply_to, i64 pitch_apply,
                unsigned* status) {
    extern __shared__ __align__(16) unsigned char tks_smem[];
    float* vs = reinterpret_cast<float*>(tks_smem);                     // [d]
    __shared__ unsigned hist[256];
    __shared__ unsigned scan_scratch[33];
    __shared__ unsigned sh_prefix, sh_need;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* __restrict__ av = a + (i64)blockIdx.x * pitch_a;
    const float* bv = b ? b + (i64)blockIdx.x * pitch_b : nullptr;      // may be the vector apply_to updates below
    for (int j = tid; j < d; j += TKS_BLOCK) vs[j] = bv ? __fsub_rn(av[j], bv[j]) : av[j];
    if (tid == 0) { sh_prefix = 0u; sh_need = (unsigned)k; }
    // radix select: after the four digits sh_prefix is the k-th largest key T and sh_need the number of
    // entries equal to T that belong to the Top-k
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = pass == 0 ? 23 : (pass == 1 ? 15 : (pass == 2 ? 7 : 0));
        const int bits = pass == 3 ? 7 : 8;
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const unsigned prefix = sh_prefix;
        for (int j = tid; j < d; j += TKS_BLOCK) {
            const unsigned key = mag_key(vs[j]);
            if ((key >> (shift + bits)) == prefix) atomicAdd(&hist[(key >> shift) & ((1u << bits) - 1u)], 1u);
        }
        __syncthreads();
        if (warp == 0) {
            // lane 0 owns the top eight bins, lane 31 the lowest eight; walk down until `need` is covered
            const unsigned need = sh_need;
            unsigned c[8], sum = 0u;
#pragma unroll
            for (int q = 0; q < 8; ++q) { c[q] = hist[255 - (8 * lane + q)]; sum += c[q]; }
            const unsigned incl = warp_incl_scan(sum), excl = incl - sum;
            if (excl < need && need <= incl) {
                unsigned rest = need - excl;
                int bin = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (rest != 0u) {
                        if (c[q] >= rest) { bin = 255 - (8 * lane + q); sh_need = rest; rest = 0u; }
                        else rest -= c[q];
                    }
                }
                sh_prefix = (prefix << bits) | (unsigned)bin;
            }
        }
        __syncthreads();
    }
    const unsigned T = sh_prefix, need_ties = sh_need;
    // contiguous piece per thread, so that thread order is index order
    const int seg = (d + TKS_BLOCK - 1) / TKS_BLOCK;
    const int j0 = min(tid * seg, d), j1 = min(j0 + seg, d);
    unsigned gt = 0u, eq = 0u;
    for (int j = j0; j < j1; ++j) {
        const unsigned key = mag_key(vs[j]);
        gt += key > T ? 1u : 0u;
        eq += key == T ? 1u : 0u;
    }
    unsigned total;
    const unsigned before = block_excl_scan((gt << 16) | eq, scan_scratch, total);     // counts <= 8192 each
    unsigned eq_before = before & 0xffffu;
    const unsigned gt_before = before >> 16;
    unsigned pos = gt_before + min(eq_before, need_ties);
    int* __restrict__ io = idx_out + (i64)blockIdx.x * k;
    float* __restrict__ vo = val_out + (i64)blockIdx.x * k;
    for (int j = j0; j < j1; ++j) {
        const float v = vs[j];
        const unsigned key = mag_key(v);
        bool take = key > T;
        if (key == T) { take = eq_before < need_ties; ++eq_before; }
        if (take) {
            io[pos] = j; vo[pos] = v; ++pos;
            flag_nonfinite(status, v);
            if (apply_to) {            // g_i <- g_i + c_i on the selected coordinate (Algorithm 2, node loop)
                float* p = apply_to + (i64)blockIdx.x * pitch_apply + j;
                *p = __fadd_rn(*p, v);
            }
        }
    }
}

}  // namespace ef21
