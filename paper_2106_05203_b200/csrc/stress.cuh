// Fused difference + exact Top-k for long vectors (d >= 2^18, k <= 8192), one pass over HBM.
//
// The vectors a_i (local gradient) and g_i are each read from HBM once per round:
//   1. sample:   65,536 entries of v_i = a_i - g_i (64 blocks of 1,024 consecutive entries) give a
//                threshold tau_i on the magnitude key under which about max(2k, k+2048) entries of
//                the whole vector are expected to lie above.
//   2. collect:  the single streaming pass.  Every warp owns a region of 4,096 consecutive entries
//                and appends the entries with key >= tau_i to its own slot array, in index order
//                (ballot ranks), so the candidate set of a vector is already sorted by index.  A
//                record is (index, v, g_i + v): the updated state value travels with the candidate.
//   3. finish:   one block per vector stages the candidates in shared memory, finds the exact k-th
//                key by radix select, breaks ties toward the lower index by an ordered scan, writes
//                the k pairs in ascending index order and stores g_i + c_i on the selected
//                coordinates (no read-modify-write: the new value came with the candidate).  On
//                request it also writes where each tile of coordinates begins in the message (the
//                offsets the aggregation needs), so no separate search kernel runs.
// The threshold only decides speed, never the result: if a vector ends up with fewer than k
// candidates, more than the staging capacity, or an overflowing region, its finish block runs the
// exact selection over the whole vector instead (slow, same output bit for bit).
#pragma once
#include "common.cuh"

namespace ef21 {

constexpr int ST_SUB = 4096;            // entries per region (one warp)
constexpr int ST_REGION_CAP = 128;      // candidate slots per region
constexpr int ST_COLLECT_WARPS = 8;
#ifndef ST_COLLECT_UNROLL
#define ST_COLLECT_UNROLL 1
#endif
#ifndef ST_COLLECT_MIN_BLOCKS
#define ST_COLLECT_MIN_BLOCKS 8
#endif
constexpr int ST_SAMPLE_BLOCKS = 64;
constexpr int ST_SAMPLE_LEN = 1024;
constexpr int ST_THREADS = 1024;        // sample / finish block size
constexpr int ST_CAND_CAP = 16384;      // candidates staged in shared memory
constexpr i64 ST_MIN_D = 262144;
constexpr int ST_MAX_K = 6144;

// All 1024 threads: given a 2048-bin histogram in shared memory (bins ordered by key digit), find
// the bin that holds the need-th largest entry.  Returns bin, number of entries in higher bins,
// and the bin's population through shared memory.
__device__ __forceinline__ void block_find_bin(const unsigned* hist, unsigned need, unsigned* scratch,
                                               unsigned* result /* [3] shared */) {
    const int p = threadIdx.x;
    const int b_hi = 2047 - 2 * p, b_lo = b_hi - 1;
    const unsigned c_hi = hist[b_hi], c_lo = hist[b_lo];
    unsigned total;
    const unsigned above = block_excl_scan(c_hi + c_lo, scratch, total);
    if (above < need && need <= above + c_hi) { result[0] = (unsigned)b_hi; result[1] = above; result[2] = c_hi; }
    else if (above + c_hi < need && need <= above + c_hi + c_lo) { result[0] = (unsigned)b_lo; result[1] = above + c_hi; result[2] = c_lo; }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// 1. threshold from a sample
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(ST_THREADS)
st_sample_kernel(const float* __restrict__ a, i64 pitch_a, const float* __restrict__ b, i64 pitch_b, i64 d,
                 unsigned rank, unsigned* __restrict__ thr, unsigned* __restrict__ flags) {
    __shared__ unsigned hist[2048];
    __shared__ unsigned scratch[33];
    __shared__ unsigned res[3];
    const int i = blockIdx.x, t = threadIdx.x;
    const float* __restrict__ av = a + (i64)i * pitch_a;
    const float* __restrict__ bv = b ? b + (i64)i * pitch_b : nullptr;
    const i64 stride = d / ST_SAMPLE_BLOCKS;            // >= ST_SAMPLE_LEN because d >= ST_MIN_D
    for (int q = t; q < 2048; q += ST_THREADS) hist[q] = 0u;
    __syncthreads();
#pragma unroll 8
    for (int s = 0; s < ST_SAMPLE_BLOCKS; ++s)
        atomicAdd(&hist[mag_key(diff_at(av, bv, (i64)s * stride + t)) >> 20], 1u);
    __syncthreads();
    block_find_bin(hist, rank, scratch, res);
    const unsigned b0 = res[0], need1 = rank - res[1];
    __syncthreads();
    for (int q = t; q < 2048; q += ST_THREADS) hist[q] = 0u;
    __syncthreads();
#pragma unroll 8
    for (int s = 0; s < ST_SAMPLE_BLOCKS; ++s) {
        const unsigned key = mag_key(diff_at(av, bv, (i64)s * stride + t));
        if ((key >> 20) == b0) atomicAdd(&hist[(key >> 10) & 1023u], 1u);
    }
    __syncthreads();
    block_find_bin(hist, need1, scratch, res);
    if (t == 0) {
        unsigned tau = (b0 << 20) | (res[0] << 10);
        thr[i] = tau ? tau : 1u;          // never collect exact zeros
        flags[i] = 0u;
    }
}

// ---------------------------------------------------------------------------------------------
// helpers of the exact selection (radix-select bookkeeping, whole-vector fallback)
// ---------------------------------------------------------------------------------------------

// Radix-select bookkeeping shared by the fast and the slow variant: digits of 11/10/10 bits.
struct SelectState { unsigned prefix, need, lo_ge, T, need_ties, done; };

__device__ __forceinline__ void select_advance(SelectState& s, int level, const unsigned* res) {
    const int bits = level == 0 ? 11 : 10, shift = level == 0 ? 20 : (level == 1 ? 10 : 0);
    s.prefix = (s.prefix << bits) | res[0];
    s.need -= res[1];
    if (s.need == res[2]) { s.lo_ge = s.prefix << shift; s.T = 0u; s.need_ties = 0u; s.done = 1u; }
    else if (level == 2) { s.T = s.prefix; s.lo_ge = s.prefix + 1u; s.need_ties = s.need; s.done = 1u; }
}

__device__ __forceinline__ bool select_match(unsigned key, int level, unsigned prefix, unsigned& bin) {
    if (level == 0) { bin = key >> 20; return true; }
    if (level == 1) { bin = (key >> 10) & 1023u; return (key >> 20) == prefix; }
    bin = key & 1023u;
    return (key >> 10) == prefix;
}

// Whole-vector exact Top-k by one block (fallback): three histogram passes, one ordered pass.
__device__ void st_slow_exact(const float* av, const float* bv, i64 d, int k,
                              int* __restrict__ idx_out, float* __restrict__ val_out, float* gi_row,
                              unsigned* hist, unsigned* scratch, unsigned* res, unsigned* status) {
    SelectState s; s.prefix = 0u; s.need = (unsigned)k; s.lo_ge = 0u; s.T = 0u; s.need_ties = 0u; s.done = 0u;
    for (int level = 0; level < 3 && !s.done; ++level) {
        for (int q = threadIdx.x; q < 2048; q += ST_THREADS) hist[q] = 0u;
        __syncthreads();
        for (i64 j = threadIdx.x; j < d; j += ST_THREADS) {
            unsigned bin;
            if (select_match(mag_key(diff_at(av, bv, j)), level, s.prefix, bin)) atomicAdd(&hist[bin], 1u);
        }
        __syncthreads();
        block_find_bin(hist, s.need, scratch, res);
        select_advance(s, level, res);
        __syncthreads();
    }
    unsigned ge_before = 0u, tie_before = 0u;
    for (i64 base = 0; base < d; base += ST_THREADS) {
        const i64 j = base + threadIdx.x;
        float val = 0.f; unsigned is_ge = 0u, is_tie = 0u;
        if (j < d) {
            val = diff_at(av, bv, j);
            const unsigned key = mag_key(val);
            is_ge = key >= s.lo_ge ? 1u : 0u;
            is_tie = (s.need_ties && key == s.T) ? 1u : 0u;
        }
        unsigned tot;
        const unsigned packed = block_excl_scan(is_ge | (is_tie << 16), scratch, tot);
        const unsigned my_ge = ge_before + (packed & 0xffffu), my_tie = tie_before + (packed >> 16);
        const bool sel = is_ge || (is_tie && my_tie < s.need_ties);
        if (sel) {
            const unsigned pos = is_ge ? my_ge + min(my_tie, s.need_ties) : my_ge + my_tie;
            if (pos < (unsigned)k) {
                idx_out[pos] = (int)j; val_out[pos] = val;
                flag_nonfinite(status, val);
                if (gi_row) gi_row[j] = __fadd_rn(gi_row[j], val);
            }
        }
        ge_before += tot & 0xffffu;
        tie_before += tot >> 16;
    }
}

// ---------------------------------------------------------------------------------------------
// 2. the streaming pass
// ---------------------------------------------------------------------------------------------
// grid = (ceil(nreg / 8), batch), block = 256 threads: one warp per region of 4,096 entries.
template <bool VEC>
__global__ void __launch_bounds__(ST_COLLECT_WARPS * 32, ST_COLLECT_MIN_BLOCKS)
st_collect_kernel(const float* __restrict__ a, i64 pitch_a, const float* __restrict__ b, i64 pitch_b, i64 d,
                  int nreg, const unsigned* __restrict__ thr, int4* __restrict__ cand,
                  int* __restrict__ region_cnt, unsigned* __restrict__ flags) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int i = blockIdx.y;
    const float* __restrict__ av = a + (i64)i * pitch_a;
    const bool has_b = b != nullptr;
    const float* __restrict__ bv = has_b ? b + (i64)i * pitch_b : nullptr;
    const int region = blockIdx.x * ST_COLLECT_WARPS + warp;
    if (region < nreg) {
        const unsigned tau = thr[i];
        const i64 base = (i64)region * ST_SUB;
        int4* out = cand + ((i64)i * nreg + region) * ST_REGION_CAP;
        const unsigned lt = (1u << lane) - 1u;
        int cnt = 0;
        constexpr int UNROLL = ST_COLLECT_UNROLL;
        for (int it0 = 0; it0 < ST_SUB / 128; it0 += UNROLL) {
            float v[UNROLL][4], gold[UNROLL][4];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const i64 j0 = base + (i64)(it0 + u) * 128 + 4 * lane;
                if (VEC && j0 + 3 < d) {
                    const float4 x4 = __ldcs(reinterpret_cast<const float4*>(av + j0));
                    if (has_b) {
                        const float4 g4 = __ldcs(reinterpret_cast<const float4*>(bv + j0));
                        gold[u][0] = g4.x; gold[u][1] = g4.y; gold[u][2] = g4.z; gold[u][3] = g4.w;
                        v[u][0] = __fsub_rn(x4.x, g4.x); v[u][1] = __fsub_rn(x4.y, g4.y);
                        v[u][2] = __fsub_rn(x4.z, g4.z); v[u][3] = __fsub_rn(x4.w, g4.w);
                    } else {
                        gold[u][0] = gold[u][1] = gold[u][2] = gold[u][3] = 0.f;
                        v[u][0] = x4.x; v[u][1] = x4.y; v[u][2] = x4.z; v[u][3] = x4.w;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        gold[u][e] = (has_b && j0 + e < d) ? bv[j0 + e] : 0.f;
                        v[u][e] = (j0 + e < d) ? (has_b ? __fsub_rn(av[j0 + e], gold[u][e]) : av[j0 + e]) : 0.f;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const i64 j0 = base + (i64)(it0 + u) * 128 + 4 * lane;
                bool pr[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) pr[e] = mag_key(v[u][e]) >= tau;
                const unsigned any = __ballot_sync(0xffffffffu, pr[0] | pr[1] | pr[2] | pr[3]);
                if (any) {
                    unsigned bm[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) bm[e] = __ballot_sync(0xffffffffu, pr[e]);
                    int pos = cnt + __popc(bm[0] & lt) + __popc(bm[1] & lt) + __popc(bm[2] & lt) + __popc(bm[3] & lt);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (pr[e]) {
                            if (pos < ST_REGION_CAP) {
                                const float gnew = __fadd_rn(gold[u][e], v[u][e]);
                                out[pos] = make_int4((int)(j0 + e), __float_as_int(v[u][e]), __float_as_int(gnew), 0);
                            }
                            ++pos;
                        }
                    cnt += __popc(bm[0]) + __popc(bm[1]) + __popc(bm[2]) + __popc(bm[3]);
                }
            }
        }
        if (lane == 0) {
            region_cnt[(i64)i * nreg + region] = cnt;
            if (cnt > ST_REGION_CAP) atomicOr(&flags[i], 1u);
        }
    }

}

// ---------------------------------------------------------------------------------------------
// 3. exact selection among the candidates (or, rarely, over the whole vector)
// ---------------------------------------------------------------------------------------------
// grid = batch, block = 1024 threads, dynamic shared memory = ST_CAND_CAP * 12 + 2048 * 4 bytes.
// gi_rows: if not null, row i receives g_i + c_i on the selected coordinates (row pitch ld); b may
// alias gi_rows.
__global__ void __launch_bounds__(ST_THREADS, 1)
st_finish_kernel(const float* a, i64 pitch_a, const float* b, i64 pitch_b, i64 d, int nreg, int k,
                 const int4* __restrict__ cand, const int* __restrict__ region_cnt,
                 const unsigned* __restrict__ flags, int* __restrict__ idx_out, float* __restrict__ val_out,
                 float* gi_rows, i64 ld, unsigned* __restrict__ slow_count,
                 int* __restrict__ tile_off, int ntiles, int tile, unsigned* status) {
    extern __shared__ __align__(16) unsigned char st_smem[];
    __shared__ unsigned scratch[33];
    __shared__ unsigned res[3];
    const int i = blockIdx.x;
    const float* av = a + (i64)i * pitch_a;
    const float* bv = b ? b + (i64)i * pitch_b : nullptr;      // may alias the g_i row written below
    int* cidx = reinterpret_cast<int*>(st_smem);                       // [ST_CAND_CAP]
    float* cval = reinterpret_cast<float*>(cidx + ST_CAND_CAP);        // [ST_CAND_CAP]
    float* cnew = cval + ST_CAND_CAP;                                  // [ST_CAND_CAP] g_i + v
    unsigned* hist = reinterpret_cast<unsigned*>(cnew + ST_CAND_CAP);  // [2048]
    int* __restrict__ io = idx_out + (i64)i * k;
    float* __restrict__ vo = val_out + (i64)i * k;
    float* gi_row = gi_rows ? gi_rows + (i64)i * ld : nullptr;

    // stage the candidates in index order: per group of 1024 regions, prefix-sum the region counts
    // (thread t holds region r0 + t), then every warp copies the lists of its 32 regions, eight
    // regions in flight, one lane per candidate
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned total = 0u;
    bool bad = flags[i] != 0u;
    for (int r0 = 0; r0 < nreg; r0 += ST_THREADS) {
        const int r = r0 + threadIdx.x;
        const unsigned c = r < nreg ? (unsigned)region_cnt[(i64)i * nreg + r] : 0u;
        unsigned tot;
        const unsigned pre = block_excl_scan(c, scratch, tot);
        if (!bad && total + tot <= (unsigned)ST_CAND_CAP) {
            const int4* __restrict__ src = cand + ((i64)i * nreg + r0 + warp * 32) * ST_REGION_CAP;
            constexpr int U = 8;
            for (int rr0 = 0; rr0 < 32; rr0 += U) {
                int4 w[U];
                unsigned cu[U], pu[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    cu[u] = __shfl_sync(0xffffffffu, c, rr0 + u);
                    pu[u] = __shfl_sync(0xffffffffu, pre, rr0 + u);
                    if ((unsigned)lane < cu[u]) w[u] = src[(rr0 + u) * ST_REGION_CAP + lane];
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if ((unsigned)lane < cu[u]) {
                        const unsigned at = total + pu[u] + (unsigned)lane;
                        cidx[at] = w[u].x; cval[at] = __int_as_float(w[u].y); cnew[at] = __int_as_float(w[u].z);
                    }
                    for (unsigned more = 32u; more < cu[u]; more += 32u) {       // rare: a list longer than a warp
                        if (more + (unsigned)lane < cu[u]) {
                            const int4 x = src[(rr0 + u) * ST_REGION_CAP + more + lane];
                            const unsigned at = total + pu[u] + more + (unsigned)lane;
                            cidx[at] = x.x; cval[at] = __int_as_float(x.y); cnew[at] = __int_as_float(x.z);
                        }
                    }
                }
            }
        }
        total += tot;
        __syncthreads();
    }
    if (bad || total < (unsigned)k || total > (unsigned)ST_CAND_CAP) {
        if (threadIdx.x == 0 && slow_count) atomicAdd(slow_count, 1u);
        st_slow_exact(av, bv, d, k, io, vo, gi_row, hist, scratch, res, status);
        if (tile_off) {
            __syncthreads();                         // the block's own writes to io are visible to it now
            int* off = tile_off + (i64)i * (ntiles + 1);
            for (int b = threadIdx.x; b <= ntiles; b += ST_THREADS) {
                const i64 bound = (i64)b * tile;
                int lo = 0, hi = k;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if ((i64)io[mid] < bound) lo = mid + 1; else hi = mid;
                }
                off[b] = lo;
            }
        }
        return;
    }

    SelectState s; s.prefix = 0u; s.need = (unsigned)k; s.lo_ge = 0u; s.T = 0u; s.need_ties = 0u; s.done = 0u;
    for (int level = 0; level < 3 && !s.done; ++level) {
        for (int q = threadIdx.x; q < 2048; q += ST_THREADS) hist[q] = 0u;
        __syncthreads();
        for (unsigned e = threadIdx.x; e < total; e += ST_THREADS) {
            unsigned bin;
            if (select_match(mag_key(cval[e]), level, s.prefix, bin)) atomicAdd(&hist[bin], 1u);
        }
        __syncthreads();
        block_find_bin(hist, s.need, scratch, res);
        select_advance(s, level, res);
        __syncthreads();
    }
    // ordered compaction: thread t owns the contiguous candidates [t*q, (t+1)*q)
    const unsigned q = (total + ST_THREADS - 1) / ST_THREADS;
    const unsigned e0 = min(threadIdx.x * q, total), e1 = min(e0 + q, total);
    unsigned n_ge = 0u, n_tie = 0u;
    for (unsigned e = e0; e < e1; ++e) {
        const unsigned key = mag_key(cval[e]);
        n_ge += key >= s.lo_ge ? 1u : 0u;
        n_tie += (s.need_ties && key == s.T) ? 1u : 0u;
    }
    unsigned tot;
    const unsigned packed = block_excl_scan(n_ge | (n_tie << 16), scratch, tot);
    // Pass A: the state update g_i + c_i on the selected coordinates (scattered stores).  Pass B, after
    // everybody has read its cnew entries: the selected (index, value) pairs go, compacted and in
    // order, into the space of cnew.  Pass C writes them out with coalesced stores and derives, from
    // neighbouring indices, where each tile of `tile` coordinates starts in the message.
    int2* out2 = reinterpret_cast<int2*>(cnew);                 // [k] <= ST_CAND_CAP / 2 pairs
    for (int pass = 0; pass < 2; ++pass) {
        unsigned my_ge = packed & 0xffffu, my_tie = packed >> 16;
        for (unsigned e = e0; e < e1; ++e) {
            const float val = cval[e];
            const unsigned key = mag_key(val);
            const bool is_ge = key >= s.lo_ge;
            const bool is_tie = s.need_ties && key == s.T;
            if (is_ge || (is_tie && my_tie < s.need_ties)) {
                const unsigned pos = is_ge ? my_ge + min(my_tie, s.need_ties) : my_ge + my_tie;
                if (pos < (unsigned)k) {
                    if (pass == 0) { if (gi_row) gi_row[cidx[e]] = cnew[e]; }      // g_i + c_i, computed when the entry was read
                    else out2[pos] = make_int2(cidx[e], __float_as_int(val));
                }
            }
            my_ge += is_ge ? 1u : 0u;
            my_tie += is_tie ? 1u : 0u;
        }
        __syncthreads();
    }
    int* off = tile_off ? tile_off + (i64)i * (ntiles + 1) : nullptr;
    for (int p0 = threadIdx.x; p0 < k; p0 += ST_THREADS) {
        const int2 me = out2[p0];
        io[p0] = me.x; vo[p0] = __int_as_float(me.y);
        flag_nonfinite(status, __int_as_float(me.y));
        if (off) {
            const int t_prev = p0 > 0 ? out2[p0 - 1].x / tile : -1;
            const int t_me = me.x / tile;
            for (int b = t_prev + 1; b <= t_me; ++b) off[b] = p0;          // tiles that begin at this entry
            if (p0 == k - 1)
                for (int b = t_me + 1; b <= ntiles; ++b) off[b] = k;       // nothing left for the tiles behind the last entry
        }
    }
}

}  // namespace ef21
