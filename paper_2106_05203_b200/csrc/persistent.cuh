// EF21 (Algorithm 2) as ONE persistent kernel for small dimensions (d <= 512, k <= 32):
// all `steps` iterations run inside a single launch, the shards stay on chip.
//
// Mapping.  Worker i is a thread-block cluster of C blocks; block c of the cluster owns a
// contiguous slice of the worker's rows, held in registers (REG), in shared memory (SMEM) or
// re-read from global memory / L2 every iteration (GMEM).  Every block keeps its own replica of
// x and g, so the only grid-wide dependency per iteration is the exchange of the n messages
// c_i (k pairs each), which plays the role of the paper's "send c_i to the master / broadcast x":
//
//   1. x <- fma(-gamma, g, x)                                   (every block, its replica)
//   2. rows in batches of RB per warp: margins a_r.x by a transposed warp reduction (lane L ends
//      up with the margin of row L/(32/RB)), residual rho_r, rank-1 accumulation rho_r a_r
//   3. block partial -> leader block of the cluster: 16-byte st.async stores into the leader's shared
//      memory that credit an mbarrier there; the senders do not wait, the leader waits (bounded) for
//      the byte count of all partials
//   4. leader block: grad_i = sum/m_i + regulariser' and v = grad_i - g_i, one coordinate per
//      thread; Top-k either by k rounds of a warp arg-max on (|v| bits, lower index wins) or, for
//      larger k, by rank counting (every coordinate counts the entries ahead of it); g_i += c_i;
//      k packed 64-bit words (epoch:16 | index:16 | value bits:32) go into a double-buffered global
//      slot array
//   5. every block polls the n*k words of this iteration's epoch (bounded spin); then each
//      coordinate thread adds the matching values in ascending worker order (few messages), or warp 0
//      folds the messages worker by worker into running sums (many messages): g += (1/n) sum c_i
//
// All summation orders are fixed by the launch shape, so two runs give identical bits.  A wait
// that exceeds its spin limit records EF21_ERR_TIMEOUT in the status word; from then on every
// block skips work but keeps arriving at the cluster barriers, so the kernel always terminates.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace ef21 {
namespace cg = cooperative_groups;

constexpr int PK_MAX_THREADS = 512;     // the kernel is instantiated for 256 and 512 threads per block
constexpr int PK_MAX_K = 32;
constexpr int PK_MAX_MSGS = 2048;       // n*k words staged in shared memory
constexpr int PK_SCAN_MAX_MSGS = 128;   // up to this many messages every coordinate thread scans them all
constexpr int PK_TABLE_MAX_BYTES = 64 * 1024;   // largest [n][ld] message table kept in shared memory
constexpr unsigned PK_NO_ENTRY = 0xffffffffu;   // table cell without a message (a NaN pattern no finite value has)
enum { PK_SRC_REG = 0, PK_SRC_SMEM = 1, PK_SRC_GMEM = 2 };

struct PersistParams {
    const float* A;            // [N][ld], padded, read-only
    const float* y;            // [N]
    const i64* row_off;        // [n+1]
    float* x;                  // [ld]
    float* g;                  // [ld]
    float* gi;                 // [n][ld]
    int* msg_idx;              // [n][k] last messages (written at the final iteration)
    float* msg_val;
    int* plus_choice;          // [n] EF21+: branch taken at the final iteration (0 Markov compressor, 1 plain)
    unsigned long long* slots; // [2][n*k]
    unsigned* status;
    int n, d, ld, k, C, steps;
    int objective;             // 0 logistic loss, 1 least squares
    int slice_rows;            // capacity (rows) of the shared-memory slice (SMEM source)
    int use_table;             // 1: received messages are scattered into a [n][ld] table in shared memory
    float gamma, lambda, inv_n;
    unsigned spin_limit;
    unsigned epoch0;           // epoch of the first iteration minus one
};

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// ---- distributed-shared-memory hand-off: remote stores that signal an mbarrier in the target block
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned map_to_rank(unsigned addr, unsigned rank) {
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init_cluster() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_parity(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0u;
}
// 16-byte store into another block's shared memory; on arrival 16 bytes are credited to that block's mbarrier.
__device__ __forceinline__ void st_async_f4(unsigned remote_dst, float4 v, unsigned remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(remote_dst), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(remote_bar) : "memory");
}

__device__ __forceinline__ float comp_of(const float4& v, int c) {
    return c == 0 ? v.x : (c == 1 ? v.y : (c == 2 ? v.z : v.w));
}

// EXTRA > 0: a warp's batch has RB + EXTRA rows; the first RB go through the transposed reduction, each
// extra row through a plain butterfly sum (for shards whose rows per warp just exceed a power of two).
// PLUS: EF21+ (Algorithm 3).  The leader also selects C(grad_i), compares the two distortions and keeps the
// better vector; a message carries the branch in bit 15 of its index field; every block keeps a replica of
// all g_i and recomputes g = (1/n) sum_i g_i (ascending i, one multiply) after each exchange.
template <int CHUNKS, int RB, int SRC, int THREADS, int EXTRA = 0, bool PLUS = false>
__global__ void __launch_bounds__(THREADS, 1) persistent_kernel(const PersistParams p) {
    constexpr int RBT = RB + EXTRA;                                            // rows per batch
    constexpr int SH = (RB == 32) ? 0 : (RB == 16 ? 1 : (RB == 8 ? 2 : 3));    // log2(32/RB)
    constexpr int WARPS = THREADS / 32;
    static_assert(RB == 4 || RB == 8 || RB == 16 || RB == 32, "RB");
    static_assert(THREADS == 256 || (THREADS == 512 && RB * CHUNKS <= 16), "512 threads leave 128 registers per thread");
    static_assert(RB * CHUNKS <= 32, "register budget");
    static_assert(EXTRA >= 0 && EXTRA <= 2, "EXTRA");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    cg::cluster_group cluster = cg::this_cluster();

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = p.C, ld = p.ld, chunks = ld >> 2;
    const int crank = (int)cluster.block_rank();
    const int worker = blockIdx.x / C;
    const int nmsg = p.n * p.k;

    // ---- shared memory carve-up -------------------------------------------------------------
    float* xs = reinterpret_cast<float*>(smem_raw);                 // [ld]
    float* gs = xs + ld;                                            // [ld]
    float* rterm = gs + ld;                                         // [ld] regulariser term at x
    float* gis = rterm + ld;                                        // [ld] g_i (leader block)
    float* vs = gis + ld;                                           // [ld] v = grad_i - g_i (leader block)
    float* red = vs + ld;                                           // [WARPS][ld]
    float* part = red + WARPS * ld;                              // [C][ld] (used in the leader)
    unsigned long long* msg = reinterpret_cast<unsigned long long*>(part + C * ld);   // [nmsg]
    float* sacc = reinterpret_cast<float*>(msg + ((nmsg + 1) & ~1));                  // [ld] per-coordinate sum of messages
    unsigned char* touched = reinterpret_cast<unsigned char*>(sacc + ld);             // [ld] coordinate received a message
    unsigned char* sel = touched + ld;                                                // [ld] leader: entry is in the Top-k
    unsigned* table = reinterpret_cast<unsigned*>(touched + ((2 * ld + 15) & ~15));   // [n][ld] value bits by (worker, coordinate)
    float* gall = reinterpret_cast<float*>(table);                                    // PLUS: [n][ld] replica of every g_i
    float* gr = gall + (PLUS ? p.n * ld : 0);                                         // PLUS, leader: [ld] grad_i
    unsigned char* selb = reinterpret_cast<unsigned char*>(gr + (PLUS ? ld : 0));     // PLUS, leader: [ld] entry is in Top-k of grad_i
    unsigned char* wflag = selb + (PLUS ? ((ld + 15) & ~15) : 0);                     // PLUS: [n] branch of each worker's message
    float* slice = PLUS ? reinterpret_cast<float*>(wflag + ((p.n + 15) & ~15))
                        : reinterpret_cast<float*>(table + (p.use_table ? p.n * ld : 0));   // SMEM source, 16-byte aligned
    __shared__ int abort_flag;
    __shared__ double dist_red[2][THREADS / 32];
    __shared__ int plus_branch;
    __shared__ __align__(8) unsigned long long part_bar;     // leader: counts the bytes of the partials

    // ---- this block's rows --------------------------------------------------------------------
    const i64 w_r0 = p.row_off[worker], w_r1 = p.row_off[worker + 1];
    const i64 m_i = w_r1 - w_r0;
    const i64 q = (m_i + C - 1) / C;
    const i64 r0 = min(w_r0 + (i64)crank * q, w_r1), r1 = min(r0 + q, w_r1);
    const int rows = (int)(r1 - r0);
    const int nbatch = (rows + RBT - 1) / RBT;

    // The launch must really have put C blocks into each cluster; otherwise nobody would send partials.
    if ((int)cluster.num_blocks() != C) {
        if (tid == 0) record_error(p.status, 7u /* EF21_ERR_UNSUPPORTED */);
        return;
    }
    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&part_bar, 1u);
        fence_mbar_init_cluster();
    }
    for (int j = tid; j < ld; j += THREADS) { xs[j] = p.x[j]; gs[j] = p.g[j]; }
    for (int j = tid; j < ld; j += THREADS) { sacc[j] = 0.f; touched[j] = 0; }
    if (PLUS) {
        for (int e = tid; e < p.n * ld; e += THREADS) gall[e] = p.gi[e];
    } else if (p.use_table) {
        for (int e = tid; e < p.n * ld; e += THREADS) table[e] = PK_NO_ENTRY;
    }
    if (SRC == PK_SRC_SMEM) {
        const float4* src = reinterpret_cast<const float4*>(p.A + r0 * (i64)ld);
        float4* dst = reinterpret_cast<float4*>(slice);
        for (int e = tid; e < rows * chunks; e += THREADS) dst[e] = src[e];
    }

    // The leader block of the cluster keeps g_i in shared memory.
    const bool leader = crank == 0;
    if (leader)
        for (int j = tid; j < ld; j += THREADS) gis[j] = p.gi[(i64)worker * ld + j];

    // REG source: the (single) batch of this warp lives in registers for the whole kernel.
    float4 a[RB][CHUNKS];
    float4 ax[EXTRA > 0 ? EXTRA : 1][CHUNKS];
    float y_reg = 0.f, y_ext[EXTRA > 0 ? EXTRA : 1];
    auto load_row = [&](int row, int cs) {
        const int c = lane + 32 * cs;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < rows && c < chunks) {
            if (SRC == PK_SRC_SMEM) v = reinterpret_cast<const float4*>(slice)[row * chunks + c];
            else v = __ldg(reinterpret_cast<const float4*>(p.A + (r0 + row) * (i64)ld) + c);
        }
        return v;
    };
    auto load_batch = [&](int b) {
        const int rb0 = b * RBT;
#pragma unroll
        for (int e = 0; e < EXTRA; ++e) {
            const int row = rb0 + RB + e;
#pragma unroll
            for (int cs = 0; cs < CHUNKS; ++cs) ax[e][cs] = load_row(row, cs);
            y_ext[e] = row < rows ? __ldg(p.y + r0 + row) : 0.f;
        }
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const int row = rb0 + r;
#pragma unroll
            for (int cs = 0; cs < CHUNKS; ++cs) a[r][cs] = load_row(row, cs);
        }
        const int myrow = rb0 + (lane >> SH);
        y_reg = myrow < rows ? __ldg(p.y + r0 + myrow) : 0.f;
    };
    if (SRC == PK_SRC_REG) load_batch(warp);     // host guarantees nbatch <= WARPS
    if (C > 1) cluster.sync(); else __syncthreads();        // barriers initialised before any remote store
    const unsigned part_bytes = (unsigned)(C - 1) * (unsigned)chunks * 16u;
    const unsigned remote_part = map_to_rank(smem_u32(part), 0u), remote_bar = map_to_rank(smem_u32(&part_bar), 0u);

    const bool rank_select = p.k > 6;      // Top-k by rank counting instead of k arg-max rounds (cheaper from about 7 rounds on)
    unsigned pad_mask = 0u;                // this lane's entries beyond d (chunk layout) can never be selected
#pragma unroll
    for (int cs = 0; cs < CHUNKS; ++cs)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (4 * (lane + 32 * cs) + e >= p.d) pad_mask |= 1u << (cs * 4 + e);
    const unsigned k_magic = (65536u + (unsigned)p.k - 1u) / (unsigned)p.k;     // u / k == (u * k_magic) >> 16 for u < 2048, k <= 32
    bool aborted = false;
    for (int t = 0; t < p.steps; ++t) {
        const unsigned epoch = (p.epoch0 + (unsigned)t + 1u) & 0xffffu;
        unsigned long long* slot = p.slots + (size_t)(epoch & 1u) * nmsg;

        if (!aborted) {
            // 1. x <- x - gamma g on this block's replica (Algorithm 2, first line of the loop)
            for (int j = tid; j < ld; j += THREADS) xs[j] = fmaf(-p.gamma, gs[j], xs[j]);
            if (leader && C > 1 && tid == 0) mbar_arrive_expect_tx(&part_bar, part_bytes);
            __syncthreads();
            if (leader)
                for (int j = tid; j < ld; j += THREADS) rterm[j] = regulariser_grad(p.lambda, xs[j]);

            // 2. partial gradient over this warp's batches
            float4 xr[CHUNKS], acc[CHUNKS];
#pragma unroll
            for (int cs = 0; cs < CHUNKS; ++cs) {
                const int c = lane + 32 * cs;
                xr[cs] = c < chunks ? reinterpret_cast<const float4*>(xs)[c] : make_float4(0.f, 0.f, 0.f, 0.f);
                acc[cs] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            for (int b = warp; b < nbatch; b += WARPS) {
                if (SRC != PK_SRC_REG) load_batch(b);
                float pd[RB];
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    float z = 0.f;
#pragma unroll
                    for (int cs = 0; cs < CHUNKS; ++cs) z = dot4(a[r][cs], xr[cs], z);
                    pd[r] = z;
                }
                const float z = reduce_rows<RB>(pd, lane);
                const float rho = loss_residual(p.objective, y_reg, z);
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const float pr = __shfl_sync(0xffffffffu, rho, r << SH);
#pragma unroll
                    for (int cs = 0; cs < CHUNKS; ++cs) acc[cs] = fma4(pr, a[r][cs], acc[cs]);
                }
#pragma unroll
                for (int e = 0; e < EXTRA; ++e) {
                    float ze = 0.f;
#pragma unroll
                    for (int cs = 0; cs < CHUNKS; ++cs) ze = dot4(ax[e][cs], xr[cs], ze);
#pragma unroll
                    for (int off = 16; off >= 1; off >>= 1) ze += __shfl_xor_sync(0xffffffffu, ze, off);
                    const float pe = loss_residual(p.objective, y_ext[e], ze);      // 0 for a row past the end (y = 0, a = 0)
#pragma unroll
                    for (int cs = 0; cs < CHUNKS; ++cs) acc[cs] = fma4(pe, ax[e][cs], acc[cs]);
                }
            }
#pragma unroll
            for (int cs = 0; cs < CHUNKS; ++cs) {
                const int c = lane + 32 * cs;
                if (c < chunks) reinterpret_cast<float4*>(red + warp * ld)[c] = acc[cs];
            }
            __syncthreads();

            // 3. block partial (warps in ascending order) -> leader's shared memory.  Remote blocks send
            //    16-byte stores that credit the leader's barrier; they do not wait for anything.
            for (int c = tid; c < chunks; c += THREADS) {
                float4 sum = reinterpret_cast<const float4*>(red)[c];
#pragma unroll
                for (int w = 1; w < WARPS; ++w) {
                    const float4 o = reinterpret_cast<const float4*>(red + w * ld)[c];
                    sum.x = __fadd_rn(sum.x, o.x); sum.y = __fadd_rn(sum.y, o.y);
                    sum.z = __fadd_rn(sum.z, o.z); sum.w = __fadd_rn(sum.w, o.w);
                }
                if (leader) reinterpret_cast<float4*>(part)[c] = sum;
                else st_async_f4(remote_part + (unsigned)(crank * ld + 4 * c) * 4u, sum, remote_bar);
            }
            if (leader) {
                __syncthreads();
                if (C > 1) {
                    // bounded: by tries and by elapsed clocks (about two seconds), whichever comes first
                    unsigned spins = 0;
                    const long long wait_t0 = clock64();
                    while (!mbar_try_wait_parity(&part_bar, (unsigned)t & 1u)) {
                        if (++spins > p.spin_limit || clock64() - wait_t0 > 4000000000ll) {
                            record_error(p.status, 5u /* EF21_ERR_TIMEOUT */);
                            abort_flag = 1;
                            break;
                        }
                    }
                    __syncthreads();
                    if (abort_flag) aborted = true;
                }
            }
        }

        if (!aborted) {
            // 4. leader: gradient, difference, Top-k, state update, publish
            if (leader) {
                const float mf = (float)m_i;
                for (int j = tid; j < ld; j += THREADS) {
                    float sum = part[j];
                    for (int cc = 1; cc < C; ++cc) sum = __fadd_rn(sum, part[cc * ld + j]);
                    const float grad = __fadd_rn(m_i > 0 ? __fdiv_rn(sum, mf) : 0.f, rterm[j]);
                    vs[j] = __fsub_rn(grad, gis[j]);
                    if (PLUS) gr[j] = grad;
                }
                __syncthreads();
                if (PLUS) {
                    // ranks of every coordinate in grad_i - g_i and in grad_i ((|.| descending, index ascending);
                    // `split` adjacent lanes share a coordinate and count a contiguous part of the entries each)
                    const int split = (ld * 4 <= THREADS) ? 4 : ((ld * 2 <= THREADS) ? 2 : 1);
                    const int part_len = (p.d + split - 1) / split;
                    for (int j0 = 0; j0 < ld; j0 += THREADS / split) {
                        const int j = j0 + tid / split, q = tid % split;
                        int rank_m = 0, rank_b = 0;
                        if (j < p.d) {
                            const unsigned km = mag_key(vs[j]), kb = mag_key(gr[j]);
                            const int i1 = min((q + 1) * part_len, p.d);
#pragma unroll 2
                            for (int i = q * part_len; i < i1; ++i) {
                                const unsigned kim = mag_key(vs[i]), kib = mag_key(gr[i]);
                                rank_m += (kim > km || (kim == km && i < j)) ? 1 : 0;
                                rank_b += (kib > kb || (kib == kb && i < j)) ? 1 : 0;
                            }
                        }
                        if (split >= 2) { rank_m += __shfl_xor_sync(0xffffffffu, rank_m, 1); rank_b += __shfl_xor_sync(0xffffffffu, rank_b, 1); }
                        if (split >= 4) { rank_m += __shfl_xor_sync(0xffffffffu, rank_m, 2); rank_b += __shfl_xor_sync(0xffffffffu, rank_b, 2); }
                        if (q == 0 && j < ld) {
                            sel[j] = (j < p.d && rank_m < p.k) ? 1 : 0;
                            selb[j] = (j < p.d && rank_b < p.k) ? 1 : 0;
                        }
                    }
                    __syncthreads();
                    // distortions M_i = ||g_i + C(grad_i - g_i) - grad_i||^2 and B_i = ||C(grad_i) - grad_i||^2 as fp64
                    // sums of the fp32 vectors, both over the coordinates in the same order
                    double dm = 0.0, db = 0.0;
                    for (int j = tid; j < p.d; j += THREADS) {
                        const float g0 = gis[j], gj = gr[j];
                        const float mj = sel[j] ? __fadd_rn(g0, vs[j]) : g0;
                        const double em = (double)mj - (double)gj;
                        dm += em * em;
                        if (!selb[j]) db += (double)gj * (double)gj;
                    }
                    dm = warp_sum(dm); db = warp_sum(db);
                    if (lane == 0) { dist_red[0][warp] = dm; dist_red[1][warp] = db; }
                    __syncthreads();
                    if (tid == 0) {
                        double M = 0.0, Bd = 0.0;
                        for (int w = 0; w < WARPS; ++w) { M += dist_red[0][w]; Bd += dist_red[1][w]; }
                        plus_branch = M <= Bd ? 0 : 1;
                    }
                    __syncthreads();
                    const int branch = plus_branch;
                    if (warp == 0) {
                        // the message: the compressed vector that was used, ascending index order from the ballot
                        // ranks; bit 15 of the index field carries the branch
                        const unsigned char* chosen_set = branch ? selb : sel;
                        const float* values = branch ? gr : vs;
                        int base = 0;
                        for (int j0 = 0; j0 < ld; j0 += 32) {
                            const int j = j0 + lane;
                            const bool chosen = j < ld && chosen_set[j] != 0;
                            const unsigned bal = __ballot_sync(0xffffffffu, chosen);
                            if (chosen) {
                                const int pos = base + __popc(bal & ((1u << lane) - 1u));
                                const float val = values[j];
                                const unsigned long long word = ((unsigned long long)epoch << 48) |
                                                                ((unsigned long long)((unsigned)j | ((unsigned)branch << 15)) << 32) |
                                                                (unsigned long long)__float_as_uint(val);
                                st_relaxed_u64(slot + worker * p.k + pos, word);
                                if (t == p.steps - 1) { p.msg_idx[worker * p.k + pos] = j; p.msg_val[worker * p.k + pos] = val; }
                            }
                            base += __popc(bal);
                        }
                        if (lane == 0 && t == p.steps - 1) p.plus_choice[worker] = branch;
                    }
                    // g_i <- the chosen vector (nobody reads gis again before the next iteration's barriers)
                    for (int j = tid; j < ld; j += THREADS)
                        gis[j] = branch ? (selb[j] ? gr[j] : 0.f) : (sel[j] ? __fadd_rn(gis[j], vs[j]) : gis[j]);
                }
                if (!PLUS && rank_select) {
                    // larger k: every coordinate counts the entries that precede it in (|v| descending, index
                    // ascending) order; the k entries of rank < k are the message.  `split` adjacent lanes share a
                    // coordinate, each counts a contiguous part of the entries, a butterfly adds the parts up.
                    const int split = (ld * 4 <= THREADS) ? 4 : ((ld * 2 <= THREADS) ? 2 : 1);
                    const int part_len = (p.d + split - 1) / split;
                    for (int j0 = 0; j0 < ld; j0 += THREADS / split) {       // uniform trip count: all lanes reach the shuffles
                        const int j = j0 + tid / split, q = tid % split;
                        int rank = 0;
                        if (j < p.d) {
                            const unsigned kj = mag_key(vs[j]);
                            const int i1 = min((q + 1) * part_len, p.d);
#pragma unroll 4
                            for (int i = q * part_len; i < i1; ++i) {
                                const unsigned ki = mag_key(vs[i]);
                                rank += (ki > kj || (ki == kj && i < j)) ? 1 : 0;
                            }
                        }
                        if (split >= 2) rank += __shfl_xor_sync(0xffffffffu, rank, 1);
                        if (split >= 4) rank += __shfl_xor_sync(0xffffffffu, rank, 2);
                        if (q == 0 && j < ld) sel[j] = (j < p.d && rank < p.k) ? 1 : 0;
                    }
                    __syncthreads();
                }
            }
            if (!PLUS && leader && warp == 0 && rank_select) {
                // ascending index order falls out of the ballot ranks
                int base = 0;
                for (int j0 = 0; j0 < ld; j0 += 32) {
                    const int j = j0 + lane;
                    const bool chosen = j < ld && sel[j] != 0;
                    const unsigned bal = __ballot_sync(0xffffffffu, chosen);
                    if (chosen) {
                        const int pos = base + __popc(bal & ((1u << lane) - 1u));
                        const float val = vs[j];
                        gis[j] = __fadd_rn(gis[j], val);
                        const unsigned long long word = ((unsigned long long)epoch << 48) | ((unsigned long long)(unsigned)j << 32) |
                                                        (unsigned long long)__float_as_uint(val);
                        st_relaxed_u64(slot + worker * p.k + pos, word);
                        if (t == p.steps - 1) { p.msg_idx[worker * p.k + pos] = j; p.msg_val[worker * p.k + pos] = val; }
                    }
                    base += __popc(bal);
                }
            }
            if (!PLUS && leader && warp == 0 && !rank_select) {
                float4 v[CHUNKS];
                unsigned taken = pad_mask;            // bit (cs*4+comp) set: not selectable
#pragma unroll
                for (int cs = 0; cs < CHUNKS; ++cs) {
                    const int c = lane + 32 * cs;
                    v[cs] = c < chunks ? reinterpret_cast<const float4*>(vs)[c] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                int my_idx = 0; float my_val = 0.f;          // lane t keeps the t-th pick
                for (int t2 = 0; t2 < p.k; ++t2) {
                    // arg-max of (|v| bits, lower index first): warp maximum of the key, then warp minimum of
                    // the index among the entries that hold it
                    int lk = -1;
#pragma unroll
                    for (int cs = 0; cs < CHUNKS; ++cs)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const bool ok = !((taken >> (cs * 4 + e)) & 1u);
                            const int key = (int)mag_key(comp_of(v[cs], e));
                            lk = (ok && key > lk) ? key : lk;
                        }
                    const int wk = __reduce_max_sync(0xffffffffu, lk);
                    unsigned li = 0xffffffffu;
#pragma unroll
                    for (int cs = 0; cs < CHUNKS; ++cs)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const bool ok = !((taken >> (cs * 4 + e)) & 1u);
                            const unsigned idx = (unsigned)(4 * (lane + 32 * cs) + e);
                            if (ok && (int)mag_key(comp_of(v[cs], e)) == wk) li = min(li, idx);
                        }
                    const unsigned widx = __reduce_min_sync(0xffffffffu, li);
                    const int wchunk = (int)(widx >> 2), wlane = wchunk & 31, wcs = wchunk >> 5, we = (int)(widx & 3u);
                    float wval = 0.f;
#pragma unroll
                    for (int cs = 0; cs < CHUNKS; ++cs)
                        if (cs == wcs) wval = comp_of(v[cs], we);
                    wval = __shfl_sync(0xffffffffu, wval, wlane);
                    if (lane == wlane) {
                        taken |= 1u << (wcs * 4 + we);
                        gis[widx] = __fadd_rn(gis[widx], wval);
                    }
                    if (lane == t2) { my_idx = (int)widx; my_val = wval; }
                }
                // ascending index order inside the message
                int rank = 0;
                for (int u = 0; u < p.k && p.k > 1; ++u) {
                    const int oi = __shfl_sync(0xffffffffu, my_idx, u);
                    rank += (lane < p.k && oi < my_idx) ? 1 : 0;
                }
                if (lane < p.k) {
                    const unsigned long long word = ((unsigned long long)epoch << 48) |
                                                    ((unsigned long long)(unsigned)my_idx << 32) |
                                                    (unsigned long long)__float_as_uint(my_val);
                    st_relaxed_u64(slot + worker * p.k + rank, word);
                    if (t == p.steps - 1) {
                        p.msg_idx[worker * p.k + rank] = my_idx;
                        p.msg_val[worker * p.k + rank] = my_val;
                    }
                }
            }

            // 5. gather all n*k message words of this epoch (bounded spin)
            auto poll_word = [&](int u, unsigned long long& w) {
                unsigned spins = 0;
                while (true) {
                    w = ld_relaxed_u64(slot + u);
                    if ((unsigned)(w >> 48) == epoch) return true;
                    ++spins;
                    if ((spins & 1023u) == 0u && ld_relaxed_u32(p.status) != 0u) { abort_flag = 1; return false; }
                    if (spins > p.spin_limit) { record_error(p.status, (unsigned)5 /* EF21_ERR_TIMEOUT */); abort_flag = 1; return false; }
                }
            };
            for (int u = tid; u < nmsg; u += THREADS) {
                unsigned long long w;
                const bool got = poll_word(u, w);
                if (!PLUS && p.use_table) {
                    const unsigned idx = (unsigned)(w >> 32) & 0xffffu;
                    if (got && idx < (unsigned)ld) table[(int)(((unsigned)u * k_magic) >> 16) * ld + (int)idx] = (unsigned)w;
                } else {
                    msg[u] = w;
                }
            }
            __syncthreads();
            if (abort_flag) aborted = true;
        }
        if (PLUS && !aborted) {
            // every block applies the n messages to its replicas of the g_i: a worker that took the plain branch
            // restarts from zero, the others add their entries; then g = (1/n) sum_i g_i, ascending i
            for (int i = tid; i < p.n; i += THREADS) wflag[i] = (unsigned char)((msg[i * p.k] >> 47) & 1ull);
            __syncthreads();
            for (int i = 0; i < p.n; ++i)
                if (wflag[i])
                    for (int j = tid; j < ld; j += THREADS) gall[i * ld + j] = 0.f;
            __syncthreads();
            for (int u = tid; u < nmsg; u += THREADS) {
                const unsigned long long w = msg[u];
                const int i = (int)(((unsigned)u * k_magic) >> 16);
                const unsigned idx = (unsigned)(w >> 32) & 0x7fffu;
                const float val = __uint_as_float((unsigned)w);
                if (idx < (unsigned)ld) gall[i * ld + (int)idx] = wflag[i] ? val : __fadd_rn(gall[i * ld + (int)idx], val);
            }
            __syncthreads();
            for (int j = tid; j < p.d; j += THREADS) {
                float sum = 0.f;
#pragma unroll 4
                for (int i = 0; i < p.n; ++i) sum = __fadd_rn(sum, gall[i * ld + j]);
                gs[j] = __fmul_rn(sum, p.inv_n);
            }
            continue;
        }
        if (!aborted && p.use_table) {
            // g_j += (1/n) * sum over workers (ascending) of the values sent for coordinate j: row i of the
            // table holds worker i's message scattered by coordinate; a cell is emptied by the thread that
            // read it (the next messages are written several barriers later)
            for (int j = tid; j < p.d; j += THREADS) {
                float s = 0.f; bool hit = false;
#pragma unroll 4
                for (int i = 0; i < p.n; ++i) {
                    const unsigned bits = table[i * ld + j];
                    const bool present = bits != PK_NO_ENTRY;
                    const float sum = __fadd_rn(s, __uint_as_float(bits));
                    s = present ? sum : s;
                    hit = hit || present;
                    table[i * ld + j] = PK_NO_ENTRY;
                }
                if (hit) gs[j] = __fadd_rn(gs[j], __fmul_rn(s, p.inv_n));
            }
            continue;
        }
        if (!aborted && nmsg > PK_SCAN_MAX_MSGS) {
            // many messages: warp 0 folds them into per-coordinate running sums, one worker at a time (a
            // worker's k <= 32 coordinates are distinct), then every coordinate applies its sum
            if (warp == 0) {
                const int kk = p.k;
                for (int i = 0; i < p.n; ++i) {
                    if (lane < kk) {
                        const unsigned long long w = msg[i * kk + lane];
                        const unsigned idx = (unsigned)(w >> 32) & 0xffffu;
                        if (idx < (unsigned)ld) { sacc[idx] = __fadd_rn(sacc[idx], __uint_as_float((unsigned)w)); touched[idx] = 1; }
                    }
                    __syncwarp();
                }
            }
            __syncthreads();
            for (int j = tid; j < p.d; j += THREADS)
                if (touched[j]) {
                    gs[j] = __fadd_rn(gs[j], __fmul_rn(sacc[j], p.inv_n));
                    sacc[j] = 0.f; touched[j] = 0;
                }
        } else if (!aborted) {
            // g_j += (1/n) * sum over workers (ascending) of the values sent for coordinate j
            for (int j = tid; j < p.d; j += THREADS) {
                float s = 0.f; bool touched = false;
#pragma unroll 4
                for (int u = 0; u < nmsg; ++u) {
                    const unsigned long long w = msg[u];
                    if ((int)((w >> 32) & 0xffffu) == j) { s = __fadd_rn(s, __uint_as_float((unsigned)w)); touched = true; }
                }
                if (touched) gs[j] = __fadd_rn(gs[j], __fmul_rn(s, p.inv_n));
            }
            // the next iteration's x update reads gs[j] in the same thread: no barrier needed here
        }
    }

    __syncthreads();
    if (C > 1) {
        if (aborted) __nanosleep(20000);         // let remote stores that were in flight land
        cluster.sync();
    }
    if (blockIdx.x == 0)
        for (int j = tid; j < ld; j += THREADS) { p.x[j] = xs[j]; p.g[j] = gs[j]; }
    if (leader)
        for (int j = tid; j < ld; j += THREADS) p.gi[(i64)worker * ld + j] = gis[j];
}

// One-block self-check of the bounded wait: spins on a word that nobody writes and must come back
// with EF21_ERR_TIMEOUT in the status word instead of hanging.
__global__ void bounded_wait_selftest_kernel(const unsigned long long* never_written, unsigned* status,
                                             unsigned spin_limit) {
    unsigned spins = 0;
    while (true) {
        const unsigned long long w = ld_relaxed_u64(never_written);
        if ((unsigned)(w >> 48) == 0xffffu) break;
        if (++spins > spin_limit) { record_error(status, 5u); break; }
    }
}

}  // namespace ef21
