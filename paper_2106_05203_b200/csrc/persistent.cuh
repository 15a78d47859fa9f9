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
// Two bodies implement these steps.  persistent_body.inc takes every step with the whole block between block
// barriers, as listed above; persistent_roles.inc lets the last warp of a block serve it (steps 1, 3, 4, 5 in one
// warp, four coordinates per lane) while the other warps only sweep rows (step 2) between two named barriers.
// Each body is compiled once per method, one translation unit each (persistent_*.cu): Algorithm 2 as described
// above, EF21+ (Algorithm 3: a second selection on grad_i, the two distortions, per-block replicas of all g_i and a
// dense mean; whole-block body only), the original EF (Algorithm 4: the leader compresses e_i + gamma grad_i, the
// messages move x directly) and the exchange skeleton (a measuring aid).  This header holds what they share.
//
// All summation orders are fixed by the launch shape, so two runs give identical bits.  A wait
// that exceeds its spin limit records EF21_ERR_TIMEOUT in the status word; from then on every
// block skips work but keeps arriving at the cluster barriers, so the kernel always terminates.
#pragma once
#include <cooperative_groups.h>
#include <cuda/std/type_traits>

#include "common.cuh"

namespace ef21 {
namespace cg = cooperative_groups;

constexpr int PK_MAX_THREADS = 512;     // the kernel is instantiated for 256 and 512 threads per block
constexpr int PK_MAX_K = 32;
constexpr int PK_MAX_MSGS = 2048;       // n*k words staged in shared memory
constexpr int PK_SCAN_MAX_MSGS = 128;   // up to this many messages every coordinate thread scans them all
constexpr int PK_TABLE_MAX_BYTES = 64 * 1024;   // largest [n][ld] message table kept in shared memory
constexpr unsigned PK_NO_ENTRY = 0xffffffffu;   // table cell without a message (a NaN pattern no finite value has)
// where a block's rows come from: registers / shared memory (loaded once), global memory (every iteration), or global
// memory through a per-iteration list of sampled row numbers (stochastic variant, Algorithm 5)
enum { PK_SRC_REG = 0, PK_SRC_SMEM = 1, PK_SRC_GMEM = 2, PK_SRC_SAMPLED = 3 };

struct PersistParams {
    const float* A;            // [N][ld], padded, read-only
    const float* y;            // [N]
    const i64* row_off;        // [n+1]
    float* x;                  // [ld]
    float* g;                  // [ld]
    float* gi;                 // [n][ld]
    int* msg_idx;              // [n][k] last messages (written at the final iteration)
    float* msg_val;
    unsigned long long* slots; // [2][n*k]
    unsigned* status;
    int n, d, ld, k, C, steps;
    int objective;             // 0 logistic loss, 1 least squares
    int slice_rows;            // capacity (rows) of the shared-memory slice (SMEM source)
    int use_table;             // 1: received messages are scattered into a [n][ld] table in shared memory
    float gamma, lambda, inv_n;
    unsigned spin_limit;
    unsigned epoch0;           // epoch of the handle's last iteration so far (0: none yet); epochs run 1..65535 and wrap to 1
    unsigned par0;             // which half of the slot array that iteration used
    int* plus_choice;          // [n] EF21+: branch taken at the final iteration (0 Markov compressor, 1 plain)
    const int* batch;          // stochastic variant (Algorithm 5): [steps][n][tau] row numbers inside each shard; null: all rows
    int tau;                   // rows per worker and iteration of the stochastic variant
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

// Named barriers of a block (id 1..15; 0 belongs to __syncthreads): `count` threads take part, some only announce
// their arrival (producers), the others wait for everybody (consumers).  Shared-memory writes made before the
// arrival are visible to the threads the barrier releases.
__device__ __forceinline__ void named_bar_sync(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int count) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Keeps the compiler from moving loads and stores from one phase of an iteration into another.  The service warp of
// the persistent kernel runs alone, so the order of its instructions is its timing: with the phases kept apart the
// iteration was 8-18 % shorter than with the order the compiler chose on its own (measured, both orders correct).
__device__ __forceinline__ void phase_fence() { asm volatile("" ::: "memory"); }

__device__ __forceinline__ float comp_of(const float4& v, int c) {
    return c == 0 ? v.x : (c == 1 ? v.y : (c == 2 ? v.z : v.w));
}

// The epoch after e.  A slot word is at most two iterations old when it is polled, so a wrapped epoch never meets
// its own value; 0 marks a word that no iteration has written (the array is cleared once, at creation).
__device__ __forceinline__ unsigned next_epoch(unsigned e) { return e >= 65535u ? 1u : e + 1u; }

// Top-k of up to 128 entries held four per lane (lane L owns entries 4L .. 4L+3 in v4), by one warp, for vectors of at
// most 128 coordinates.  Every lane first orders its own four entries by (|.| bits descending, index ascending); a round
// then is the warp maximum of the lanes' best remaining keys, the warp minimum of the indices that hold it (the lower
// index wins a tie), and the owner dropping that entry -- two redux and a handful of predicated moves, nothing is
// recomputed.  pad_bits: bit e set = entry 4L+e lies beyond d and is never taken.  Returns the lane's 4-bit mask of
// selected entries; position receives the number of selected entries in lower lanes, so that a lane can emit its picks
// in ascending index order at position, position + 1, ...
__device__ __forceinline__ unsigned warp_topk_four_per_lane(const float4& v4, unsigned pad_bits, int k, int lane, int& position) {
    // composite (key, 3 - e): larger is better; -1 marks an entry that cannot be taken
    long long c[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const long long key = ((pad_bits >> e) & 1u) ? -1ll : (long long)mag_key(comp_of(v4, e));
        c[e] = key < 0 ? -1ll : ((key << 2) | (long long)(3 - e));
    }
    auto order = [&](int a, int b) { const long long hi = max(c[a], c[b]), lo = min(c[a], c[b]); c[a] = hi; c[b] = lo; };
    order(0, 1); order(2, 3); order(0, 2); order(1, 3); order(1, 2);
    int k0 = (int)(c[0] >> 2), k1 = (int)(c[1] >> 2), k2 = (int)(c[2] >> 2), k3 = (int)(c[3] >> 2);       // -1 stays -1
    int e0 = 3 - (int)(c[0] & 3), e1 = 3 - (int)(c[1] & 3), e2 = 3 - (int)(c[2] & 3), e3 = 3 - (int)(c[3] & 3);
    unsigned mask = 0u;
    for (int round = 0; round < k; ++round) {
        const int wk = __reduce_max_sync(0xffffffffu, k0);
        const unsigned mine = (k0 == wk && k0 >= 0) ? (unsigned)(4 * lane + e0) : 0xffffffffu;
        const unsigned widx = __reduce_min_sync(0xffffffffu, mine);
        if (mine == widx && mine != 0xffffffffu) {
            mask |= 1u << e0;
            k0 = k1; e0 = e1; k1 = k2; e1 = e2; k2 = k3; e2 = e3; k3 = -1;
        }
    }
    const unsigned cnt = (unsigned)__popc(mask), lt = (1u << lane) - 1u;
    const unsigned b0 = __ballot_sync(0xffffffffu, cnt & 1u), b1 = __ballot_sync(0xffffffffu, cnt & 2u), b2 = __ballot_sync(0xffffffffu, cnt & 4u);
    position = __popc(b0 & lt) + 2 * __popc(b1 & lt) + 4 * __popc(b2 & lt);
    return mask;
}

typedef void (*PersistKernel)(const PersistParams);

// One lookup per method (each in a translation unit of its own, so that they compile side by side):
// the kernel instantiated for (chunk slots per lane, rows per warp batch, row source, threads per block,
// extra rows per batch), or nullptr if that shape is not instantiated.
// Two bodies exist.  "roles" (persistent_roles.inc): the last warp of a block serves it, the others only sweep rows;
// Top-k by warp arg-max rounds -- for k <= PK_ROLES_MAX_K.  "wide" (persistent_body.inc): every step is taken by the
// whole block between block barriers, Top-k by rank counting over all threads for larger k -- any k <= PK_MAX_K, and
// the only body of Algorithm 3.
constexpr int PK_ROLES_MAX_K = 8;
PersistKernel pk_lookup_ef21(int chunks, int rb, int src, int threads, int extra);          // Algorithm 2, roles
PersistKernel pk_lookup_ef(int chunks, int rb, int src, int threads, int extra);            // Algorithm 4, roles
PersistKernel pk_lookup_floor(int chunks, int rb, int src, int threads, int extra);         // exchange skeleton, roles
PersistKernel pk_lookup_wide_ef21(int chunks, int rb, int src, int threads, int extra);     // Algorithm 2, wide
PersistKernel pk_lookup_plus(int chunks, int rb, int src, int threads, int extra);          // Algorithm 3, wide
PersistKernel pk_lookup_wide_ef(int chunks, int rb, int src, int threads, int extra);       // Algorithm 4, wide
PersistKernel pk_lookup_wide_floor(int chunks, int rb, int src, int threads, int extra);    // exchange skeleton, wide

}  // namespace ef21
