// libef21: C-ABI entry points (see include/ef21.h) and the host-side orchestration.
#include "../../include/ef21.h"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "apply.cuh"
#include "common.cuh"
#include "ef.cuh"
#include "grad.cuh"
#include "persistent.cuh"
#include "wait_selftest.cuh"
#include "plus.cuh"
#include "stress.cuh"
#include "topk.cuh"

using namespace ef21;

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }
inline i64 ceil_div(i64 a, i64 b) { return (a + b - 1) / b; }

// ---------------------------------------------------------------------------------------------
// Workspace layouts
// ---------------------------------------------------------------------------------------------

struct TopkLayout {
    size_t state, hist, chunks, total;
    int nchunks;
    // one-pass path for long vectors (stress.cuh); fast == false: sections absent
    bool fast;
    int nreg;
    size_t thr, flags, done, slow_count, region_cnt, cand;
};

bool fast_topk_eligible(i64 d, i64 k) { return d >= ST_MIN_D && k <= ST_MAX_K; }

// The three sections every Top-k call needs (selection state, histogram, per-chunk counts); the
// one-pass sections are absent.
TopkLayout topk_layout_general(i64 batch, i64 d) {
    TopkLayout L{};
    L.nchunks = (int)ceil_div(d, TK_CHUNK);
    size_t o = 0;
    L.state = o; o += align_up((size_t)batch * sizeof(TkState));
    L.hist = o; o += align_up((size_t)batch * TK_BINS * sizeof(unsigned));
    L.chunks = o; o += align_up((size_t)batch * (size_t)L.nchunks * sizeof(uint2));
    L.fast = false;
    L.nreg = (int)ceil_div(d, ST_SUB);
    L.total = o;
    return L;
}

TopkLayout topk_layout(i64 batch, i64 d, i64 k) {
    TopkLayout L = topk_layout_general(batch, d);
    size_t o = L.total;
    L.fast = fast_topk_eligible(d, k);
    if (L.fast) {
        L.thr = o; o += align_up((size_t)batch * 4);
        L.flags = o; o += align_up((size_t)batch * 4);
        L.done = o; o += align_up((size_t)batch * 4);
        L.slow_count = o; o += align_up(4);
        L.region_cnt = o; o += align_up((size_t)batch * L.nreg * 4);
        L.cand = o; o += align_up((size_t)batch * L.nreg * ST_REGION_CAP * sizeof(int4));
    }
    L.total = o;
    return L;
}

typedef void (*GradTileKernel)(const float*, const float*, const float*, const RowTile*, int, int, float*, double*,
                               const int*, int, const i64*, unsigned*);

// The one-read gradient kernel for rows of up to 1,024 columns (chunk slots = float4 per lane and row); wider
// rows use the two-sweep kernel.
GradTileKernel grad_stream_lookup(i64 ld) {
    const i64 slots = (ld / 4 + 31) / 32;
    if (slots <= 1) return grad_stream_kernel<1, 16>;
    if (slots == 2) return grad_stream_kernel<2, 8>;
    if (slots == 3) return grad_stream_kernel<3, 4>;
    if (slots == 4) return grad_stream_kernel<4, 4>;
    if (slots <= 6) return grad_stream_kernel<6, 2>;
    if (slots <= 8) return grad_stream_kernel<8, 2>;
    return nullptr;
}

int grad_tile_rows(i64 N, i64 ld) {
    // two-sweep kernel: a tile's rows should stay in L1 for the second sweep; one-read kernel: any size
    i64 cap = grad_stream_lookup(ld) ? GRAD_TILE_MAX_ROWS : 65536 / (ld * 4);
    if (cap < 1) cap = 1;
    if (cap > GRAD_TILE_MAX_ROWS) cap = GRAD_TILE_MAX_ROWS;
    i64 want = ceil_div(N, 4 * 148);
    if (want < 8) want = 8;
    return (int)(want < cap ? want : cap);
}

struct Layout {
    i64 ld;            // padded vector pitch (floats), multiple of 4
    int agg_tiles;     // tiles of AGG_TILE coordinates
    int tile_rows;     // rows per gradient tile
    i64 max_tiles;     // capacity of the gradient tile table
    size_t status, x, g, gi, msg_idx, msg_val, topk, agg_off, eval_out, slots;
    size_t msg2_idx, msg2_val, plus_old, plus_choice, plus_bitmap;    // EF21+ (Algorithm 3)
    size_t A, y, row_off, tile_begin, tiles, partial, loss_partial, grad, mb_tile_begin, mb_tiles;
    size_t total;
    TopkLayout tk;
};

Layout make_layout(i64 n, i64 d, i64 k, i64 N) {
    Layout L;
    L.ld = (d + 3) / 4 * 4;
    L.agg_tiles = (int)ceil_div(d, AGG_TILE);
    L.tk = topk_layout(n, d, k);
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o += align_up(bytes); return at; };
    L.status = take(256);
    L.x = take((size_t)L.ld * 4);
    L.g = take((size_t)L.ld * 4);
    L.gi = take((size_t)n * L.ld * 4);
    L.msg_idx = take((size_t)n * k * 4);
    L.msg_val = take((size_t)n * k * 4);
    L.topk = take(L.tk.total);
    L.agg_off = take((size_t)n * (L.agg_tiles + 1) * 4);
    L.eval_out = take(256);
    L.slots = take((size_t)2 * n * k * 8);
    L.msg2_idx = take((size_t)n * k * 4);
    L.msg2_val = take((size_t)n * k * 4);
    L.plus_old = take((size_t)n * k * 4);
    L.plus_choice = take((size_t)n * 4);
    L.plus_bitmap = take((size_t)n * ((d + 31) / 32) * 4);
    L.tile_rows = 0; L.max_tiles = 0;
    L.A = L.y = L.row_off = L.tile_begin = L.tiles = L.partial = L.loss_partial = L.grad = L.mb_tile_begin = L.mb_tiles = 0;
    if (N > 0) {
        L.tile_rows = grad_tile_rows(N, L.ld);
        L.max_tiles = N / L.tile_rows + n;
        L.A = take((size_t)N * L.ld * 4);
        L.y = take((size_t)N * 4);
        L.row_off = take((size_t)(n + 1) * 8);
        L.tile_begin = take((size_t)(n + 1) * 4);
        L.tiles = take((size_t)L.max_tiles * sizeof(RowTile));
        L.partial = take((size_t)L.max_tiles * L.ld * 4);
        L.loss_partial = take((size_t)L.max_tiles * 8);
        L.grad = take((size_t)n * L.ld * 4);
        L.mb_tile_begin = take((size_t)(n + 1) * 4);
        L.mb_tiles = take((size_t)L.max_tiles * sizeof(RowTile));
    }
    L.total = o;
    return L;
}

bool valid_shape(i64 n, i64 d, i64 k, i64 N) {
    return n >= 1 && d >= 1 && k >= 1 && k <= d && d < ((i64)1 << 31) && N >= 0 && n <= 65535;
}

}  // namespace

// Launch plan of the persistent path (made by plan_persistent, kept in the handle until something it depends on changes).
struct PersistPlan {
    bool ok;
    bool roles;         // persistent_roles.inc (the last warp serves the block) instead of whole-block steps
    int C, rb, src, chunks, threads, extra;
    size_t smem;
    PersistKernel kernel;
};

struct ef21_ctx {
    int n; i64 d; int k; float gamma, lambda; i64 N;
    cudaStream_t stream;
    int device;         // the device that was current at ef21_create
    char* ws;
    Layout L;
    bool shards_loaded, inited;
    int num_tiles;
    int path, last_path;
    bool agg_off_ready;                 // the last selection already wrote the aggregation's tile offsets
    bool agg_off_static;                // one tile only: the offsets are (0, k) whatever the messages; written once
    int pk_cluster, pk_rb, pk_src, pk_threads;      // forced persistent-kernel shape (0 / -1 = automatic)
    int pk_used_cluster, pk_used_rb, pk_used_src, pk_used_threads;
    PersistPlan plan; bool plan_valid;  // cached plan of ef21_step's persistent launch
    PersistPlan mb_plan; bool mb_plan_valid; int mb_plan_tau;      // the same for the stochastic variant with mb_plan_tau rows
    unsigned pk_epoch, pk_par;          // epoch and slot half of the last persistent iteration (see PersistParams)
    int pk_body, pk_used_body;          // persistent kernel body: 0 automatic, 1 compute warps + service warp, 2 whole-block steps
    unsigned spin_limit;
    bool force_general_topk;
    int variant;                        // EF21_VARIANT_*
    int objective;                      // EF21_OBJECTIVE_*
    cudaStream_t aux_stream;            // created on first use: overlaps the next threshold estimate
    cudaEvent_t ev_fork, ev_join;
    cudaStream_t cap_stream;            // library-owned stream on which the iteration graph is captured
    cudaGraphExec_t iter_graph;         // one launch-path iteration of ef21_step, captured on first use
    int iter_graph_key;                 // what it was captured for (variant, objective)
    i64 iter_graph_launches;            // kernel launches inside it
    bool iter_graph_off;                // capture failed once: keep to plain launches
    i64 launches;
    std::vector<i64> row_off;
    std::vector<RowTile> tiles;
    std::vector<int> tile_begin;
    std::vector<RowTile> mb_tiles;      // tile table of the minibatch lists, rebuilt when tau changes
    std::vector<int> mb_tile_begin;
    int mb_tau;

    template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
    float* x() const { return at<float>(L.x); }
    float* g() const { return at<float>(L.g); }
    float* gi() const { return at<float>(L.gi); }
    int* msg_idx() const { return at<int>(L.msg_idx); }
    float* msg_val() const { return at<float>(L.msg_val); }
    unsigned* status() const { return at<unsigned>(L.status); }
};

#define CU(call)                                         \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) return EF21_ERR_CUDA;    \
    } while (0)
#define EF(call)                                         \
    do {                                                 \
        ef21_status s__ = (call);                        \
        if (s__ != EF21_OK) return s__;                  \
    } while (0)

namespace {

struct TopkBuffers {
    TkState* state; unsigned* hist; uint2* chunks; int nchunks;
    bool fast; int nreg;
    unsigned* thr; unsigned* flags; unsigned* done; unsigned* slow_count; int* region_cnt; int4* cand;
};

TopkBuffers topk_buffers(char* base, const TopkLayout& L) {
    TopkBuffers B;
    B.state = reinterpret_cast<TkState*>(base + L.state);
    B.hist = reinterpret_cast<unsigned*>(base + L.hist);
    B.chunks = reinterpret_cast<uint2*>(base + L.chunks);
    B.nchunks = L.nchunks;
    B.fast = L.fast; B.nreg = L.nreg;
    B.thr = reinterpret_cast<unsigned*>(base + L.thr);
    B.flags = reinterpret_cast<unsigned*>(base + L.flags);
    B.done = reinterpret_cast<unsigned*>(base + L.done);
    B.slow_count = reinterpret_cast<unsigned*>(base + L.slow_count);
    B.region_cnt = reinterpret_cast<int*>(base + L.region_cnt);
    B.cand = reinterpret_cast<int4*>(base + L.cand);
    return B;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Threshold estimate of the one-pass Top-k (first of its three kernels).
ef21_status enqueue_topk_fast_sample(cudaStream_t st, const float* a, i64 pitch_a, const float* b, i64 pitch_b,
                                     int batch, i64 d, int k, const TopkBuffers& B, i64* launches) {
    const i64 target = std::max<i64>(2 * (i64)k, (i64)k + 2048);
    i64 rank = ceil_div(target * (i64)(ST_SAMPLE_BLOCKS * ST_SAMPLE_LEN), d);
    rank = std::min<i64>(std::max<i64>(rank, 32), ST_SAMPLE_BLOCKS * ST_SAMPLE_LEN / 2);
    st_sample_kernel<<<batch, ST_THREADS, 0, st>>>(a, pitch_a, b, pitch_b, d, (unsigned)rank, B.thr, B.flags);
    if (launches) *launches += 1;
    CU(cudaGetLastError());
    return EF21_OK;
}

// Exact Top-k of v = a - b for long vectors in one pass over a and b (see stress.cuh).  If gi_rows
// is given, g_i += c_i is applied by the same kernel that writes the messages.
ef21_status enqueue_topk_fast(cudaStream_t st, const float* a, i64 pitch_a, const float* b, i64 pitch_b,
                              int batch, i64 d, int k, int* idx_out, float* val_out, float* gi_rows, i64 ld,
                              const TopkBuffers& B, i64* launches, unsigned* status, bool sampled = false,
                              int* tile_off = nullptr, int ntiles = 0) {
    const size_t finish_smem = (size_t)ST_CAND_CAP * 12 + 2048 * 4;
    {
        // the shared-memory opt-in is a per-device attribute of the kernel: set once per device ordinal
        constexpr int MAX_DEVICES = 64;
        static std::mutex mu;
        static bool smem_set[MAX_DEVICES] = {};
        int dev = -1;
        CU(cudaGetDevice(&dev));
        std::lock_guard<std::mutex> lock(mu);
        if (dev < 0 || dev >= MAX_DEVICES || !smem_set[dev]) {
            CU(cudaFuncSetAttribute(st_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)finish_smem));
            if (dev >= 0 && dev < MAX_DEVICES) smem_set[dev] = true;
        }
    }
    if (!sampled) EF(enqueue_topk_fast_sample(st, a, pitch_a, b, pitch_b, batch, d, k, B, launches));
    dim3 grid((unsigned)ceil_div(B.nreg, ST_COLLECT_WARPS), (unsigned)batch);
    const bool vec = aligned16(a) && pitch_a % 4 == 0 && (!b || (aligned16(b) && pitch_b % 4 == 0));
    auto collect = vec ? st_collect_kernel<true> : st_collect_kernel<false>;
    collect<<<grid, ST_COLLECT_WARPS * 32, 0, st>>>(a, pitch_a, b, pitch_b, d, B.nreg, B.thr, B.cand, B.region_cnt, B.flags);
    st_finish_kernel<<<batch, ST_THREADS, finish_smem, st>>>(a, pitch_a, b, pitch_b, d, B.nreg, k, B.cand, B.region_cnt,
                                                             B.flags, idx_out, val_out, gi_rows, ld, B.slow_count, tile_off,
                                                             ntiles, AGG_TILE, status);
    if (launches) *launches += 2;
    CU(cudaGetLastError());
    return EF21_OK;
}

// Exact Top-k of v = a - b for `batch` vectors (b may be null); general multi-block path.
ef21_status enqueue_topk_general(cudaStream_t st, const float* a, i64 pitch_a, const float* b, i64 pitch_b,
                                 int batch, i64 d, int k, int* idx_out, float* val_out,
                                 const TopkBuffers& B, i64* launches, unsigned* status, float* apply_to = nullptr,
                                 i64 pitch_apply = 0, bool* applied = nullptr) {
    if (applied) *applied = false;
    if (d <= TKS_MAX_D) {
        // short vectors: the whole selection in one launch, one block per vector (no scratch); the same
        // launch adds the messages to apply_to if the caller asks for it
        tk_small_kernel<<<batch, TKS_BLOCK, (size_t)d * 4, st>>>(a, pitch_a, b, pitch_b, (int)d, k, idx_out, val_out,
                                                                 apply_to, pitch_apply, status);
        if (applied) *applied = apply_to != nullptr;
        if (launches) *launches += 1;
        CU(cudaGetLastError());
        return EF21_OK;
    }
    tk_reset_kernel<<<batch, 256, 0, st>>>(B.state, B.hist, batch, (unsigned)k);
    dim3 grid((unsigned)B.nchunks, (unsigned)batch);
    for (int level = 0; level < 3; ++level) {
        tk_hist_kernel<<<grid, TK_BLOCK, 0, st>>>(a, pitch_a, b, pitch_b, d, level, B.state, B.hist);
        tk_find_kernel<<<batch, 1024, 0, st>>>(B.state, B.hist, level);
    }
    tk_count_kernel<<<grid, TK_BLOCK, 0, st>>>(a, pitch_a, b, pitch_b, d, B.state, B.chunks, B.nchunks);
    tk_scan_kernel<<<batch, 1024, 0, st>>>(B.chunks, B.nchunks);
    tk_write_kernel<<<grid, TK_BLOCK, 0, st>>>(a, pitch_a, b, pitch_b, d, B.state, B.chunks, B.nchunks, k,
                                               idx_out, val_out, status);
    if (launches) *launches += 10;
    CU(cudaGetLastError());
    return EF21_OK;
}

ef21_status enqueue_grads(ef21_ctx* c, bool with_loss) {
    if (c->num_tiles > 0) {
        GradTileKernel stream = grad_stream_lookup(c->L.ld);
        if (stream)
            stream<<<c->num_tiles, GRAD_STREAM_BLOCK, (size_t)(GRAD_STREAM_BLOCK / 32) * c->L.ld * 4, c->stream>>>(
                c->at<float>(c->L.A), c->at<float>(c->L.y), c->x(), c->at<RowTile>(c->L.tiles), (int)c->L.ld, c->objective,
                c->at<float>(c->L.partial), with_loss ? c->at<double>(c->L.loss_partial) : nullptr, nullptr, 0,
                c->at<i64>(c->L.row_off), c->status());
        else
            grad_tiles_kernel<<<c->num_tiles, GRAD_BLOCK, 0, c->stream>>>(
                c->at<float>(c->L.A), c->at<float>(c->L.y), c->x(), c->at<RowTile>(c->L.tiles), (int)c->L.ld, c->objective,
                c->at<float>(c->L.partial), with_loss ? c->at<double>(c->L.loss_partial) : nullptr, nullptr, 0,
                c->at<i64>(c->L.row_off), c->status());
        c->launches += 1;
    }
    dim3 grid((unsigned)ceil_div(c->L.ld, GRAD_FINISH_COLS), (unsigned)c->n);
    grad_finish_kernel<<<grid, GRAD_FINISH_COLS * GRAD_FINISH_LANES, 0, c->stream>>>(
        c->at<float>(c->L.partial), c->at<int>(c->L.tile_begin), c->at<i64>(c->L.row_off), c->x(), c->lambda, (int)c->d,
        (int)c->L.ld, c->at<float>(c->L.grad), 0);
    c->launches += 1;
    CU(cudaGetLastError());
    return EF21_OK;
}

// Minibatch gradients (Algorithm 5): worker i averages over the tau rows batch[i][0..tau) of its shard.
ef21_status enqueue_minibatch_grads(ef21_ctx* c, const int* batch_dev, int tau) {
    if (c->mb_tau != tau) {            // (re)build the tile table of the batch lists
        const int R = c->L.tile_rows;
        c->mb_tiles.clear();
        c->mb_tile_begin.assign(c->n + 1, 0);
        for (int i = 0; i < c->n; ++i) {
            c->mb_tile_begin[i] = (int)c->mb_tiles.size();
            for (int r = 0; r < tau; r += R) {
                RowTile t; t.row0 = r; t.rows = std::min(R, tau - r); t.worker = i;
                c->mb_tiles.push_back(t);
            }
        }
        c->mb_tile_begin[c->n] = (int)c->mb_tiles.size();
        if ((i64)c->mb_tiles.size() > c->L.max_tiles) return EF21_ERR_WORKSPACE;
        CU(cudaMemcpyAsync(c->at<int>(c->L.mb_tile_begin), c->mb_tile_begin.data(), (size_t)(c->n + 1) * 4,
                           cudaMemcpyHostToDevice, c->stream));
        CU(cudaMemcpyAsync(c->at<RowTile>(c->L.mb_tiles), c->mb_tiles.data(), c->mb_tiles.size() * sizeof(RowTile),
                           cudaMemcpyHostToDevice, c->stream));
        CU(cudaStreamSynchronize(c->stream));      // the host vectors may be rebuilt by the next call
        c->mb_tau = tau;
    }
    GradTileKernel stream = grad_stream_lookup(c->L.ld);
    if (stream)
        stream<<<(unsigned)c->mb_tiles.size(), GRAD_STREAM_BLOCK, (size_t)(GRAD_STREAM_BLOCK / 32) * c->L.ld * 4, c->stream>>>(
            c->at<float>(c->L.A), c->at<float>(c->L.y), c->x(), c->at<RowTile>(c->L.mb_tiles), (int)c->L.ld, c->objective,
            c->at<float>(c->L.partial), nullptr, batch_dev, tau, c->at<i64>(c->L.row_off), c->status());
    else
        grad_tiles_kernel<<<(unsigned)c->mb_tiles.size(), GRAD_BLOCK, 0, c->stream>>>(
            c->at<float>(c->L.A), c->at<float>(c->L.y), c->x(), c->at<RowTile>(c->L.mb_tiles), (int)c->L.ld, c->objective,
            c->at<float>(c->L.partial), nullptr, batch_dev, tau, c->at<i64>(c->L.row_off), c->status());
    dim3 grid((unsigned)ceil_div(c->L.ld, GRAD_FINISH_COLS), (unsigned)c->n);
    grad_finish_kernel<<<grid, GRAD_FINISH_COLS * GRAD_FINISH_LANES, 0, c->stream>>>(
        c->at<float>(c->L.partial), c->at<int>(c->L.mb_tile_begin), c->at<i64>(c->L.row_off), c->x(), c->lambda, (int)c->d,
        (int)c->L.ld, c->at<float>(c->L.grad), tau);
    c->launches += 2;
    CU(cudaGetLastError());
    return EF21_OK;
}

// Selection half of a message round: c_i = C(a_i - g_i) and g_i += c_i.  sampled: the threshold
// kernel of the one-pass Top-k has already run for these inputs.
ef21_status enqueue_round_select(ef21_ctx* c, const float* a, i64 pitch_a, bool sampled) {
    TopkBuffers B = topk_buffers(c->ws + c->L.topk, c->L.tk);
    if (B.fast && !c->force_general_topk) {
        // the finish kernel also leaves the per-tile offsets of the messages for the aggregation
        EF(enqueue_topk_fast(c->stream, a, pitch_a, c->gi(), c->L.ld, c->n, c->d, c->k, c->msg_idx(), c->msg_val(),
                             c->gi(), c->L.ld, B, &c->launches, c->status(), sampled, c->at<int>(c->L.agg_off), c->L.agg_tiles));
        c->agg_off_ready = true;
    } else {
        c->agg_off_ready = false;
        bool applied = false;
        EF(enqueue_topk_general(c->stream, a, pitch_a, c->gi(), c->L.ld, c->n, c->d, c->k, c->msg_idx(),
                                c->msg_val(), B, &c->launches, c->status(), c->gi(), c->L.ld, &applied));
        if (!applied) {
            const i64 total = (i64)c->n * c->k;
            apply_messages_kernel<<<(unsigned)ceil_div(total, 256), 256, 0, c->stream>>>(c->msg_idx(), c->msg_val(), total,
                                                                                        c->k, c->L.ld, c->gi());
            c->launches += 1;
        }
    }
    CU(cudaGetLastError());
    return EF21_OK;
}

ef21_status enqueue_aggregate_into(ef21_ctx* c, float* target, float factor, bool update_x);

// Aggregation half: g += (1/n) sum c_i (and, if update_x, x <- x - gamma g_old in the same kernel).
ef21_status enqueue_round_aggregate(ef21_ctx* c, bool update_x) {
    return enqueue_aggregate_into(c, c->g(), 1.0f / (float)c->n, update_x);
}

// target_j += factor * (sum over workers, ascending, of the values sent for coordinate j).
ef21_status enqueue_aggregate_into(ef21_ctx* c, float* target, float factor, bool update_x) {
    if (!c->agg_off_ready && !(c->L.agg_tiles == 1 && c->agg_off_static)) {
        const i64 noff = (i64)c->n * (c->L.agg_tiles + 1);
        agg_offsets_kernel<<<(unsigned)ceil_div(noff, 256), 256, 0, c->stream>>>(c->msg_idx(), c->n, c->k,
                                                                                c->L.agg_tiles, c->at<int>(c->L.agg_off));
        c->launches += 1;
        c->agg_off_static = c->L.agg_tiles == 1;
    }
    c->agg_off_ready = false;
    auto kern = c->n <= AGG_STAGE_MAX_N
                    ? (update_x ? aggregate_staged_kernel<true> : aggregate_staged_kernel<false>)
                    : (update_x ? aggregate_kernel<true> : aggregate_kernel<false>);
    kern<<<c->L.agg_tiles, AGG_BLOCK, 0, c->stream>>>(c->msg_idx(), c->msg_val(), c->at<int>(c->L.agg_off), c->n, c->k,
                                                      c->L.agg_tiles, c->d, factor, c->gamma, target, c->x());
    c->launches += 1;
    CU(cudaGetLastError());
    return EF21_OK;
}

ef21_status enqueue_round(ef21_ctx* c, const float* a, i64 pitch_a, bool update_x) {
    EF(enqueue_round_select(c, a, pitch_a, false));
    return enqueue_round_aggregate(c, update_x);
}

// One round of EF21+ (Algorithm 3) on local gradients a: both compressed vectors, the choice by
// distortion, g_i <- chosen, g = (1/n) sum g_i.
ef21_status enqueue_plus_round(ef21_ctx* c, const float* a, i64 pitch_a) {
    TopkBuffers B = topk_buffers(c->ws + c->L.topk, c->L.tk);
    int* idx_b = c->at<int>(c->L.msg2_idx);
    float* val_b = c->at<float>(c->L.msg2_val);
    if (B.fast && !c->force_general_topk) {
        EF(enqueue_topk_fast(c->stream, a, pitch_a, c->gi(), c->L.ld, c->n, c->d, c->k, c->msg_idx(), c->msg_val(),
                             nullptr, 0, B, &c->launches, c->status()));
        EF(enqueue_topk_fast(c->stream, a, pitch_a, nullptr, 0, c->n, c->d, c->k, idx_b, val_b, nullptr, 0, B, &c->launches, c->status()));
    } else {
        EF(enqueue_topk_general(c->stream, a, pitch_a, c->gi(), c->L.ld, c->n, c->d, c->k, c->msg_idx(), c->msg_val(), B,
                                &c->launches, c->status()));
        EF(enqueue_topk_general(c->stream, a, pitch_a, nullptr, 0, c->n, c->d, c->k, idx_b, val_b, B, &c->launches, c->status()));
    }
    plus_choose_kernel<<<c->n, PLUS_BLOCK, 0, c->stream>>>(a, pitch_a, c->gi(), c->L.ld, c->d, c->k, c->msg_idx(), c->msg_val(),
                                                          idx_b, val_b, c->at<float>(c->L.plus_old), c->at<unsigned>(c->L.plus_bitmap),
                                                          c->at<int>(c->L.plus_choice));
    const unsigned blocks = (unsigned)std::min<i64>(ceil_div(c->d, 256), 148 * 8);
    dense_mean_kernel<<<blocks, 256, 0, c->stream>>>(c->gi(), c->L.ld, c->n, c->d, 1.0f / (float)c->n, c->g());
    c->launches += 2;
    CU(cudaGetLastError());
    return EF21_OK;
}

// One iteration of the original error feedback method (Algorithm 4) on local gradients a, from the
// state (x, e_i): e_i becomes p_i = e_i + gamma a_i, the messages are w_i = C(p_i), the master moves
// x by -(1/n) sum w_i, and e_i <- p_i - w_i.
ef21_status enqueue_ef_round(ef21_ctx* c, const float* a, i64 pitch_a) {
    TopkBuffers B = topk_buffers(c->ws + c->L.topk, c->L.tk);
    const unsigned blocks = (unsigned)std::min<i64>(ceil_div((i64)c->n * c->d, 256), 148 * 16);
    ef_compose_kernel<<<blocks, 256, 0, c->stream>>>(a, pitch_a, c->gi(), c->L.ld, c->n, c->d, c->gamma);
    c->launches += 1;
    if (B.fast && !c->force_general_topk) {
        EF(enqueue_topk_fast(c->stream, c->gi(), c->L.ld, nullptr, 0, c->n, c->d, c->k, c->msg_idx(), c->msg_val(),
                             nullptr, 0, B, &c->launches, c->status()));
    } else {
        EF(enqueue_topk_general(c->stream, c->gi(), c->L.ld, nullptr, 0, c->n, c->d, c->k, c->msg_idx(), c->msg_val(), B,
                                &c->launches, c->status()));
    }
    const i64 total = (i64)c->n * c->k;
    ef_subtract_sent_kernel<<<(unsigned)ceil_div(total, 256), 256, 0, c->stream>>>(c->msg_idx(), c->msg_val(), total, c->k,
                                                                                  c->L.ld, c->gi());
    c->launches += 1;
    c->agg_off_ready = false;
    CU(cudaGetLastError());
    return enqueue_aggregate_into(c, c->x(), -(1.0f / (float)c->n), false);
}

ef21_status enqueue_x_update(ef21_ctx* c) {
    const unsigned blocks = (unsigned)std::min<i64>(ceil_div(c->d, 256), 148 * 8);
    x_update_kernel<<<blocks, 256, 0, c->stream>>>(c->g(), c->x(), c->d, c->gamma);
    c->launches += 1;
    CU(cudaGetLastError());
    return EF21_OK;
}

ef21_status zero_state(ef21_ctx* c) {
    CU(cudaMemsetAsync(c->gi(), 0, (size_t)c->n * c->L.ld * 4, c->stream));
    CU(cudaMemsetAsync(c->g(), 0, (size_t)c->L.ld * 4, c->stream));
    return EF21_OK;
}

ef21_status init_from(ef21_ctx* c, const float* V, i64 pitch, int mode) {
    EF(zero_state(c));
    if (mode == EF21_INIT_COMPRESSED) {
        EF(enqueue_round(c, V, pitch, false));
    } else if (mode == EF21_INIT_GRADIENT) {
        const unsigned blocks = (unsigned)std::min<i64>(ceil_div(c->d, 256), 148 * 8);
        dense_init_kernel<<<blocks, 256, 0, c->stream>>>(V, pitch, c->n, c->d, c->L.ld, 1.0f / (float)c->n,
                                                        c->gi(), c->g());
        c->launches += 1;
        CU(cudaGetLastError());
    }
    c->inited = true;
    return EF21_OK;
}

ef21_status finish_load(ef21_ctx* c, const i64* row_offsets_host) {
    // Validate and build the tile table.
    if (row_offsets_host[0] != 0 || row_offsets_host[c->n] != c->N) return EF21_ERR_INVALID_ARG;
    for (int i = 0; i < c->n; ++i)
        if (row_offsets_host[i + 1] < row_offsets_host[i]) return EF21_ERR_INVALID_ARG;
    c->row_off.assign(row_offsets_host, row_offsets_host + c->n + 1);
    c->tiles.clear();
    c->tile_begin.assign(c->n + 1, 0);
    const int R = c->L.tile_rows;
    for (int i = 0; i < c->n; ++i) {
        c->tile_begin[i] = (int)c->tiles.size();
        for (i64 r = c->row_off[i]; r < c->row_off[i + 1]; r += R) {
            RowTile t;
            t.row0 = r;
            t.rows = (int)std::min<i64>(R, c->row_off[i + 1] - r);
            t.worker = i;
            c->tiles.push_back(t);
        }
    }
    c->tile_begin[c->n] = (int)c->tiles.size();
    c->num_tiles = (int)c->tiles.size();
    if ((i64)c->num_tiles > c->L.max_tiles) return EF21_ERR_WORKSPACE;
    // a captured launch-path iteration has the old tile count baked into its grid
    if (c->iter_graph) { cudaGraphExecDestroy(c->iter_graph); c->iter_graph = nullptr; }
    c->plan_valid = false; c->mb_plan_valid = false;
    CU(cudaMemcpyAsync(c->at<i64>(c->L.row_off), c->row_off.data(), (size_t)(c->n + 1) * 8, cudaMemcpyHostToDevice, c->stream));
    CU(cudaMemcpyAsync(c->at<int>(c->L.tile_begin), c->tile_begin.data(), (size_t)(c->n + 1) * 4, cudaMemcpyHostToDevice, c->stream));
    if (c->num_tiles > 0)
        CU(cudaMemcpyAsync(c->at<RowTile>(c->L.tiles), c->tiles.data(), (size_t)c->num_tiles * sizeof(RowTile),
                           cudaMemcpyHostToDevice, c->stream));
    c->shards_loaded = true;
    return EF21_OK;
}


// ---------------------------------------------------------------------------------------------
// Persistent path
// ---------------------------------------------------------------------------------------------


// From two entries per worker on, the received messages are scattered into a [n][ld] table in shared
// memory (if that table is small): aggregation then costs n reads per coordinate instead of n*k.
bool pk_use_table(int n, int ld, int k) { return k >= 2 && (size_t)n * ld * 4 <= (size_t)PK_TABLE_MAX_BYTES; }

size_t pk_smem_bytes(bool plus, int n, int k, int ld, int C, int nmsg, int src, i64 rows_cta, int threads) {
    size_t b = (size_t)(6 + threads / 32 + C) * ld * 4 + (size_t)((nmsg + 1) & ~1) * 8 + (size_t)((2 * ld + 15) & ~15);
    if (plus) b += (size_t)n * ld * 4 + (size_t)ld * 4 + (size_t)((ld + 15) & ~15) + (size_t)((n + 15) & ~15) + (size_t)2 * (threads / 32) * 8 + 16;   // replicas of all g_i, grad_i, second selection, branches, distortion partials
    else if (pk_use_table(n, ld, k)) b += (size_t)n * ld * 4;
    if (src == PK_SRC_SMEM) b += (size_t)rows_cta * ld * 4;
    return b;
}

// Shared memory of the kernel whose last warp serves the block (persistent_roles.inc): x, g, g_i, message
// sums, one partial per compute warp, the partials of the cluster's blocks, the message flags, the row slice.
size_t pk_roles_smem_bytes(int ld, int C, int src, i64 rows_cta, int threads) {
    size_t b = (size_t)(6 + threads / 32 + C) * ld * 4 + (size_t)((ld + 15) & ~15);
    if (src == PK_SRC_SMEM) b += (size_t)rows_cta * ld * 4;
    return b;
}

PersistPlan plan_persistent_body(ef21_ctx* c, bool roles, int tau = 0);

// Chooses the kernel body, cluster size, block size, rows per batch and the source of the shard rows; checks
// that all n clusters can be resident at once (the blocks wait on one another through global memory).
PersistPlan plan_persistent(ef21_ctx* c) {
    // Automatic choice: the serving-warp body for Top-1 (2.6 against 3.2 us per iteration on the mushrooms-shaped
    // workload, 3.4 against 4.0 on the a9a-shaped one, the same 10.4 on the w8a-shaped one, measured); with more
    // entries per message its k arg-max rounds in one warp cost more than the whole block counting ranks.
    const bool roles_can = c->variant != EF21_VARIANT_EF21_PLUS && c->k <= PK_ROLES_MAX_K;
    const bool roles_first = c->pk_body == 1 || (c->pk_body == 0 && c->k == 1);
    if (roles_can && roles_first) {
        PersistPlan P = plan_persistent_body(c, true);
        if (P.ok || c->pk_body == 1) return P;
    }
    if (c->pk_body == 1) { PersistPlan P; P.ok = false; return P; }
    return plan_persistent_body(c, false);
}

// tau > 0: plan for the stochastic variant (tau sampled rows per worker and iteration, read from global memory).
PersistPlan plan_persistent_body(ef21_ctx* c, bool roles, int tau) {
    PersistPlan P; P.ok = false; P.roles = roles;
    const int ld = (int)c->L.ld;
    if (!c->shards_loaded || ld > 512 || c->k > PK_MAX_K || (i64)c->n * c->k > PK_MAX_MSGS) return P;
    const bool plus = c->variant == EF21_VARIANT_EF21_PLUS;
    if (plus && (size_t)c->n * ld * 4 > (size_t)PK_TABLE_MAX_BYTES) return P;      // every block keeps all g_i
    int dev = 0, sms = 0, max_smem = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return P;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    const int chunk_slots = (ld / 4 + 31) / 32;
    const int max_rb256 = chunk_slots == 1 ? 32 : (chunk_slots == 2 ? 16 : 8);      // rb * chunk_slots <= 32
    const int max_rb512 = chunk_slots == 1 ? 16 : (chunk_slots == 2 ? 8 : 4);       // rb * chunk_slots <= 16
    i64 max_m = 0;
    for (int i = 0; i < c->n; ++i) max_m = std::max<i64>(max_m, c->row_off[i + 1] - c->row_off[i]);
    if (tau > 0) max_m = tau;
    const int nmsg = c->n * c->k;

    // One candidate shape for a cluster size: rows in registers with 8 warps if they fit, else with 16
    // warps, else staged in shared memory or streamed from L2 with 16 warps.
    auto shape_for = [&](int C, int& rb, int& src, int& threads, int& extra) {
        const i64 rows_cta = ceil_div(std::max<i64>(max_m, 1), C);
        rb = 0; extra = 0;
        for (int cand = 8; cand <= max_rb256 && !rb; cand *= 2)
            if (ceil_div(rows_cta, cand) <= 8) { rb = cand; src = PK_SRC_REG; threads = 256; }
        for (int cand = 4; cand <= max_rb512 && !rb; cand *= 2)
            if (ceil_div(rows_cta, cand) <= 16) { rb = cand; src = PK_SRC_REG; threads = 512; }
        // one row more than 16 per warp still fits the registers of 16 warps (one chunk slot)
        if (!rb && chunk_slots == 1 && ceil_div(rows_cta, 17) <= 16 && c->pk_threads == 0 && c->pk_rb == 0 && c->pk_src < 0) {
            rb = 16; extra = 1; src = PK_SRC_REG; threads = 512;
        }
        if (!rb) {
            rb = max_rb512; threads = 512;
            const size_t with_slice = roles ? pk_roles_smem_bytes(ld, C, PK_SRC_SMEM, rows_cta, threads)
                                            : pk_smem_bytes(plus, c->n, c->k, ld, C, nmsg, PK_SRC_SMEM, rows_cta, threads);
            src = with_slice <= (size_t)max_smem - 1024 ? PK_SRC_SMEM : PK_SRC_GMEM;
        }
        if (c->pk_threads > 0) {
            threads = c->pk_threads;
            const int cap = threads == 512 ? max_rb512 : max_rb256;
            if (rb > cap) rb = cap;
            if (src == PK_SRC_REG && ceil_div(rows_cta, rb) > threads / 32) src = PK_SRC_SMEM;
        }
        if (c->pk_rb > 0) {
            rb = c->pk_rb;
            if (src == PK_SRC_REG && ceil_div(rows_cta, rb) > threads / 32) src = PK_SRC_SMEM;
        }
        if (c->pk_src >= 0) src = c->pk_src;
        if (tau > 0) src = PK_SRC_SAMPLED;       // sampled rows change every iteration: read through the list
        return rows_cta;
    };

    // Order in which cluster sizes are tried: the smallest one that keeps a block's rows in registers
    // (fewer blocks = fewer senders and pollers), then the largest first.
    int order[9], norder = 0;
    if (c->pk_cluster > 0) {
        order[norder++] = c->pk_cluster;
    } else {
        int pref = 0;
        for (int C = 1; C <= 8 && !pref; ++C) {
            if ((i64)c->n * C > sms) break;
            int rb, src, threads, extra;
            shape_for(C, rb, src, threads, extra);
            if ((src == PK_SRC_REG || tau > 0) && threads == 256 && rb <= 16) pref = C;
        }
        if (pref) order[norder++] = pref;
        for (int C = 8; C >= 1; --C)
            if (C != pref) order[norder++] = C;
    }
    for (int oi = 0; oi < norder; ++oi) {
        const int C = order[oi];
        if ((i64)c->n * C > sms) continue;
        int rb = 0, src = PK_SRC_GMEM, threads = 256, extra = 0;
        const i64 rows_cta = shape_for(C, rb, src, threads, extra);
        if (c->pk_cluster == 0 && C > 1 && rows_cta < 8) continue;       // do not split below one batch
        if (src == PK_SRC_REG && ceil_div(rows_cta, rb + extra) > threads / 32) continue;
        const size_t smem = roles ? pk_roles_smem_bytes(ld, C, src, rows_cta, threads)
                                  : pk_smem_bytes(plus, c->n, c->k, ld, C, nmsg, src, rows_cta, threads);
        if (smem > (size_t)max_smem - 1024) continue;
        PersistKernel kern;
        if (roles)
            kern = c->variant == EF21_VARIANT_EF ? pk_lookup_ef(chunk_slots, rb, src, threads, extra)
                                                   : pk_lookup_ef21(chunk_slots, rb, src, threads, extra);
        else
            kern = c->variant == EF21_VARIANT_EF ? pk_lookup_wide_ef(chunk_slots, rb, src, threads, extra)
                   : (plus ? pk_lookup_plus(chunk_slots, rb, src, threads, extra)
                           : pk_lookup_wide_ef21(chunk_slots, rb, src, threads, extra));
        if (!kern) continue;
        const int block_threads = threads;
        // the device's opt-in limit (less the kernel's static part), so that no other handle's plan for the same
        // kernel can lower it under this one's need
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024) != cudaSuccess) {
            cudaGetLastError();
            continue;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(c->n * C)); cfg.blockDim = dim3((unsigned)block_threads); cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        int active = 0;
        if (cudaOccupancyMaxActiveClusters(&active, kern, &cfg) != cudaSuccess) { cudaGetLastError(); continue; }
        if (active < c->n) continue;
        P.ok = true; P.C = C; P.rb = rb; P.src = src; P.chunks = chunk_slots; P.threads = threads; P.extra = extra; P.smem = smem; P.kernel = kern;
        return P;
    }
    return P;
}

// Persistent launches of different handles must not overlap on a device.  Each needs all of its clusters resident at
// once (they wait on one another through global memory); two launches that each got part of the SMs would wait for
// the other's until their bounded waits expire.  Launches on one stream are ordered by the stream.  A launch on another
// stream than the device's last persistent launch first waits (on the device, not on the host) for everything enqueued
// on that stream so far.
struct PersistGate {
    std::mutex mu;
    bool any = false;              // a persistent launch has been enqueued on this device
    bool detached = false;         // its handle is gone: `ev` stands for the work, the stream is not touched again
    cudaStream_t last_stream = nullptr;
    cudaEvent_t ev = nullptr;
};
constexpr int GATE_DEVICES = 64;
PersistGate g_gate[GATE_DEVICES];

PersistGate* gate_of_device(int dev) { return (dev >= 0 && dev < GATE_DEVICES) ? &g_gate[dev] : nullptr; }

ef21_status gate_order_after_last(PersistGate* G, cudaStream_t stream) {
    if (!G->any || (!G->detached && G->last_stream == stream)) return EF21_OK;
    if (!G->ev) CU(cudaEventCreateWithFlags(&G->ev, cudaEventDisableTiming));
    if (!G->detached) CU(cudaEventRecord(G->ev, G->last_stream));
    CU(cudaStreamWaitEvent(stream, G->ev, 0));
    return EF21_OK;
}

// Called when a handle goes away: its stream may be destroyed by the caller afterwards, so what it has enqueued is
// pinned to the event now.
void gate_forget_stream(int dev, cudaStream_t stream) {
    PersistGate* G = gate_of_device(dev);
    if (!G) return;
    std::lock_guard<std::mutex> lock(G->mu);
    if (!G->any || G->detached || G->last_stream != stream) return;
    if (!G->ev && cudaEventCreateWithFlags(&G->ev, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); G->any = false; return; }
    if (cudaEventRecord(G->ev, stream) != cudaSuccess) { cudaGetLastError(); G->any = false; return; }
    G->detached = true;
}

ef21_status run_persistent(ef21_ctx* c, const PersistPlan& P, int steps, const int* batch = nullptr, int tau = 0) {
    PersistGate* G = gate_of_device(c->device);
    std::unique_lock<std::mutex> gate_lock;
    if (G) {
        gate_lock = std::unique_lock<std::mutex>(G->mu);
        EF(gate_order_after_last(G, c->stream));
    }
    PersistParams p;
    p.batch = batch; p.tau = tau;
    p.A = c->at<float>(c->L.A); p.y = c->at<float>(c->L.y); p.row_off = c->at<i64>(c->L.row_off);
    p.x = c->x(); p.g = c->g(); p.gi = c->gi(); p.msg_idx = c->msg_idx(); p.msg_val = c->msg_val();
    p.plus_choice = c->at<int>(c->L.plus_choice);
    p.slots = c->at<unsigned long long>(c->L.slots); p.status = c->status();
    p.n = c->n; p.d = (int)c->d; p.ld = (int)c->L.ld; p.k = c->k; p.C = P.C; p.steps = steps;
    p.objective = c->objective;
    p.slice_rows = 0; p.use_table = (c->variant != EF21_VARIANT_EF21_PLUS && pk_use_table(c->n, (int)c->L.ld, c->k)) ? 1 : 0; p.gamma = c->gamma; p.lambda = c->lambda; p.inv_n = 1.0f / (float)c->n;
    // the epochs run on from launch to launch, so the slot array (cleared once, at creation) needs no clearing here
    p.spin_limit = c->spin_limit; p.epoch0 = c->pk_epoch; p.par0 = c->pk_par;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(c->n * P.C)); cfg.blockDim = dim3((unsigned)P.threads);
    cfg.dynamicSmemBytes = P.smem;
    cfg.stream = c->stream;
    // A plain cluster launch: that all n clusters fit on the device at once was checked with the
    // occupancy query when the plan was made.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)P.C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, P.kernel, p);
    if (e != cudaSuccess) { cudaGetLastError(); return EF21_ERR_CUDA; }
    if (G) { G->any = true; G->detached = false; G->last_stream = c->stream; }
    c->launches += 1;
    c->pk_epoch = (unsigned)(((i64)c->pk_epoch + steps - 1) % 65535) + 1u;
    c->pk_par = (c->pk_par + (unsigned)steps) & 1u;
    c->pk_used_cluster = P.C; c->pk_used_rb = P.rb; c->pk_used_src = P.src; c->pk_used_threads = P.threads;
    c->pk_used_body = P.roles ? 1 : 2;
    return EF21_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------

extern "C" {

const char* ef21_status_string(ef21_status s) {
    switch (s) {
        case EF21_OK: return "ok";
        case EF21_ERR_INVALID_ARG: return "invalid argument";
        case EF21_ERR_STATE: return "call order violated";
        case EF21_ERR_WORKSPACE: return "workspace too small or misaligned";
        case EF21_ERR_CUDA: return "CUDA runtime error";
        case EF21_ERR_TIMEOUT: return "bounded device wait expired";
        case EF21_ERR_NONFINITE: return "non-finite value";
        case EF21_ERR_UNSUPPORTED: return "shape not supported by the requested path";
    }
    return "unknown status";
}

size_t ef21_workspace_bytes(int32_t n, int64_t d, int32_t k, int64_t total_rows) {
    if (!valid_shape(n, d, k, total_rows)) return 0;
    return make_layout(n, d, k, total_rows).total;
}

ef21_status ef21_create(ef21_ctx** out, int32_t n, int64_t d, int32_t k, float gamma, float lambda,
                        int64_t total_rows, void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
    if (!out || !valid_shape(n, d, k, total_rows)) return EF21_ERR_INVALID_ARG;
    if (!(gamma > 0.f) || !std::isfinite(gamma) || !(lambda >= 0.f) || !std::isfinite(lambda)) return EF21_ERR_INVALID_ARG;
    if (!workspace_dev) return EF21_ERR_INVALID_ARG;
    Layout L = make_layout(n, d, k, total_rows);
    if (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace_dev) % ALIGN) != 0) return EF21_ERR_WORKSPACE;
    ef21_ctx* c = new (std::nothrow) ef21_ctx();
    if (!c) return EF21_ERR_INVALID_ARG;
    c->n = n; c->d = d; c->k = k; c->gamma = gamma; c->lambda = lambda; c->N = total_rows;
    c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    c->device = -1;
    if (cudaGetDevice(&c->device) != cudaSuccess) { cudaGetLastError(); c->device = -1; }
    c->ws = static_cast<char*>(workspace_dev);
    c->L = L;
    c->shards_loaded = false; c->inited = false; c->num_tiles = 0;
    c->path = EF21_PATH_AUTO; c->last_path = 0; c->launches = 0;
    c->pk_cluster = 0; c->pk_rb = 0; c->pk_src = -1; c->pk_threads = 0; c->agg_off_ready = false; c->agg_off_static = false;
    c->pk_used_cluster = c->pk_used_rb = 0; c->pk_used_src = -1; c->pk_used_threads = 0;
    c->pk_body = 0; c->pk_used_body = 0; c->pk_epoch = 0u; c->pk_par = 0u; c->plan_valid = false; c->mb_plan_valid = false; c->mb_plan_tau = 0;
    c->spin_limit = 1u << 22;
    c->force_general_topk = false;
    c->variant = EF21_VARIANT_EF21;
    c->mb_tau = -1;
    c->objective = EF21_OBJECTIVE_LOGISTIC;
    c->aux_stream = nullptr; c->ev_fork = nullptr; c->ev_join = nullptr;
    cudaError_t e = cudaMemsetAsync(c->ws + L.status, 0, 256, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->x(), 0, (size_t)L.ld * 4, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->g(), 0, (size_t)L.ld * 4, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->gi(), 0, (size_t)n * L.ld * 4, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->msg_idx(), 0, (size_t)n * k * 4, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->msg_val(), 0, (size_t)n * k * 4, c->stream);
    if (e == cudaSuccess && L.tk.fast) e = cudaMemsetAsync(c->ws + L.topk + L.tk.slow_count, 0, 4, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.plus_choice, 0, (size_t)n * 4, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.slots, 0, (size_t)2 * n * k * 8, c->stream);
    if (e != cudaSuccess) { delete c; return EF21_ERR_CUDA; }
    *out = c;
    return EF21_OK;
}

void ef21_destroy(ef21_ctx* ctx) {
    if (!ctx) return;
    gate_forget_stream(ctx->device, ctx->stream);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->aux_stream) cudaStreamDestroy(ctx->aux_stream);
    if (ctx->iter_graph) cudaGraphExecDestroy(ctx->iter_graph);
    if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
    delete ctx;
}

ef21_status ef21_load_shards(ef21_ctx* c, const float* A_dev, const float* y_dev, const int64_t* row_offsets_host) {
    if (!c || !row_offsets_host) return EF21_ERR_INVALID_ARG;
    if (c->N == 0) return EF21_ERR_STATE;
    if (!A_dev || !y_dev) return EF21_ERR_INVALID_ARG;
    const unsigned blocks = (unsigned)std::min<i64>(ceil_div(c->N * c->L.ld, 256), 148 * 16);
    pad_rows_kernel<<<blocks, 256, 0, c->stream>>>(A_dev, c->N, (int)c->d, (int)c->L.ld, c->at<float>(c->L.A));
    c->launches += 1;
    CU(cudaGetLastError());
    CU(cudaMemcpyAsync(c->at<float>(c->L.y), y_dev, (size_t)c->N * 4, cudaMemcpyDeviceToDevice, c->stream));
    return finish_load(c, reinterpret_cast<const i64*>(row_offsets_host));
}

ef21_status ef21_load_shards_host(ef21_ctx* c, const float* A_host, const float* y_host, const int64_t* row_offsets_host) {
    if (!c || !row_offsets_host) return EF21_ERR_INVALID_ARG;
    if (c->N == 0) return EF21_ERR_STATE;
    if (!A_host || !y_host) return EF21_ERR_INVALID_ARG;
    // Host rows have pitch d; the device layout has pitch ld with zero padding.
    if (c->L.ld != c->d) CU(cudaMemsetAsync(c->at<float>(c->L.A), 0, (size_t)c->N * c->L.ld * 4, c->stream));
    CU(cudaMemcpy2DAsync(c->at<float>(c->L.A), (size_t)c->L.ld * 4, A_host, (size_t)c->d * 4, (size_t)c->d * 4,
                         (size_t)c->N, cudaMemcpyHostToDevice, c->stream));
    CU(cudaMemcpyAsync(c->at<float>(c->L.y), y_host, (size_t)c->N * 4, cudaMemcpyHostToDevice, c->stream));
    return finish_load(c, reinterpret_cast<const i64*>(row_offsets_host));
}

ef21_status ef21_set_x(ef21_ctx* c, const float* x0_dev) {
    if (!c || !x0_dev) return EF21_ERR_INVALID_ARG;
    CU(cudaMemcpyAsync(c->x(), x0_dev, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
    return EF21_OK;
}

ef21_status ef21_init(ef21_ctx* c, int32_t mode) {
    if (!c || mode < 0 || mode > 2) return EF21_ERR_INVALID_ARG;
    if (mode == EF21_INIT_ZERO) {
        EF(zero_state(c));
        c->inited = true;
        return EF21_OK;
    }
    if (!c->shards_loaded) return EF21_ERR_STATE;
    EF(enqueue_grads(c, false));
    return init_from(c, c->at<float>(c->L.grad), c->L.ld, mode);
}

ef21_status ef21_init_grads(ef21_ctx* c, const float* V_dev, int32_t mode) {
    if (!c || mode < 0 || mode > 2) return EF21_ERR_INVALID_ARG;
    if (mode != EF21_INIT_ZERO && !V_dev) return EF21_ERR_INVALID_ARG;
    return init_from(c, V_dev, c->d, mode);
}

// One iteration of ef21_step on the launch path, as plain kernel launches on the handle's stream.
static ef21_status enqueue_launch_iteration(ef21_ctx* c) {
    if (c->variant == EF21_VARIANT_EF) {
        EF(enqueue_grads(c, false));
        return enqueue_ef_round(c, c->at<float>(c->L.grad), c->L.ld);
    }
    EF(enqueue_x_update(c));
    EF(enqueue_grads(c, false));
    if (c->variant == EF21_VARIANT_EF21_PLUS) return enqueue_plus_round(c, c->at<float>(c->L.grad), c->L.ld);
    return enqueue_round(c, c->at<float>(c->L.grad), c->L.ld, false);
}

// `steps` launch-path iterations.  Short vectors (the one-launch Top-k) make an iteration a fixed list of
// five to nine small kernels whose cost is their launches: from the second iteration of a call on, the
// list is replayed as a CUDA graph captured once per handle and method.  The first iteration always
// runs as plain launches (it may still write the one-time aggregation offsets).  Anything that stands
// in the way (the caller's stream is itself being captured, capture or instantiation fails) leaves the
// plain launches, which give the same results.
static ef21_status run_launch_iterations(ef21_ctx* c, int steps) {
    int done = 0;
    const bool graphable = c->d <= TKS_MAX_D && steps >= 3 && !c->iter_graph_off;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (graphable && cudaStreamIsCapturing(c->stream, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) {
        EF(enqueue_launch_iteration(c));
        done = 1;
        const int key = c->variant * 16 + c->objective;
        if (c->iter_graph && c->iter_graph_key != key) { cudaGraphExecDestroy(c->iter_graph); c->iter_graph = nullptr; }
        if (!c->iter_graph) {
            const i64 before = c->launches;
            cudaGraph_t graph = nullptr;
            // captured on a stream of the library's own (the caller's may be the legacy default stream, which
            // cannot be captured); the graph is then launched into the caller's stream
            bool ok = c->cap_stream || cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) == cudaSuccess;
            ok = ok && cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
            if (ok) {
                cudaStream_t user_stream = c->stream;
                c->stream = c->cap_stream;
                const ef21_status st = enqueue_launch_iteration(c);
                c->stream = user_stream;
                ok = cudaStreamEndCapture(c->cap_stream, &graph) == cudaSuccess && st == EF21_OK && graph != nullptr;
            }
            if (ok) ok = cudaGraphInstantiate(&c->iter_graph, graph, 0) == cudaSuccess;
            if (graph) cudaGraphDestroy(graph);
            c->iter_graph_launches = c->launches - before;
            c->launches = before;                         // the captured iteration has not run
            if (!ok) {
                cudaGetLastError();
                if (c->iter_graph) { cudaGraphExecDestroy(c->iter_graph); c->iter_graph = nullptr; }
                c->iter_graph_off = true;
            } else {
                c->iter_graph_key = key;
            }
        }
        if (c->iter_graph) {
            for (; done < steps; ++done) {
                CU(cudaGraphLaunch(c->iter_graph, c->stream));
                c->launches += c->iter_graph_launches;
            }
        }
    } else {
        cudaGetLastError();
    }
    for (; done < steps; ++done) EF(enqueue_launch_iteration(c));
    c->last_path = EF21_PATH_LAUNCHES;
    return EF21_OK;
}

ef21_status ef21_step(ef21_ctx* c, int32_t steps) {
    if (!c || steps < 0) return EF21_ERR_INVALID_ARG;
    if (!c->shards_loaded || !c->inited) return EF21_ERR_STATE;
    if (steps == 0) return EF21_OK;
    if (c->path != EF21_PATH_LAUNCHES) {
        // planning asks the runtime several questions (attributes, occupancy of the cluster launch): once per
        // handle and setting, not once per call
        if (!c->plan_valid) { c->plan = plan_persistent(c); c->plan_valid = true; }
        const PersistPlan& P = c->plan;
        if (P.ok) {
            EF(run_persistent(c, P, steps));
            c->last_path = EF21_PATH_PERSISTENT;
            return EF21_OK;
        }
        if (c->path == EF21_PATH_PERSISTENT) return EF21_ERR_UNSUPPORTED;
    }
    return run_launch_iterations(c, steps);
}

ef21_status ef21_step_grads(ef21_ctx* c, const float* V_dev, int32_t steps) {
    if (!c || !V_dev || steps < 0) return EF21_ERR_INVALID_ARG;
    if (!c->inited) return EF21_ERR_STATE;
    if (c->variant == EF21_VARIANT_EF) {
        for (int t = 0; t < steps; ++t) EF(enqueue_ef_round(c, V_dev, c->d));
        c->last_path = EF21_PATH_LAUNCHES;
        return EF21_OK;
    }
    if (c->variant == EF21_VARIANT_EF21_PLUS) {
        for (int t = 0; t < steps; ++t) {
            EF(enqueue_x_update(c));
            EF(enqueue_plus_round(c, V_dev, c->d));
        }
        c->last_path = EF21_PATH_LAUNCHES;
        return EF21_OK;
    }
    const bool fast = c->L.tk.fast && !c->force_general_topk;
    if (fast && steps > 1 && !c->aux_stream) {
        if (cudaStreamCreateWithFlags(&c->aux_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            return EF21_ERR_CUDA;
        }
    }
    TopkBuffers B = topk_buffers(c->ws + c->L.topk, c->L.tk);
    if (!(fast && steps > 1)) {
        for (int t = 0; t < steps; ++t) {
            EF(enqueue_round_select(c, V_dev, c->d, false));
            EF(enqueue_round_aggregate(c, true));
        }
        c->last_path = EF21_PATH_LAUNCHES;
        return EF21_OK;
    }
    // Same V at every step: the threshold estimate of round t+1 needs V and g_i^{t+1} only, so it
    // follows the finish kernel of round t directly on this stream, and the aggregation of round t (g
    // and x) runs beside it on the second stream; the streaming pass of round t+1 waits for both.
    cudaStream_t main_stream = c->stream;
    for (int t = 0; t < steps; ++t) {
        // (letting the streaming pass start while the aggregation still runs made the pass 15-20 % slower)
        if (t > 0) CU(cudaStreamWaitEvent(main_stream, c->ev_join, 0));
        EF(enqueue_round_select(c, V_dev, c->d, t > 0));
        CU(cudaEventRecord(c->ev_fork, main_stream));
        CU(cudaStreamWaitEvent(c->aux_stream, c->ev_fork, 0));
        c->stream = c->aux_stream;
        const ef21_status agg = enqueue_round_aggregate(c, true);
        c->stream = main_stream;
        EF(agg);
        CU(cudaEventRecord(c->ev_join, c->aux_stream));
        if (t + 1 < steps)
            EF(enqueue_topk_fast_sample(main_stream, V_dev, c->d, c->gi(), c->L.ld, c->n, c->d, c->k, B, &c->launches));
    }
    CU(cudaStreamWaitEvent(main_stream, c->ev_join, 0));
    c->last_path = EF21_PATH_LAUNCHES;
    return EF21_OK;
}

ef21_status ef21_step_minibatches(ef21_ctx* c, const int32_t* batches_dev, int32_t tau, int32_t steps) {
    if (!c || !batches_dev || tau < 1 || steps < 0) return EF21_ERR_INVALID_ARG;
    if (!c->shards_loaded || !c->inited) return EF21_ERR_STATE;
    if (c->variant != EF21_VARIANT_EF21) return EF21_ERR_UNSUPPORTED;
    for (int i = 0; i < c->n; ++i)
        if (c->row_off[i + 1] - c->row_off[i] < tau) return EF21_ERR_INVALID_ARG;
    if (steps == 0) return EF21_OK;
    if (c->path != EF21_PATH_LAUNCHES && c->k <= PK_ROLES_MAX_K && c->pk_body != 2) {
        if (!c->mb_plan_valid || c->mb_plan_tau != tau) {
            c->mb_plan = plan_persistent_body(c, true, tau);
            c->mb_plan_tau = tau; c->mb_plan_valid = true;
        }
        if (c->mb_plan.ok) {
            EF(run_persistent(c, c->mb_plan, steps, batches_dev, tau));
            c->last_path = EF21_PATH_PERSISTENT;
            return EF21_OK;
        }
    }
    if (c->path == EF21_PATH_PERSISTENT) return EF21_ERR_UNSUPPORTED;
    for (int t = 0; t < steps; ++t) {
        EF(enqueue_x_update(c));
        EF(enqueue_minibatch_grads(c, batches_dev + (size_t)t * c->n * tau, tau));
        EF(enqueue_round(c, c->at<float>(c->L.grad), c->L.ld, false));
    }
    c->last_path = EF21_PATH_LAUNCHES;
    return EF21_OK;
}

ef21_status ef21_step_minibatch(ef21_ctx* c, const int32_t* batch_dev, int32_t tau) {
    return ef21_step_minibatches(c, batch_dev, tau, 1);
}

ef21_status ef21_step_randk(ef21_ctx* c, const float* V_dev, const int32_t* sets_dev, int32_t steps) {
    if (!c || !sets_dev || steps < 0) return EF21_ERR_INVALID_ARG;
    if (!c->inited || (!V_dev && !c->shards_loaded)) return EF21_ERR_STATE;
    if (c->variant != EF21_VARIANT_EF21) return EF21_ERR_UNSUPPORTED;
    const i64 total = (i64)c->n * c->k;
    for (int t = 0; t < steps; ++t) {
        EF(enqueue_x_update(c));
        if (!V_dev) EF(enqueue_grads(c, false));
        const float* a = V_dev ? V_dev : c->at<float>(c->L.grad);
        const i64 pitch = V_dev ? c->d : c->L.ld;
        randk_select_kernel<<<(unsigned)ceil_div(total, 256), 256, 0, c->stream>>>(
            a, pitch, c->gi(), c->L.ld, sets_dev + (size_t)t * total, total, c->k, c->d, c->msg_idx(), c->msg_val(), c->status());
        c->launches += 1;
        CU(cudaGetLastError());
        c->agg_off_ready = false;
        EF(enqueue_round_aggregate(c, false));
    }
    c->last_path = EF21_PATH_LAUNCHES;
    return EF21_OK;
}

ef21_status ef21_local_grads(ef21_ctx* c, float* grads_out_dev) {
    if (!c || !grads_out_dev) return EF21_ERR_INVALID_ARG;
    if (!c->shards_loaded) return EF21_ERR_STATE;
    EF(enqueue_grads(c, false));
    CU(cudaMemcpy2DAsync(grads_out_dev, (size_t)c->d * 4, c->at<float>(c->L.grad), (size_t)c->L.ld * 4,
                         (size_t)c->d * 4, (size_t)c->n, cudaMemcpyDeviceToDevice, c->stream));
    return EF21_OK;
}

size_t ef21_topk_workspace_bytes(int32_t batch, int64_t d, int32_t k) {
    if (batch < 1 || batch > 65535 || !valid_shape(1, d, k, 0)) return 0;
    return topk_layout(batch, d, k).total;
}

ef21_status ef21_topk(const float* v_dev, int32_t batch, int64_t d, int32_t k, int32_t* idx_out_dev,
                      float* val_out_dev, void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
    if (!v_dev || !idx_out_dev || !val_out_dev || batch < 1 || batch > 65535 || !valid_shape(1, d, k, 0))
        return EF21_ERR_INVALID_ARG;
    TopkLayout L = topk_layout(batch, d, k);
    if (!workspace_dev || workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace_dev) % ALIGN) != 0)
        return EF21_ERR_WORKSPACE;
    TopkBuffers B = topk_buffers(static_cast<char*>(workspace_dev), L);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (B.fast)
        return enqueue_topk_fast(st, v_dev, d, nullptr, 0, batch, d, k, idx_out_dev, val_out_dev, nullptr, 0, B, nullptr, nullptr);
    return enqueue_topk_general(st, v_dev, d, nullptr, 0, batch, d, k, idx_out_dev, val_out_dev, B, nullptr, nullptr);
}

// ---------------------------------------------------------------------------------------------
// Top-k without any caller-provided or allocated scratch
// ---------------------------------------------------------------------------------------------
// Scratch of ef21_topk_static: lives in the library image, so every GPU that loads the library
// holds these bytes until the process exits.
constexpr size_t TOPK_STATIC_SCRATCH_BYTES = (size_t)1 << 20;
constexpr int TOPK_STATIC_MAX_BATCH = 64;
constexpr i64 TOPK_STATIC_MAX_CHUNKS = 16384;      // batch * ceil(d / 4096)
static __device__ __align__(256) unsigned char g_topk_static_scratch[TOPK_STATIC_SCRATCH_BYTES];

// Device address of the scratch array on the current device.  In host code the array's name is only
// a handle for the runtime, not an address a kernel could use, so the address is asked for once
// per device (with that device current) and cached.
static ef21_status topk_static_scratch(void** out) {
    constexpr int MAX_DEVICES = 64;
    static std::mutex mu;
    static void* addr[MAX_DEVICES] = {};
    int dev = -1;
    CU(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return EF21_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        CU(cudaGetSymbolAddress(&p, g_topk_static_scratch));
        if (!p) return EF21_ERR_CUDA;
        addr[dev] = p;
    }
    *out = addr[dev];
    return EF21_OK;
}

ef21_status ef21_topk_static(const float* v_dev, int32_t batch, int64_t d, int32_t k, int32_t* idx_out_dev,
                             float* val_out_dev, void* cuda_stream) {
    if (!v_dev || !idx_out_dev || !val_out_dev || batch < 1 || !valid_shape(1, d, k, 0)) return EF21_ERR_INVALID_ARG;
    if (batch > TOPK_STATIC_MAX_BATCH || (i64)batch * ceil_div(d, TK_CHUNK) > TOPK_STATIC_MAX_CHUNKS)
        return EF21_ERR_UNSUPPORTED;                     // beyond the built-in scratch
    const TopkLayout L = topk_layout_general(batch, d);      // the same three sections ef21_topk lays out
    if (L.total > TOPK_STATIC_SCRATCH_BYTES) return EF21_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    EF(topk_static_scratch(&scratch));
    TopkBuffers B = topk_buffers(static_cast<char*>(scratch), L);
    // tk_reset_kernel clears the selection state and the histograms of the vectors in use; the
    // per-chunk counts are fully rewritten before they are read.
    return enqueue_topk_general(reinterpret_cast<cudaStream_t>(cuda_stream), v_dev, d, nullptr, 0, batch, d, k,
                                idx_out_dev, val_out_dev, B, nullptr, nullptr);
}

static ef21_status copy_state_out(ef21_ctx* c, float* x, float* g, float* gi, int32_t* li, float* lv, cudaMemcpyKind kind) {
    if (x) CU(cudaMemcpyAsync(x, c->x(), (size_t)c->d * 4, kind, c->stream));
    if (g) CU(cudaMemcpyAsync(g, c->g(), (size_t)c->d * 4, kind, c->stream));
    if (gi) CU(cudaMemcpy2DAsync(gi, (size_t)c->d * 4, c->gi(), (size_t)c->L.ld * 4, (size_t)c->d * 4, (size_t)c->n, kind, c->stream));
    if (li) CU(cudaMemcpyAsync(li, c->msg_idx(), (size_t)c->n * c->k * 4, kind, c->stream));
    if (lv) CU(cudaMemcpyAsync(lv, c->msg_val(), (size_t)c->n * c->k * 4, kind, c->stream));
    return EF21_OK;
}

ef21_status ef21_get_state(ef21_ctx* c, float* x_dev, float* g_dev, float* gi_dev, int32_t* last_idx_dev, float* last_val_dev) {
    if (!c) return EF21_ERR_INVALID_ARG;
    return copy_state_out(c, x_dev, g_dev, gi_dev, last_idx_dev, last_val_dev, cudaMemcpyDeviceToDevice);
}

ef21_status ef21_get_state_host(ef21_ctx* c, float* x_host, float* g_host, float* gi_host, int32_t* last_idx_host, float* last_val_host) {
    if (!c) return EF21_ERR_INVALID_ARG;
    EF(copy_state_out(c, x_host, g_host, gi_host, last_idx_host, last_val_host, cudaMemcpyDeviceToHost));
    CU(cudaStreamSynchronize(c->stream));
    return EF21_OK;
}

ef21_status ef21_set_state(ef21_ctx* c, const float* x_dev, const float* g_dev, const float* gi_dev) {
    if (!c) return EF21_ERR_INVALID_ARG;
    if (x_dev) CU(cudaMemcpyAsync(c->x(), x_dev, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
    if (g_dev) CU(cudaMemcpyAsync(c->g(), g_dev, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
    if (gi_dev) CU(cudaMemcpy2DAsync(c->gi(), (size_t)c->L.ld * 4, gi_dev, (size_t)c->d * 4, (size_t)c->d * 4, (size_t)c->n,
                                     cudaMemcpyDeviceToDevice, c->stream));
    c->inited = true;
    return EF21_OK;
}

ef21_status ef21_eval(ef21_ctx* c, double* f, double* grad_norm2, double* G) {
    if (!c) return EF21_ERR_INVALID_ARG;
    if (!c->shards_loaded) return EF21_ERR_STATE;
    EF(enqueue_grads(c, true));
    eval_reduce_kernel<<<1, 1024, 0, c->stream>>>(c->at<double>(c->L.loss_partial), c->at<int>(c->L.tile_begin),
                                                  c->at<i64>(c->L.row_off), c->at<float>(c->L.grad), c->gi(), c->x(),
                                                  c->lambda, c->n, (int)c->d, (int)c->L.ld, c->at<double>(c->L.eval_out));
    c->launches += 1;
    CU(cudaGetLastError());
    double out[3];
    CU(cudaMemcpyAsync(out, c->at<double>(c->L.eval_out), sizeof out, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    if (f) *f = out[0];
    if (grad_norm2) *grad_norm2 = out[1];
    if (G) *G = out[2];
    if (!std::isfinite(out[0]) || !std::isfinite(out[1]) || !std::isfinite(out[2])) return EF21_ERR_NONFINITE;
    return EF21_OK;
}

ef21_status ef21_poll(ef21_ctx* c) {
    if (!c) return EF21_ERR_INVALID_ARG;
    unsigned word = 0;
    CU(cudaMemcpyAsync(&word, c->status(), 4, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    if (word == 0) return EF21_OK;
    return word <= EF21_ERR_UNSUPPORTED ? (ef21_status)word : EF21_ERR_CUDA;
}

ef21_status ef21_set_path(ef21_ctx* c, int32_t path) {
    if (!c || path < EF21_PATH_AUTO || path > EF21_PATH_PERSISTENT) return EF21_ERR_INVALID_ARG;
    c->path = path;
    return EF21_OK;
}

ef21_status ef21_set_persistent_shape(ef21_ctx* c, int32_t cluster_blocks, int32_t rows_per_batch, int32_t row_source) {
    if (!c || cluster_blocks < 0 || cluster_blocks > 8) return EF21_ERR_INVALID_ARG;
    if (rows_per_batch != 0 && rows_per_batch != 4 && rows_per_batch != 8 && rows_per_batch != 16 && rows_per_batch != 32) return EF21_ERR_INVALID_ARG;
    if (row_source < -1 || row_source > 2) return EF21_ERR_INVALID_ARG;
    c->pk_cluster = cluster_blocks; c->pk_rb = rows_per_batch; c->pk_src = row_source;
    c->plan_valid = false; c->mb_plan_valid = false;
    return EF21_OK;
}

ef21_status ef21_set_persistent_threads(ef21_ctx* c, int32_t threads_per_block) {
    if (!c || (threads_per_block != 0 && threads_per_block != 256 && threads_per_block != 512)) return EF21_ERR_INVALID_ARG;
    c->pk_threads = threads_per_block;
    c->plan_valid = false; c->mb_plan_valid = false;
    return EF21_OK;
}

int32_t ef21_get_persistent_threads(const ef21_ctx* c) { return c ? c->pk_used_threads : 0; }

ef21_status ef21_set_persistent_body(ef21_ctx* c, int32_t body) {
    if (!c || body < 0 || body > 2) return EF21_ERR_INVALID_ARG;
    c->pk_body = body;
    c->plan_valid = false; c->mb_plan_valid = false;
    return EF21_OK;
}

int32_t ef21_get_persistent_body(const ef21_ctx* c) { return c ? c->pk_used_body : 0; }

ef21_status ef21_get_persistent_shape(const ef21_ctx* c, int32_t* cluster_blocks, int32_t* rows_per_batch, int32_t* row_source) {
    if (!c) return EF21_ERR_INVALID_ARG;
    if (cluster_blocks) *cluster_blocks = c->pk_used_cluster;
    if (rows_per_batch) *rows_per_batch = c->pk_used_rb;
    if (row_source) *row_source = c->pk_used_src;
    return EF21_OK;
}

ef21_status ef21_set_objective(ef21_ctx* c, int32_t objective) {
    if (!c || (objective != EF21_OBJECTIVE_LOGISTIC && objective != EF21_OBJECTIVE_LEAST_SQUARES)) return EF21_ERR_INVALID_ARG;
    c->objective = objective;
    return EF21_OK;
}

ef21_status ef21_set_variant(ef21_ctx* c, int32_t variant) {
    if (!c || variant < EF21_VARIANT_EF21 || variant > EF21_VARIANT_EF) return EF21_ERR_INVALID_ARG;
    c->variant = variant;
    c->plan_valid = false; c->mb_plan_valid = false;
    return EF21_OK;
}

ef21_status ef21_get_plus_choice(ef21_ctx* c, int32_t* choice_host) {
    if (!c || !choice_host) return EF21_ERR_INVALID_ARG;
    CU(cudaMemcpyAsync(choice_host, c->at<int>(c->L.plus_choice), (size_t)c->n * 4, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    return EF21_OK;
}

ef21_status ef21_set_topk_algorithm(ef21_ctx* c, int32_t algorithm) {
    if (!c || algorithm < 0 || algorithm > 1) return EF21_ERR_INVALID_ARG;
    c->force_general_topk = algorithm == 1;
    return EF21_OK;
}

ef21_status ef21_fallback_count(ef21_ctx* c, int64_t* count) {
    if (!c || !count) return EF21_ERR_INVALID_ARG;
    unsigned v = 0;
    if (c->L.tk.fast) {
        CU(cudaMemcpyAsync(&v, c->ws + c->L.topk + c->L.tk.slow_count, 4, cudaMemcpyDeviceToHost, c->stream));
        CU(cudaStreamSynchronize(c->stream));
    }
    *count = (int64_t)v;
    return EF21_OK;
}

ef21_status ef21_clear_status(ef21_ctx* c) {
    if (!c) return EF21_ERR_INVALID_ARG;
    CU(cudaMemsetAsync(c->status(), 0, 256, c->stream));
    return EF21_OK;
}

ef21_status ef21_selftest_bounded_wait(ef21_ctx* c, uint32_t spin_limit) {
    if (!c || spin_limit == 0 || spin_limit > (1u << 24)) return EF21_ERR_INVALID_ARG;
    CU(cudaMemsetAsync(c->at<unsigned long long>(c->L.slots), 0, 8, c->stream));
    bounded_wait_selftest_kernel<<<1, 1, 0, c->stream>>>(c->at<unsigned long long>(c->L.slots), c->status(), spin_limit);
    c->launches += 1;
    CU(cudaGetLastError());
    return EF21_OK;
}

ef21_status ef21_selftest_exchange_floor(ef21_ctx* c, int32_t steps) {
    if (!c || steps < 1) return EF21_ERR_INVALID_ARG;
    if (!c->shards_loaded || !c->inited) return EF21_ERR_STATE;
    if (c->variant != EF21_VARIANT_EF21) return EF21_ERR_UNSUPPORTED;
    // the shape ef21_step itself would launch, with the skeleton kernel of the same instantiation in its place
    PersistPlan P = plan_persistent(c);
    if (!P.ok) return EF21_ERR_UNSUPPORTED;
    P.kernel = P.roles ? pk_lookup_floor(P.chunks, P.rb, P.src, P.threads, P.extra)
                       : pk_lookup_wide_floor(P.chunks, P.rb, P.src, P.threads, P.extra);
    if (!P.kernel) return EF21_ERR_UNSUPPORTED;
    int dev = 0, max_smem = 0;
    CU(cudaGetDevice(&dev));
    CU(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    CU(cudaFuncSetAttribute(P.kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
    return run_persistent(c, P, steps);
}

int32_t ef21_last_path(const ef21_ctx* c) { return c ? c->last_path : 0; }
int64_t ef21_launch_count(const ef21_ctx* c) { return c ? c->launches : 0; }

}  // extern "C"
