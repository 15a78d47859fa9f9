/*
 * libef21 -- the data-parallel hot path of EF21 on one GPU, C ABI.
 *
 * EF21 (Richtarik, Sokolov, Fatkhullin, "EF21: A New, Simpler, Theoretically
 * Better, and Practically Faster Error Feedback") keeps on every worker i a
 * vector g_i and on the master their average g.  One iteration of its
 * Algorithm 2 is
 *
 *     x^{t+1}   = x^t - gamma g^t                        (master, broadcast)
 *     c_i^t     = C( grad f_i(x^{t+1}) - g_i^t )         (every worker)
 *     g_i^{t+1} = g_i^t + c_i^t                          (every worker)
 *     g^{t+1}   = g^t + (1/n) sum_i c_i^t                (master)
 *
 * with C the Top-k compressor of Section 2.1 and, for the built-in objective,
 * f_i the logistic loss with nonconvex regulariser of Section 5, Eq. 19, on
 * worker i's rows.  The n workers of the paper are n shards resident on one
 * device; "send" and "broadcast" are device buffers.
 *
 * Conventions
 *   - Every function returns an ef21_status (0 = success) and never throws or
 *     aborts.  On failure output arguments are left untouched.
 *   - Pointers named *_dev are device pointers, *_host are host pointers.
 *   - The library never allocates or frees device memory: the caller owns
 *     every device buffer, including the workspace handed to ef21_create /
 *     ef21_topk, and keeps it alive until ef21_destroy / stream completion.
 *   - All work is enqueued on the stream given at creation and is
 *     asynchronous unless stated otherwise; calls on one handle must not
 *     overlap.  Errors detected on the device (a bounded wait that expired)
 *     are reported by ef21_poll.
 *   - Vectors are fp32, indices int32, labels fp32 in {-1,+1}.
 *   - Top-k keeps the k entries of largest |v_j|, comparing the bit patterns
 *     of |v_j|; equal magnitudes go to the lower index; exactly k (index,
 *     value) pairs are produced, indices ascending, values with their sign.
 *   - State updates are single IEEE fp32 operations in a fixed order, so the
 *     results are reproducible bit for bit from run to run:
 *       v = grad - g_i;  g_i[j] += c;  s_j = ((0 + c_{i1,j}) + c_{i2,j}) + ...
 *       over ascending worker index;  g_j += s_j * (1.0f/n);  x_j = fma(-gamma, g_j, x_j).
 */
#ifndef EF21_H
#define EF21_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ef21_ctx ef21_ctx; /* opaque host-side handle */

typedef enum {
    EF21_OK = 0,
    EF21_ERR_INVALID_ARG = 1, /* null pointer, size out of range, non-finite scalar */
    EF21_ERR_STATE = 2,       /* call order violated (e.g. step before init) */
    EF21_ERR_WORKSPACE = 3,   /* workspace too small or not 256-byte aligned */
    EF21_ERR_CUDA = 4,        /* a CUDA runtime call failed */
    EF21_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired */
    EF21_ERR_NONFINITE = 6,   /* NaN/Inf met where a finite value is required */
    EF21_ERR_UNSUPPORTED = 7  /* the requested execution path cannot run this shape */
} ef21_status;

/* How ef21_init chooses g_i^0 (Algorithm 2, input line; Section 3.3 notes that the
 * theory holds for any g_i^0). */
enum {
    EF21_INIT_COMPRESSED = 0, /* g_i^0 = C(grad f_i(x^0)),  g^0 = (1/n) sum_i g_i^0 */
    EF21_INIT_ZERO = 1,       /* g_i^0 = 0,                 g^0 = 0 */
    EF21_INIT_GRADIENT = 2    /* g_i^0 = grad f_i(x^0),     g^0 = (1/n) sum_i g_i^0 */
};

/* Execution paths of ef21_step; results are bit-identical across paths given
 * bit-identical local gradients. */
enum {
    EF21_PATH_AUTO = 0,       /* pick the fastest path that supports the shape */
    EF21_PATH_LAUNCHES = 1,   /* one kernel launch per stage, any shape */
    EF21_PATH_PERSISTENT = 2  /* one cluster kernel for all steps; shards on chip */
};

/* Local objective f_i on worker i's rows (a_r, y_r); both get the regulariser lambda sum_j x_j^2/(1+x_j^2)
 * added (pass lambda = 0 for none). */
enum {
    EF21_OBJECTIVE_LOGISTIC = 0,      /* (1/m_i) sum_r log(1 + exp(-y_r a_r.x))   (Section 5, Eq. 19) */
    EF21_OBJECTIVE_LEAST_SQUARES = 1  /* (1/m_i) sum_r (a_r.x - y_r)^2            (Appendix A.2, least squares) */
};

/* Which method ef21_step / ef21_step_grads run. */
enum {
    EF21_VARIANT_EF21 = 0,      /* Algorithm 2 */
    EF21_VARIANT_EF21_PLUS = 1, /* Algorithm 3: per worker the better of C and the Markov compressor */
    EF21_VARIANT_EF = 2         /* Algorithm 4: the original error feedback method (Section 4.1) */
};

const char* ef21_status_string(ef21_status s);

/* Bytes of device workspace ef21_create needs for n workers, dimension d, k kept
 * entries and total_rows rows over all shards (0 if only supplied gradients are
 * used).  Returns 0 for invalid arguments (n < 1, d < 1, k < 1, k > d, d >= 2^31,
 * total_rows < 0). */
size_t ef21_workspace_bytes(int32_t n, int64_t d, int32_t k, int64_t total_rows);

/* Creates a handle.  workspace_dev: at least ef21_workspace_bytes(...) bytes, 256-byte
 * aligned, owned by the caller, used exclusively by this handle.  cuda_stream: a
 * cudaStream_t (NULL = default stream).  gamma > 0 and lambda >= 0 must be finite.
 * total_rows is the capacity for ef21_load_shards. */
ef21_status ef21_create(ef21_ctx** out, int32_t n, int64_t d, int32_t k, float gamma, float lambda,
                        int64_t total_rows, void* workspace_dev, size_t workspace_bytes,
                        void* cuda_stream);
void ef21_destroy(ef21_ctx* ctx); /* frees host memory only; NULL is allowed */

/* Worker i owns rows [row_offsets_host[i], row_offsets_host[i+1]) of A (row-major,
 * leading dimension d) and of y; row_offsets_host has n+1 non-decreasing entries, the
 * first 0, the last = total_rows given at creation.  A and y are copied into the
 * workspace (padded row pitch), so the caller may release them once the stream has
 * passed this call.  The _host variant takes host pointers and issues the
 * host-to-device copies itself. (Section 5: data split over n clients.) */
ef21_status ef21_load_shards(ef21_ctx* ctx, const float* A_dev, const float* y_dev,
                             const int64_t* row_offsets_host);
ef21_status ef21_load_shards_host(ef21_ctx* ctx, const float* A_host, const float* y_host,
                                  const int64_t* row_offsets_host);

/* x^0 (default: the zero vector).  d floats. */
ef21_status ef21_set_x(ef21_ctx* ctx, const float* x0_dev);

/* Algorithm 2, input line: builds g_i^0 and g^0 from the local gradients at x^0
 * (mode: EF21_INIT_*).  Modes 0 and 2 need shards; mode 1 does not. */
ef21_status ef21_init(ef21_ctx* ctx, int32_t mode);
/* The same with caller-supplied local gradients V_dev[n][d] (leading dimension d). */
ef21_status ef21_init_grads(ef21_ctx* ctx, const float* V_dev, int32_t mode);

/* `steps` iterations of Algorithm 2's loop (x update, local gradients of Eq. 19,
 * difference, Top-k, g_i update, aggregation).  After init and t steps in total the
 * state is (x^t, g^t, g_i^t) in the paper's indexing.
 * On the launch-per-stage path with d <= 8,192 and steps >= 3, the iterations after the first are
 * replayed as a CUDA graph that the handle captures once (on a stream of its own; the CUDA runtime
 * keeps the graph's resources until ef21_destroy) and launches into the handle's stream; if that
 * stream is itself being captured, or the capture fails, the kernels are launched one by one.
 * Results are identical either way.
 * On the persistent path one launch holds all of its thread-block clusters on the device at once.  Launches
 * of several handles are therefore kept from overlapping: a persistent launch on another stream than the
 * device's previous one is ordered (on the device, by an event; the host does not wait) after everything
 * that stream holds so far.  The device meant is the one current at ef21_create; keep it current for the
 * handle's calls. */
ef21_status ef21_step(ef21_ctx* ctx, int32_t steps);
/* The same loop with grad f_i replaced by the caller's V_dev[n][d], re-used unchanged at
 * each of the `steps` iterations (the static input sequence of Section 3.1); call with
 * steps = 1 and fresh V for a changing sequence.  V must stay valid until the stream has
 * passed this call.  With steps > 1 on long vectors the library orders part of the work on a second
 * stream of its own (created on first use, joined back into the handle's stream before the call's
 * work ends), so a later operation on the handle's stream still sees the complete result. */
ef21_status ef21_step_grads(ef21_ctx* ctx, const float* V_dev, int32_t steps);

/* `steps` iterations of the stochastic variant (Appendix, Algorithm 5): the loop of Algorithm 2 with
 * grad f_i(x^{t+1}) replaced by the minibatch estimate over tau rows of worker i's shard, averaged over tau,
 * plus the regulariser term.  batches_dev[steps][n][tau] holds, for every iteration and worker, the row
 * numbers inside the shard (int32; the caller draws them, e.g. without replacement); it must stay valid until
 * the stream has passed the call.  Every shard needs at least tau rows.  An index outside its shard is
 * replaced by row 0 and EF21_ERR_INVALID_ARG is recorded in the status word (ef21_poll).  EF21_VARIANT_EF21
 * only.  Shapes the persistent path takes (d <= 512, k <= 8) run all iterations in one launch, the sampled rows
 * read from global memory each iteration; others run launch by launch.  ef21_step_minibatch is the same call
 * for one iteration. */
ef21_status ef21_step_minibatches(ef21_ctx* ctx, const int32_t* batches_dev, int32_t tau, int32_t steps);
ef21_status ef21_step_minibatch(ef21_ctx* ctx, const int32_t* batch_dev, int32_t tau);

/* `steps` iterations of Algorithm 2 with the scaled Rand-k compressor in place of Top-k (Appendix, Lemma 8 and
 * Example 2: Rand-k, which keeps k uniformly drawn coordinates times d/k, scaled by 1/(1 + omega) = k/d -- the
 * factors cancel, the compressor keeps the drawn entries as they are and lies in B(k/d)).  The library draws
 * nothing: sets_dev[steps][n][k] holds, for every iteration and worker, the k drawn coordinates, distinct and in
 * ascending order (int32); an entry outside [0, d) or out of order is replaced and EF21_ERR_INVALID_ARG is
 * recorded in the status word.  V_dev[n][d], if not NULL, stands for the local gradients at every iteration (as in
 * ef21_step_grads); otherwise the gradients of the objective on the loaded shards are used.  Launch path;
 * EF21_VARIANT_EF21 only.  Given the same gradients the result is bit-identical to the plain definition. */
ef21_status ef21_step_randk(ef21_ctx* ctx, const float* V_dev, const int32_t* sets_dev, int32_t steps);

/* grad f_i(x) for the current x and all workers, written to grads_out_dev[n][d]
 * (Eq. 19 differentiated; state is not changed). */
ef21_status ef21_local_grads(ef21_ctx* ctx, float* grads_out_dev);

/* Standalone Top-k compressor (Section 2.1) on `batch` vectors v_dev[batch][d] (leading
 * dimension d): idx_out_dev[batch][k] ascending, val_out_dev[batch][k].  The workspace
 * needs ef21_topk_workspace_bytes(batch, d, k) bytes, 256-byte aligned. */
size_t ef21_topk_workspace_bytes(int32_t batch, int64_t d, int32_t k);
ef21_status ef21_topk(const float* v_dev, int32_t batch, int64_t d, int32_t k,
                      int32_t* idx_out_dev, float* val_out_dev,
                      void* workspace_dev, size_t workspace_bytes, void* cuda_stream);

/* Top-k for callers that cannot hand over or allocate device scratch.  (The paper has no
 * counterpart: this is a packaging variant of ef21_topk, same result bit for bit.)
 *
 * Who needs it: code that runs where the CUDA allocator is off limits -- a host thread that may
 * not block on the implicit synchronisation of cudaMalloc/cudaFree, a plug-in inside a framework
 * that owns all device memory and hands out none, a process whose memory was carved up at start
 * and must not grow.  Such a caller passes only its input and the two output arrays; the
 * scratch is a fixed 1 MiB array inside the library image (every GPU that loads the library
 * holds it until the process exits).  The function calls no cudaMalloc, cudaFree or allocating
 * library routine.
 *
 * Limits: batch <= 64 and batch * ceil(d / 4096) <= 16384 (e.g. 64 vectors of 2^20 entries, or
 * one of 2^26); beyond that the call returns EF21_ERR_UNSUPPORTED and does nothing.  Vectors
 * of up to 8,192 entries take the one-launch kernel (which needs no scratch), longer ones the
 * multi-pass radix select.
 * The first call on a device looks up the device address of the scratch array
 * (cudaGetSymbolAddress, with that device current) and caches it; make that first call outside
 * of any stream capture.
 * All calls in a process share the one scratch array, which keeps the previous call's contents:
 * every call clears what it needs at zero on the stream before use.  Two calls whose kernels can
 * overlap on the GPU (different streams without an ordering between them) race on it; order
 * them.  Arguments as for ef21_topk. */
ef21_status ef21_topk_static(const float* v_dev, int32_t batch, int64_t d, int32_t k,
                             int32_t* idx_out_dev, float* val_out_dev, void* cuda_stream);

/* Copies of the state; any pointer may be NULL.  gi is [n][d]; last_idx/last_val are the
 * most recent messages c_i, [n][k] each.  set_state also marks the handle initialised
 * (resume / teacher forcing); x, g or gi left NULL keep their current contents. */
ef21_status ef21_get_state(ef21_ctx* ctx, float* x_dev, float* g_dev, float* gi_dev,
                           int32_t* last_idx_dev, float* last_val_dev);
ef21_status ef21_get_state_host(ef21_ctx* ctx, float* x_host, float* g_host, float* gi_host,
                                int32_t* last_idx_host, float* last_val_host); /* synchronises */
ef21_status ef21_set_state(ef21_ctx* ctx, const float* x_dev, const float* g_dev, const float* gi_dev);

/* Diagnostics at the current state (synchronises): f(x) of Eq. 19 / Eq. 1, ||grad f(x)||^2,
 * and G^t = (1/n) sum_i ||g_i - grad f_i(x)||^2 of Section 3.3.  Any pointer may be NULL.  If one of
 * the three is NaN or Inf the values are still written and EF21_ERR_NONFINITE is returned. */
ef21_status ef21_eval(ef21_ctx* ctx, double* f, double* grad_norm2, double* G);

/* Synchronises the stream and returns the device status word: EF21_OK, or the first
 * error a kernel recorded, or EF21_ERR_CUDA.
 *   EF21_ERR_NONFINITE: a compressor of this handle (init, step, step_grads, step_minibatch, any
 *     method) selected a NaN or Inf.  The compressor of Section 2.1 is defined on real vectors; a
 *     non-finite entry has the largest key (bit-pattern order), so it is always selected and one
 *     anywhere in a compressed vector -- a supplied gradient, or a gradient at a non-finite x -- is
 *     noticed in the step that meets it.  The state is unspecified from that step on: restore it with
 *     ef21_set_state and call ef21_clear_status.  The standalone ef21_topk has no status word and does
 *     not check.
 *   EF21_ERR_TIMEOUT: a bounded wait of the persistent kernel expired (its clusters were not all
 *     running at once, e.g. another kernel of the process held SMs).  The blocks leave the iteration
 *     loop at different iterations, so the state (x, g, g_i, last messages) is unspecified afterwards:
 *     restore it with ef21_set_state, call ef21_clear_status, and use EF21_PATH_LAUNCHES if the
 *     device stays shared.
 *   EF21_ERR_INVALID_ARG: ef21_step_minibatch met a row number outside its shard. */
ef21_status ef21_poll(ef21_ctx* ctx);

/* Selects the local objective (EF21_OBJECTIVE_*) used by ef21_init, ef21_step, ef21_local_grads and
 * ef21_eval; default logistic.  Both execution paths support both objectives. */
ef21_status ef21_set_objective(ef21_ctx* ctx, int32_t objective);

/* Selects the method (EF21_VARIANT_*) that ef21_step / ef21_step_grads run; default Algorithm 2.
 *
 * EF21+ (Section 3.4, Algorithm 3).  With EF21_VARIANT_EF21_PLUS every step computes, per worker,
 * b_i = C(grad f_i(x)) and m_i = g_i + C(grad f_i(x) - g_i), the distortions B_i = ||b_i - grad f_i(x)||^2
 * and M_i = ||m_i - grad f_i(x)||^2 (fp64 sums of the fp32 vectors), sets g_i = m_i if M_i <= B_i and
 * g_i = b_i otherwise, and recomputes g = (1/n) sum_i g_i (ascending i, then one multiply).  Both
 * execution paths run it; the persistent kernel needs n * d * 4 <= 64 KB (every block keeps a copy
 * of all g_i), otherwise the launch path is taken.  The "last message" of ef21_get_state is the
 * compressed vector that was used.  Initialisation is that of Algorithm 2.
 *
 * The original error feedback method, EF (Section 4.1, Algorithm 4), with EF21_VARIANT_EF.  The
 * per-worker state is the error e_i, kept where Algorithm 2 keeps g_i (the gi argument of
 * ef21_get_state / ef21_set_state); g is not used.  Algorithm 4 starts from e_i^0 = 0: call
 * ef21_init(ctx, EF21_INIT_ZERO).  One step from (x^t, e_i^t) computes
 *     w_i^t = C(e_i^t + gamma grad f_i(x^t)),   x^{t+1} = x^t - (1/n) sum_i w_i^t,
 *     e_i^{t+1} = e_i^t + gamma grad f_i(x^t) - w_i^t
 * so after t steps the state is Algorithm 4's (x^t, e_i^t); the algorithm's own loop forms w_i^{t+1}
 * at the end of iteration t, here it is formed at the start of the next step from the same x^{t+1}
 * and e_i^{t+1}.  The "last message" of ef21_get_state is w_i^{t-1}.  gamma * grad, the sum with
 * e_i, the difference with w_i, the factor 1/n and the update of x are single rounded fp32
 * operations; the sum over workers runs in ascending worker order.  ef21_step_grads uses the
 * supplied vectors in place of grad f_i.  Both execution paths run ef21_step; ef21_step_minibatch
 * is not available. */
ef21_status ef21_set_variant(ef21_ctx* ctx, int32_t variant);
/* choice_host[n]: 0 where the last EF21+ step kept the Markov compressor, 1 where it took C(grad);
 * synchronises. */
ef21_status ef21_get_plus_choice(ef21_ctx* ctx, int32_t* choice_host);

/* Top-k algorithm used inside the EF21 rounds of the launch path: 0 = automatic (long vectors,
 * d >= 2^18 and k <= 6144, take the one-pass path: sampled threshold, single streaming pass,
 * exact selection among the candidates; everything else takes the multi-pass radix select),
 * 1 = always the multi-pass radix select.  Both give the same bits. */
ef21_status ef21_set_topk_algorithm(ef21_ctx* ctx, int32_t algorithm);
/* Number of vectors, since creation, for which the one-pass Top-k had to fall back to the exact
 * selection over the whole vector (threshold missed or too many ties); synchronises. */
ef21_status ef21_fallback_count(ef21_ctx* ctx, int64_t* count);

/* Clears the device status word (after an error has been read with ef21_poll). */
ef21_status ef21_clear_status(ef21_ctx* ctx);

/* Self-check of the bounded device-side wait used by the persistent path: one thread spins
 * at most spin_limit (1 .. 2^24) times on a word that nothing writes, then records
 * EF21_ERR_TIMEOUT, which the next ef21_poll returns.  The device and the context stay usable. */
ef21_status ef21_selftest_bounded_wait(ef21_ctx* ctx, uint32_t spin_limit);

/* Measuring aid: `steps` iterations of the persistent path's exchange skeleton for this handle's shape -- the
 * same clusters, barriers, hand-off of the block partials to the cluster leader, publication and polling
 * of the n*k message words, every wait bounded as in ef21_step -- with all arithmetic of the method left
 * out (no row sweep, no selection, no aggregation).  The state is not touched.  Timing it gives the cost
 * of the two dependencies Algorithm 2 has per iteration (broadcast of x^{t+1}, collection of the c_i^t) on
 * this device, a floor under the iteration time of ef21_step.  EF21_ERR_UNSUPPORTED if the shape has no
 * persistent path. */
ef21_status ef21_selftest_exchange_floor(ef21_ctx* ctx, int32_t steps);

/* Tuning of the persistent path (Algorithm 2 as one kernel; worker i = one thread-block
 * cluster): blocks per cluster (1..8, 0 = automatic), rows per warp batch (4, 8, 16, 32, 0 =
 * automatic) and where the shard rows live (0 registers, 1 shared memory, 2 global memory /
 * L2, -1 = automatic; get_ also reports 3 = global memory through the sampled row numbers of
 * ef21_step_minibatches).  A shape that cannot run makes ef21_step fall back (path AUTO) or
 * return EF21_ERR_UNSUPPORTED (path PERSISTENT).  get_ reports what the last persistent
 * launch used. */
ef21_status ef21_set_persistent_shape(ef21_ctx* ctx, int32_t cluster_blocks, int32_t rows_per_batch,
                                      int32_t row_source);
ef21_status ef21_get_persistent_shape(const ef21_ctx* ctx, int32_t* cluster_blocks,
                                      int32_t* rows_per_batch, int32_t* row_source);

/* Threads per block of the persistent path: 256, 512 or 0 = automatic (512 exists only for batches
 * of at most 16 float4 registers per lane).  get_ reports what the last persistent launch used. */
ef21_status ef21_set_persistent_threads(ef21_ctx* ctx, int32_t threads_per_block);
int32_t ef21_get_persistent_threads(const ef21_ctx* ctx);

/* Body of the persistent kernel: 0 = automatic, 1 = one warp of every block serves it (adds the warps' partials,
 * and in the leader forms the gradient, selects by warp arg-max rounds; every block's serving warp gathers the
 * messages and updates g and x) while the other warps only sweep rows and never meet a block-wide barrier;
 * k <= 8, Algorithms 2 and 4.  2 = every step is taken by the whole block between block barriers (any k <= 32;
 * the only body of Algorithm 3).  Both give the same bits.  A forced body that cannot run the shape behaves as
 * in ef21_set_persistent_shape.  get_ reports what the last persistent launch used. */
ef21_status ef21_set_persistent_body(ef21_ctx* ctx, int32_t body);
int32_t ef21_get_persistent_body(const ef21_ctx* ctx);

/* Forces an execution path (EF21_PATH_*) for later ef21_step calls. */
ef21_status ef21_set_path(ef21_ctx* ctx, int32_t path);
/* The path the last ef21_step / ef21_step_grads actually used (EF21_PATH_*), 0 if none yet. */
int32_t ef21_last_path(const ef21_ctx* ctx);
/* Kernel launches enqueued by this handle since creation (copies are not counted). */
int64_t ef21_launch_count(const ef21_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* EF21_H */
