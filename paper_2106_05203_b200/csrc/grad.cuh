// Local gradients of the logistic loss with nonconvex regulariser (Section 5, Eq. 19),
// launch-per-stage path: works for any shape.
//
//   grad f_i(x)_j = (1/m_i) sum_{r in shard i} rho_r a_rj + 2 lambda x_j / (1 + x_j^2)^2,
//   rho_r = -y_r / (1 + exp(y_r a_r.x)).
//
// Rows are cut into tiles that never straddle two workers; one block handles one tile and leaves the
// tile's partial sum of rho_r a_r.  Rows of up to 1,024 columns go through grad_stream_kernel (one
// read of every row, rows held in registers between the margin and the accumulation); wider rows
// through grad_tiles_kernel: a warp per row forms the margin a_r.x and the residual rho_r, then
// every thread owns column chunks and accumulates rho_r a_r over the tile's rows in ascending row
// order (the second sweep hits L1/L2).  A second kernel adds the tile partials of a worker in a
// fixed order, divides by m_i and adds the regulariser term.  Every order is fixed, so results
// are reproducible.
#pragma once
#include "common.cuh"

namespace ef21 {

struct RowTile {
    i64 row0;      // first row (global row index)
    int rows;      // rows in this tile
    int worker;    // owner
};

constexpr int GRAD_TILE_MAX_ROWS = 256;
constexpr int GRAD_BLOCK = 256;

// A: [N][ld] (ld % 4 == 0, padding columns are zero), x: [ld] (padding zero).
// partial: [num_tiles][ld].  loss_partial (optional): [num_tiles] doubles, sum of the per-row losses
// over the tile's rows.
// gather (optional): minibatch mode.  A tile then covers positions [row0, row0 + rows) of its worker's
// index list gather[worker * gather_pitch + ...]; each entry is a row number inside the worker's shard.
// An entry outside the shard records EF21_ERR_INVALID_ARG in the status word and is replaced by row 0.
__global__ void __launch_bounds__(GRAD_BLOCK)
grad_tiles_kernel(const float* __restrict__ A, const float* __restrict__ y, const float* __restrict__ x,
                  const RowTile* __restrict__ tiles, int ld, int objective, float* __restrict__ partial,
                  double* __restrict__ loss_partial, const int* __restrict__ gather, int gather_pitch,
                  const i64* __restrict__ row_off, unsigned* __restrict__ status) {
    __shared__ float rho[GRAD_TILE_MAX_ROWS];
    __shared__ i64 rowid[GRAD_TILE_MAX_ROWS];
    __shared__ double loss_w[GRAD_BLOCK / 32];
    const RowTile t = tiles[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = GRAD_BLOCK / 32;
    const int chunks = ld >> 2;
    for (int r = threadIdx.x; r < t.rows; r += GRAD_BLOCK) {
        i64 row = t.row0 + r;
        if (gather) {
            const i64 lo = row_off[t.worker], m = row_off[t.worker + 1] - lo;
            i64 pick = gather[(i64)t.worker * gather_pitch + t.row0 + r];
            if (pick < 0 || pick >= m) { record_error(status, 1u /* EF21_ERR_INVALID_ARG */); pick = 0; }
            row = lo + pick;
        }
        rowid[r] = row;
    }
    __syncthreads();
    const float4* __restrict__ x4 = reinterpret_cast<const float4*>(x);
    double loss_acc = 0.0;
    for (int r = warp; r < t.rows; r += nwarps) {
        const float4* __restrict__ row = reinterpret_cast<const float4*>(A + rowid[r] * (i64)ld);
        float z = 0.f;
        for (int c = lane; c < chunks; c += 32) {
            float4 a = row[c];
            float4 xv = __ldg(x4 + c);
            z = fmaf(a.x, xv.x, z); z = fmaf(a.y, xv.y, z); z = fmaf(a.z, xv.z, z); z = fmaf(a.w, xv.w, z);
        }
        z = warp_sum(z);
        if (lane == 0) {
            float yr = y[rowid[r]];
            rho[r] = loss_residual(objective, yr, z);
            if (loss_partial) {
                if (objective == 0) {
                    double u = -(double)yr * (double)z;
                    loss_acc += (u > 0.0 ? u : 0.0) + log1p(exp(-fabs(u)));
                } else {
                    double e = (double)z - (double)yr;
                    loss_acc += e * e;
                }
            }
        }
    }
    if (loss_partial) {
        if (lane == 0) loss_w[warp] = loss_acc;
    }
    __syncthreads();
    if (loss_partial && threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < nwarps; ++w) s += loss_w[w];
        loss_partial[blockIdx.x] = s;
    }
    float4* __restrict__ out = reinterpret_cast<float4*>(partial + (i64)blockIdx.x * ld);
    for (int c = threadIdx.x; c < chunks; c += GRAD_BLOCK) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int r = 0; r < t.rows; ++r) {
            const float4 a = reinterpret_cast<const float4*>(A + rowid[r] * (i64)ld)[c];
            float p = rho[r];
            acc.x = fmaf(p, a.x, acc.x); acc.y = fmaf(p, a.y, acc.y);
            acc.z = fmaf(p, a.z, acc.z); acc.w = fmaf(p, a.w, acc.w);
        }
        out[c] = acc;
    }
}

// The same tile partials for rows of up to 1,024 columns, from ONE read of every row: a warp takes RB rows
// at a time into registers (CHUNKS float4 per lane and row), forms the RB margins by a transposed warp
// reduction, the residuals, and adds rho_r a_r from the registers into its own accumulator; the warps'
// accumulators are added in ascending warp order.  RB * CHUNKS * 16 bytes per lane are in flight per warp,
// which is what keeps HBM busy when the shards do not fit in L2.
constexpr int GRAD_STREAM_BLOCK = 256;

template <int CHUNKS, int RB>
__global__ void __launch_bounds__(GRAD_STREAM_BLOCK)
grad_stream_kernel(const float* __restrict__ A, const float* __restrict__ y, const float* __restrict__ x,
                   const RowTile* __restrict__ tiles, int ld, int objective, float* __restrict__ partial,
                   double* __restrict__ loss_partial, const int* __restrict__ gather, int gather_pitch,
                   const i64* __restrict__ row_off, unsigned* __restrict__ status) {
    constexpr int SH = (RB == 32) ? 0 : (RB == 16 ? 1 : (RB == 8 ? 2 : (RB == 4 ? 3 : 4)));    // log2(32/RB)
    constexpr int WARPS = GRAD_STREAM_BLOCK / 32;
    static_assert(RB == 2 || RB == 4 || RB == 8 || RB == 16, "RB");
    static_assert(RB * CHUNKS <= 16, "register budget");
    extern __shared__ __align__(16) unsigned char grad_smem[];
    float* red = reinterpret_cast<float*>(grad_smem);                       // [WARPS][ld]
    __shared__ i64 rowid[GRAD_TILE_MAX_ROWS];
    __shared__ double loss_w[WARPS];
    const RowTile t = tiles[blockIdx.x];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunks = ld >> 2;
    for (int r = tid; r < t.rows; r += GRAD_STREAM_BLOCK) {
        i64 row = t.row0 + r;
        if (gather) {
            const i64 lo = row_off[t.worker], m = row_off[t.worker + 1] - lo;
            i64 pick = gather[(i64)t.worker * gather_pitch + t.row0 + r];
            if (pick < 0 || pick >= m) { record_error(status, 1u /* EF21_ERR_INVALID_ARG */); pick = 0; }
            row = lo + pick;
        }
        rowid[r] = row;
    }
    __syncthreads();
    float4 xr[CHUNKS], acc[CHUNKS];
#pragma unroll
    for (int cs = 0; cs < CHUNKS; ++cs) {
        const int c = lane + 32 * cs;
        xr[cs] = c < chunks ? __ldg(reinterpret_cast<const float4*>(x) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        acc[cs] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    double loss_acc = 0.0;
    const int nbatch = (t.rows + RB - 1) / RB;
    for (int b = warp; b < nbatch; b += WARPS) {
        const int rb0 = b * RB;
        float4 a[RB][CHUNKS];
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const int row = rb0 + r;
            const float4* __restrict__ src = reinterpret_cast<const float4*>(A + (row < t.rows ? rowid[row] : 0) * (i64)ld);
#pragma unroll
            for (int cs = 0; cs < CHUNKS; ++cs) {
                const int c = lane + 32 * cs;
                a[r][cs] = (row < t.rows && c < chunks) ? __ldg(src + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        const int myrow = rb0 + (lane >> SH);                 // the row whose margin this lane ends up with
        const bool mine = myrow < t.rows;
        const float yr = mine ? __ldg(y + rowid[myrow]) : 0.f;
        float pd[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            float z = 0.f;
#pragma unroll
            for (int cs = 0; cs < CHUNKS; ++cs) z = dot4(a[r][cs], xr[cs], z);
            pd[r] = z;
        }
        const float z = reduce_rows<RB>(pd, lane);
        const float rho = loss_residual(objective, yr, z);        // 0 for a row past the end (y = 0, a = 0)
        if (loss_partial && mine && (lane & ((1 << SH) - 1)) == 0) {
            if (objective == 0) {
                const double u = -(double)yr * (double)z;
                loss_acc += (u > 0.0 ? u : 0.0) + log1p(exp(-fabs(u)));
            } else {
                const double e = (double)z - (double)yr;
                loss_acc += e * e;
            }
        }
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const float pr = __shfl_sync(0xffffffffu, rho, r << SH);
#pragma unroll
            for (int cs = 0; cs < CHUNKS; ++cs) acc[cs] = fma4(pr, a[r][cs], acc[cs]);
        }
    }
#pragma unroll
    for (int cs = 0; cs < CHUNKS; ++cs) {
        const int c = lane + 32 * cs;
        if (c < chunks) reinterpret_cast<float4*>(red + warp * ld)[c] = acc[cs];
    }
    if (loss_partial) {
        loss_acc = warp_sum(loss_acc);
        if (lane == 0) loss_w[warp] = loss_acc;
    }
    __syncthreads();
    if (loss_partial && tid == 0) {
        double s = 0.0;
        for (int w = 0; w < WARPS; ++w) s += loss_w[w];
        loss_partial[blockIdx.x] = s;
    }
    float4* __restrict__ out = reinterpret_cast<float4*>(partial + (i64)blockIdx.x * ld);
    for (int c = tid; c < chunks; c += GRAD_STREAM_BLOCK) {
        float4 sum = reinterpret_cast<const float4*>(red)[c];
#pragma unroll
        for (int w = 1; w < WARPS; ++w) {
            const float4 o = reinterpret_cast<const float4*>(red + w * ld)[c];
            sum.x = __fadd_rn(sum.x, o.x); sum.y = __fadd_rn(sum.y, o.y);
            sum.z = __fadd_rn(sum.z, o.z); sum.w = __fadd_rn(sum.w, o.w);
        }
        out[c] = sum;
    }
}

// grad[i][j] = (sum over worker i's tiles of partial[tile][j]) / m_i + regulariser'(x_j); padding -> 0.
// tile_begin: [n+1] first tile of each worker.  A block covers GRAD_FINISH_COLS columns of one worker with
// GRAD_FINISH_LANES threads per column: thread q adds the tiles q, q + LANES, ... in ascending order, then
// the LANES sums of a column are added in ascending q (a fixed order, so results are reproducible).
constexpr int GRAD_FINISH_COLS = 32;
constexpr int GRAD_FINISH_LANES = 8;

__global__ void __launch_bounds__(GRAD_FINISH_COLS * GRAD_FINISH_LANES)
grad_finish_kernel(const float* __restrict__ partial, const int* __restrict__ tile_begin,
                   const i64* __restrict__ row_off, const float* __restrict__ x,
                   float lambda, int d, int ld, float* __restrict__ grad, int batch_rows) {
    __shared__ float part[GRAD_FINISH_LANES][GRAD_FINISH_COLS];
    const int i = blockIdx.y;
    const int col = threadIdx.x % GRAD_FINISH_COLS, q = threadIdx.x / GRAD_FINISH_COLS;
    const int j = blockIdx.x * GRAD_FINISH_COLS + col;
    float acc = 0.f;
    if (j < d) {
        const int t1 = tile_begin[i + 1];
#pragma unroll 4
        for (int t = tile_begin[i] + q; t < t1; t += GRAD_FINISH_LANES) acc = __fadd_rn(acc, partial[(i64)t * ld + j]);
    }
    part[q][col] = acc;
    __syncthreads();
    if (q != 0 || j >= ld) return;
    float out = 0.f;
    if (j < d) {
        float sum = part[0][col];
#pragma unroll
        for (int w = 1; w < GRAD_FINISH_LANES; ++w) sum = __fadd_rn(sum, part[w][col]);
        const i64 m = batch_rows > 0 ? (i64)batch_rows : row_off[i + 1] - row_off[i];   // minibatch: average over its rows
        const float data = m > 0 ? __fdiv_rn(sum, (float)m) : 0.f;
        out = __fadd_rn(data, regulariser_grad(lambda, x[j]));
    }
    grad[(i64)i * ld + j] = out;
}

// Copies A[N][d] into the padded layout Ap[N][ld], zero-filling the padding columns.
__global__ void pad_rows_kernel(const float* __restrict__ A, i64 N, int d, int ld, float* __restrict__ Ap) {
    const i64 total = N * (i64)ld;
    for (i64 e = blockIdx.x * (i64)blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
        const i64 r = e / ld;
        const int c = (int)(e - r * ld);
        Ap[e] = c < d ? A[r * (i64)d + c] : 0.f;
    }
}

// Diagnostics: f(x), ||grad f(x)||^2, G = (1/n) sum_i ||g_i - grad_i||^2, in fp64, one block.
// out[0] = f, out[1] = ||grad f||^2, out[2] = G.
__global__ void __launch_bounds__(1024)
eval_reduce_kernel(const double* __restrict__ loss_partial, const int* __restrict__ tile_begin,
                   const i64* __restrict__ row_off, const float* __restrict__ grad,
                   const float* __restrict__ gi, const float* __restrict__ x, float lambda,
                   int n, int d, int ld, double* __restrict__ out) {
    __shared__ double red[3][32];
    double f = 0.0, nrm = 0.0, G = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        double s = 0.0;
        for (int t = tile_begin[i]; t < tile_begin[i + 1]; ++t) s += loss_partial[t];
        const i64 m = row_off[i + 1] - row_off[i];
        if (m > 0) f += s / (double)m;
    }
    f /= (double)n;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        double xj = (double)x[j];
        f += (double)lambda * xj * xj / (1.0 + xj * xj);
        double s = 0.0;
        for (int i = 0; i < n; ++i) {
            double gr = (double)grad[(i64)i * ld + j];
            s += gr;
            double e = (double)gi[(i64)i * ld + j] - gr;
            G += e * e;
        }
        s /= (double)n;
        nrm += s * s;
    }
    G /= (double)n;
    f = warp_sum(f); nrm = warp_sum(nrm); G = warp_sum(G);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { red[0][warp] = f; red[1][warp] = nrm; red[2][warp] = G; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0, c = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { a += red[0][w]; b += red[1][w]; c += red[2][w]; }
        out[0] = a; out[1] = b; out[2] = c;
    }
}

}  // namespace ef21
