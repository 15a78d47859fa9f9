// Local gradients of the logistic loss with nonconvex regulariser (Section 5, Eq. 19),
// launch-per-stage path: works for any shape.
//
//   grad f_i(x)_j = (1/m_i) sum_{r in shard i} rho_r a_rj + 2 lambda x_j / (1 + x_j^2)^2,
//   rho_r = -y_r / (1 + exp(y_r a_r.x)).
//
// Rows are cut into tiles that never straddle two workers.  One block handles one tile: a warp
// per row forms the margin a_r.x and the residual rho_r, then every thread owns column chunks
// and accumulates rho_r a_r over the tile's rows in ascending row order (the second sweep hits
// L1/L2).  A second kernel adds the tile partials of a worker in ascending tile order, divides
// by m_i and adds the regulariser term.  Every order is fixed, so results are reproducible.
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
        for (int r = 0; r < t.rows; ++r) {
            const float4 a = reinterpret_cast<const float4*>(A + rowid[r] * (i64)ld)[c];
            float p = rho[r];
            acc.x = fmaf(p, a.x, acc.x); acc.y = fmaf(p, a.y, acc.y);
            acc.z = fmaf(p, a.z, acc.z); acc.w = fmaf(p, a.w, acc.w);
        }
        out[c] = acc;
    }
}

// grad[i][j] = (sum over worker i's tiles of partial[tile][j]) / m_i + regulariser'(x_j); padding -> 0.
// tile_begin: [n+1] first tile of each worker; rows_of: [n] m_i.
__global__ void grad_finish_kernel(const float* __restrict__ partial, const int* __restrict__ tile_begin,
                                   const i64* __restrict__ row_off, const float* __restrict__ x,
                                   float lambda, int d, int ld, float* __restrict__ grad, int batch_rows) {
    const int i = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= ld) return;
    float out = 0.f;
    if (j < d) {
        float acc = 0.f;
        for (int t = tile_begin[i]; t < tile_begin[i + 1]; ++t) acc = __fadd_rn(acc, partial[(i64)t * ld + j]);
        const i64 m = batch_rows > 0 ? (i64)batch_rows : row_off[i + 1] - row_off[i];   // minibatch: average over its rows
        float data = m > 0 ? __fdiv_rn(acc, (float)m) : 0.f;
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
