// QR orthonormalisation for Power(A, Q) = qr(A Q).Q (Sec. 3.2 of the paper), fp64, in place.
//
// The factorisation wanted is the unique one with a positive diagonal of R.  It is computed by
// a right-looking block Gram-Schmidt: for each panel of kPanel columns
//   1. orthonormalise the panel by Cholesky-QR applied twice (Gram matrix -> Cholesky factor
//      -> multiply by its inverse); the Cholesky factor has a positive diagonal, so the signs
//      come out as required;
//   2. project the panel out of all trailing columns: C = P^T A_trail, A_trail -= P C.
// In fp64 the loss of orthogonality of this scheme is ~ cond * 1e-16, far below the fp32
// rounding of the stored bases, and the result agrees with Householder QR to the same level.
// Reductions are done in a fixed order (per-chunk partial sums, then a serial sum), so the
// result is bit-reproducible from run to run.
#include "br_internal.h"

namespace br {
namespace {

constexpr int kPanel = 32;      // panel width
constexpr int kRows = 128;      // rows per CTA in the panel kernels
constexpr int kProjCols = 64;   // columns per CTA in the projection kernel
constexpr int kProjSplit = 8;   // row chunks (split of the contraction) in the projection

// S_c = P_c^T P_c for the row chunk c of the panel P = A[:, j0:j0+bw].
__global__ void __launch_bounds__(256)
k_panel_gram(const double* __restrict__ A, int64_t k, int64_t j0, int bw, double* __restrict__ partial) {
  __shared__ double Ps[kRows][kPanel + 1];
  const int64_t r0 = (int64_t)blockIdx.x * kRows;
  for (int idx = threadIdx.x; idx < kRows * kPanel; idx += 256) {
    int r = idx / kPanel, c = idx % kPanel;
    double v = 0.0;
    if (r0 + r < k && c < bw) v = A[(r0 + r) * k + j0 + c];
    Ps[r][c] = v;
  }
  __syncthreads();
  // 1024 outputs, 4 per thread
  for (int o = threadIdx.x; o < kPanel * kPanel; o += 256) {
    int i = o / kPanel, j = o % kPanel;
    double s = 0.0;
#pragma unroll 8
    for (int r = 0; r < kRows; ++r) s = fma(Ps[r][i], Ps[r][j], s);
    partial[(int64_t)blockIdx.x * kPanel * kPanel + o] = s;
  }
}

// Sum the partial Gram matrices in chunk order, Cholesky-factor S = R^T R, write R^{-1}.
__global__ void __launch_bounds__(256)
k_panel_chol(const double* __restrict__ partial, int nchunks, int bw, double* __restrict__ Rinv,
             int* __restrict__ status) {
  __shared__ double S[kPanel][kPanel + 1];
  __shared__ double Ri[kPanel][kPanel + 1];
  __shared__ double diag0[kPanel];
  for (int o = threadIdx.x; o < kPanel * kPanel; o += 256) {
    double s = 0.0;
    for (int c = 0; c < nchunks; ++c) s += partial[(int64_t)c * kPanel * kPanel + o];
    S[o / kPanel][o % kPanel] = s;
  }
  __syncthreads();
  if (threadIdx.x < kPanel) diag0[threadIdx.x] = S[threadIdx.x][threadIdx.x];
  __syncthreads();
  for (int c = 0; c < bw; ++c) {
    if (threadIdx.x == 0) {
      double piv = S[c][c];
      // a pivot below (1e-12)^2 of the column's squared norm: numerically rank deficient
      double floor_ = diag0[c] * 1e-24;
      if (!(floor_ > 1e-300)) floor_ = 1e-300;
      if (!(piv > floor_)) {
        piv = floor_;
        atomicMax(status, (int)BR_WARN_RANK_DEFICIENT);
      }
      S[c][c] = sqrt(piv);
    }
    __syncthreads();
    const double d = S[c][c];
    for (int j = c + 1 + threadIdx.x; j < bw; j += 256) S[c][j] /= d;
    __syncthreads();
    const int rem = bw - c - 1;
    for (int o = threadIdx.x; o < rem * rem; o += 256) {
      int i = c + 1 + o / rem, j = c + 1 + o % rem;
      if (j >= i) S[i][j] -= S[c][i] * S[c][j];
    }
    __syncthreads();
  }
  // invert the upper-triangular R (stored in the upper part of S): one column per thread
  if (threadIdx.x < kPanel) {
    const int j = threadIdx.x;
    for (int i = 0; i < kPanel; ++i) Ri[i][j] = 0.0;
    if (j < bw) {
      Ri[j][j] = 1.0 / S[j][j];
      for (int i = j - 1; i >= 0; --i) {
        double s = 0.0;
        for (int l = i + 1; l <= j; ++l) s = fma(S[i][l], Ri[l][j], s);
        Ri[i][j] = -s / S[i][i];
      }
    }
  }
  __syncthreads();
  for (int o = threadIdx.x; o < kPanel * kPanel; o += 256) Rinv[o] = Ri[o / kPanel][o % kPanel];
}

// P <- P R^{-1}
__global__ void __launch_bounds__(256)
k_panel_apply(double* __restrict__ A, int64_t k, int64_t j0, int bw, const double* __restrict__ Rinv) {
  __shared__ double Ps[kRows][kPanel + 1];
  __shared__ double Ri[kPanel][kPanel + 1];
  const int64_t r0 = (int64_t)blockIdx.x * kRows;
  for (int idx = threadIdx.x; idx < kPanel * kPanel; idx += 256) Ri[idx / kPanel][idx % kPanel] = Rinv[idx];
  for (int idx = threadIdx.x; idx < kRows * kPanel; idx += 256) {
    int r = idx / kPanel, c = idx % kPanel;
    double v = 0.0;
    if (r0 + r < k && c < bw) v = A[(r0 + r) * k + j0 + c];
    Ps[r][c] = v;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < kRows * kPanel; idx += 256) {
    int r = idx / kPanel, c = idx % kPanel;
    if (r0 + r >= k || c >= bw) continue;
    double s = 0.0;
    for (int i = 0; i <= c; ++i) s = fma(Ps[r][i], Ri[i][c], s);
    A[(r0 + r) * k + j0 + c] = s;
  }
}

// partial[z][i][j] = sum over the row chunk z of P[r][i] * T[r][j], T = A[:, jt0 + j].
__global__ void __launch_bounds__(256)
k_trail_project(const double* __restrict__ A, int64_t k, int64_t j0, int bw, int64_t jt0,
                int64_t ntrail, int64_t rows_per_chunk, double* __restrict__ partial) {
  constexpr int RB = 32;  // rows staged per iteration
  __shared__ double Ps[RB][kPanel + 1];
  __shared__ double Ts[RB][kProjCols + 1];
  const int64_t c0 = (int64_t)blockIdx.x * kProjCols;
  const int64_t rbeg = (int64_t)blockIdx.y * rows_per_chunk;
  int64_t rend = rbeg + rows_per_chunk;
  if (rend > k) rend = k;
  // thread -> 8 outputs: i in {ti*2, ti*2+1}, j in {tj*4 .. tj*4+3}
  const int ti = threadIdx.x / 16, tj = threadIdx.x % 16;
  double acc[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
  for (int64_t rb = rbeg; rb < rend; rb += RB) {
    for (int idx = threadIdx.x; idx < RB * kPanel; idx += 256) {
      int r = idx / kPanel, c = idx % kPanel;
      double v = 0.0;
      if (rb + r < rend && c < bw) v = A[(rb + r) * k + j0 + c];
      Ps[r][c] = v;
    }
    for (int idx = threadIdx.x; idx < RB * kProjCols; idx += 256) {
      int r = idx / kProjCols, c = idx % kProjCols;
      double v = 0.0;
      if (rb + r < rend && c0 + c < ntrail) v = A[(rb + r) * k + jt0 + c0 + c];
      Ts[r][c] = v;
    }
    __syncthreads();
#pragma unroll 8
    for (int r = 0; r < RB; ++r) {
      double p0 = Ps[r][ti * 2], p1 = Ps[r][ti * 2 + 1];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        double tv = Ts[r][tj * 4 + j];
        acc[0][j] = fma(p0, tv, acc[0][j]);
        acc[1][j] = fma(p1, tv, acc[1][j]);
      }
    }
    __syncthreads();
  }
  double* out = partial + (int64_t)blockIdx.y * kPanel * ntrail;
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int64_t col = c0 + tj * 4 + j;
      if (col < ntrail) out[(int64_t)(ti * 2 + a) * ntrail + col] = acc[a][j];
    }
}

// C[i][j] = sum_z partial[z][i][j] in chunk order.
__global__ void __launch_bounds__(256)
k_trail_reduce(const double* __restrict__ partial, int nsplit, int64_t n, double* __restrict__ C) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    double s = 0.0;
    for (int z = 0; z < nsplit; ++z) s += partial[(int64_t)z * n + i];
    C[i] = s;
  }
}

inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }

}  // namespace

size_t qr_work_doubles(int64_t k) {
  const int64_t nchunks = cdiv(k, kRows);
  return (size_t)(nchunks * kPanel * kPanel + kPanel * kPanel + (int64_t)kProjSplit * kPanel * k +
                  (int64_t)kPanel * k);
}

cudaError_t qr_pos_inplace(double* A, int64_t k, double* work, int* status, cudaStream_t s,
                           int64_t* launches, double* flops) {
  const int nchunks = (int)cdiv(k, kRows);
  double* partial = work;
  double* Rinv = partial + (int64_t)nchunks * kPanel * kPanel;
  double* proj = Rinv + kPanel * kPanel;
  double* C = proj + (int64_t)kProjSplit * kPanel * k;
  int64_t nl = 0;
  double fl = 0.0;
  cudaError_t e = cudaSuccess;
  for (int64_t j0 = 0; j0 < k; j0 += kPanel) {
    const int bw = (int)((k - j0 < kPanel) ? (k - j0) : kPanel);
    for (int pass = 0; pass < 2; ++pass) {
      k_panel_gram<<<nchunks, 256, 0, s>>>(A, k, j0, bw, partial);
      k_panel_chol<<<1, 256, 0, s>>>(partial, nchunks, bw, Rinv, status);
      k_panel_apply<<<nchunks, 256, 0, s>>>(A, k, j0, bw, Rinv);
      nl += 3;
      fl += 3.0 * (double)k * bw * bw;
    }
    const int64_t jt0 = j0 + bw, ntrail = k - jt0;
    if (ntrail > 0) {
      const int64_t rows_per_chunk = cdiv(cdiv(k, kProjSplit), 32) * 32;
      const int nsplit = (int)cdiv(k, rows_per_chunk);
      dim3 grid((unsigned)cdiv(ntrail, kProjCols), (unsigned)nsplit);
      k_trail_project<<<grid, 256, 0, s>>>(A, k, j0, bw, jt0, ntrail, rows_per_chunk, proj);
      const int64_t n = (int64_t)kPanel * ntrail;
      k_trail_reduce<<<(unsigned)((cdiv(n, 256) < 1184) ? cdiv(n, 256) : 1184), 256, 0, s>>>(proj, nsplit, n, C);
      // A_trail -= P C
      e = dgemm(0, 0, k, ntrail, bw, -1.0, A + j0, k, C, ntrail, 1.0, A + jt0, k, s);
      if (e != cudaSuccess) return e;
      nl += 3;
      fl += 4.0 * (double)k * bw * ntrail;
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (launches) *launches += nl;
  if (flops) *flops += fl;
  return cudaSuccess;
}

}  // namespace br
