// QR orthonormalisation for Power(A, Q) = qr(A Q).Q (Sec. 3.2 of the paper), fp64, in place.
//
// The factorisation wanted is the unique one with a positive diagonal of R.  It is computed by
// a right-looking block Gram-Schmidt whose floating-point work is almost entirely fp64 matrix
// products (dgemm.cu): for each panel P of up to 128 columns
//   1. orthonormalise the panel by Cholesky-QR: Gram matrix S = P^T P (split over the rows),
//      Cholesky factor S = R^T R and its inverse in one CTA, P <- P R^-1.  The Cholesky factor
//      has a positive diagonal, so the signs come out as required.  The step is repeated once
//      unless the first Cholesky factorisation showed the panel to be nearly orthogonal already
//      (see k_chol_inverse), which is the usual case once the basis tracks the factor;
//   2. project the panel out of all trailing columns: C = P^T A_trail, A_trail -= P C.
// In fp64 the loss of orthogonality of this scheme is ~ cond * 1e-16, far below the fp32
// rounding of the stored bases, and the result agrees with Householder QR to the same level.
// All reductions are done in a fixed order, so the result is bit-reproducible from run to run.
#include <algorithm>

#include "br_internal.h"

namespace br {
namespace {

constexpr int kB = 128;          // widest panel
constexpr double kDefectLimit = 0.1;

inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int panel_width(int64_t k) { return k >= 1024 ? 128 : 64; }
inline int gram_splits(int64_t k) { return (int)std::min<int64_t>(64, std::max<int64_t>(1, cdiv(k, 128))); }
inline int proj_splits_max(int64_t k) { return k >= 1024 ? 8 : 2; }
// sub-buffers of the work area start on 256-byte boundaries
inline int64_t pad32(int64_t doubles) { return (doubles + 31) / 32 * 32; }

// Cholesky factorisation S = R^T R of a bw x bw Gram matrix (bw <= 128) and R^-1, in one CTA.
//
// The matrix lives in registers: thread (ty, tx) of the 16 x 16 grid owns rows ty + 16 a and
// columns tx + 16 b (a, b < 8), a cyclic distribution that keeps every thread busy while the
// elimination shrinks the active part.  Step c scales row c by 1 / R_cc, shares it through shared
// memory and subtracts R_ci times it from every row i > c.  The same row operations applied to the
// identity give R^-T; because column j of the Gram matrix is dead once step j is done and column j
// of R^-T is still a unit vector until then, both share one register array: entry (i, j) holds the
// Gram entry while j > c and the entry of R^-T afterwards.
//
// A pivot that underflows 1e-24 of the column's squared norm is clamped and reported as a
// numerically rank-deficient factor.  defect = sum_c (1 - pivot_c / S_cc) bounds the squared
// Frobenius distance of the column-scaled Gram matrix from the identity (up to a factor ~2): when
// it is small the panel was close to orthogonal and one Cholesky-QR pass is accurate to rounding,
// so *skip_next is set and the kernels of the second pass return at once.
__global__ void __launch_bounds__(256)
k_chol_inverse(const double* __restrict__ S, int bw, double* __restrict__ Rinv, int* __restrict__ status,
               int* __restrict__ skip_next, const int* __restrict__ skip_self) {
  if (skip_self && *skip_self) return;
  __shared__ double rowZ[2][kB];
  __shared__ double defect_sm;
  const int t = threadIdx.x, ty = t >> 4, tx = t & 15, lane = t & 31;
  double Z[8][8];
  double d0[8];
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int i = ty + 16 * a;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const int j = tx + 16 * b;
      Z[a][b] = (i < bw && j < bw) ? S[(int64_t)i * bw + j] : (i == j ? 1.0 : 0.0);
    }
    d0[a] = Z[a][a];        // meaningful on the diagonal threads (ty == tx) only
  }
  if (t == 0) defect_sm = 0.0;
  __syncthreads();

  for (int c = 0; c < bw; ++c) {
    const int buf = c & 1, ca = c >> 4, cr = c & 15;
    if (ty == cr) {
      // the 16 owners of row c are one half of a warp
      double zr[8];
#pragma unroll
      for (int a = 0; a < 8; ++a)
        if (a == ca) {
#pragma unroll
          for (int b = 0; b < 8; ++b) zr[b] = Z[a][b];
        }
      double piv = 0.0;
      if (tx == cr) {
        double orig = 0.0;
#pragma unroll
        for (int b = 0; b < 8; ++b)
          if (b == ca) { piv = zr[b]; orig = d0[b]; }
        double floor_ = orig * 1e-24;
        if (!(floor_ > 1e-300)) floor_ = 1e-300;
        if (!(piv > floor_)) {
          piv = floor_;
          atomicMax(status, (int)BR_WARN_RANK_DEFICIENT);
        }
        defect_sm += (orig > 0.0) ? fmax(0.0, 1.0 - piv / orig) : 1.0;
      }
      const unsigned half = (lane < 16) ? 0x0000FFFFu : 0xFFFF0000u;
      piv = __shfl_sync(half, piv, (lane & 16) | cr);
      const double inv_d = 1.0 / sqrt(piv);
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        const int j = tx + 16 * b;
        const double v = (j == c) ? inv_d : zr[b] * inv_d;
        zr[b] = v;
        rowZ[buf][j] = v;
      }
#pragma unroll
      for (int a = 0; a < 8; ++a)
        if (a == ca) {
#pragma unroll
          for (int b = 0; b < 8; ++b) Z[a][b] = zr[b];
        }
    }
    __syncthreads();
    double rj[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) rj[b] = rowZ[buf][tx + 16 * b];
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      const int i = ty + 16 * a;
      if (i > c) {
        const double f = rowZ[buf][i];        // R_ci (row c of R, by symmetry of the Gram matrix)
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          const double old = (tx + 16 * b == c) ? 0.0 : Z[a][b];
          Z[a][b] = fma(-f, rj[b], old);
        }
      }
    }
  }
  __syncthreads();
  if (t == 0 && skip_next) *skip_next = (defect_sm <= kDefectLimit) ? 1 : 0;
  // Z holds R^-T in its lower triangle: R^-1 (i, j) = Z (j, i)
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int i = ty + 16 * a;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const int j = tx + 16 * b;
      if (i < bw && j < bw) Rinv[(int64_t)j * bw + i] = (j <= i) ? Z[a][b] : 0.0;
    }
  }
}

}  // namespace

size_t qr_work_doubles(int64_t k) {
  const int64_t b = std::min<int64_t>(panel_width(k), k);
  return (size_t)(pad32((int64_t)gram_splits(k) * b * b) + 2 * pad32(b * b) + 64 +
                  pad32((int64_t)proj_splits_max(k) * b * k) + pad32(b * k));
}

cudaError_t qr_pos_inplace(double* A, int64_t k, double* work, int* status, cudaStream_t s,
                           int64_t* launches, double* flops) {
  const int64_t b = std::min<int64_t>(panel_width(k), k);
  const int sg = gram_splits(k);
  double* gram_part = work;
  double* S = gram_part + pad32((int64_t)sg * b * b);
  double* Rinv = S + pad32(b * b);
  int* skip2 = reinterpret_cast<int*>(Rinv + pad32(b * b));      // 64 doubles reserved for flags
  double* proj_part = Rinv + pad32(b * b) + 64;
  double* C = proj_part + pad32((int64_t)proj_splits_max(k) * b * k);
  int64_t nl = 0;
  double fl = 0.0;
  cudaError_t e = cudaSuccess;
  for (int64_t j0 = 0; j0 < k; j0 += b) {
    const int bw = (int)std::min<int64_t>(b, k - j0);
    double* P = A + j0;
    for (int pass = 0; pass < 2; ++pass) {
      const int* skip = pass ? skip2 : nullptr;
      // S = P^T P
      if ((e = dgemm_ex(1, 0, bw, bw, k, 1.0, P, k, P, k, 0.0, S, bw, sg, gram_part, skip, s)) != cudaSuccess) return e;
      k_chol_inverse<<<1, 256, 0, s>>>(S, bw, Rinv, status, pass ? nullptr : skip2, skip);
      // P <- P R^-1 (in place: a CTA reads only the rows it writes, and writes after its last read)
      if ((e = dgemm_ex(0, 0, k, bw, bw, 1.0, P, k, Rinv, bw, 0.0, P, k, 1, nullptr, skip, s)) != cudaSuccess) return e;
      nl += 3 + (sg > 1 ? 1 : 0);
      fl += 4.0 * (double)k * bw * bw;
    }
    const int64_t jt0 = j0 + bw, ntrail = k - jt0;
    if (ntrail > 0) {
      int sp = (int)cdiv(296, cdiv(ntrail, 128));
      sp = std::max(1, std::min(sp, std::min(proj_splits_max(k), (int)std::max<int64_t>(1, k / 256))));
      // C = P^T A_trail ; A_trail -= P C
      if ((e = dgemm_ex(1, 0, bw, ntrail, k, 1.0, P, k, A + jt0, k, 0.0, C, ntrail, sp, proj_part, nullptr, s)) != cudaSuccess) return e;
      if ((e = dgemm_ex(0, 0, k, ntrail, bw, -1.0, P, k, C, ntrail, 1.0, A + jt0, k, 1, nullptr, nullptr, s)) != cudaSuccess) return e;
      nl += 2 + (sp > 1 ? 1 : 0);
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
