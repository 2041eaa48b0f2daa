// QR orthonormalisation for Power(A, Q) = qr(A Q).Q (Sec. 3.2 of the paper), fp64, in place.
//
// The factorisation wanted is the unique one with a positive diagonal of R.  It is computed by
// a recursive block Gram-Schmidt whose floating-point work is almost entirely large fp64 matrix
// products (dgemm.cu):
//   orth(columns):  if the block is at most one panel (128 columns) wide, orthonormalise it by
//                   Cholesky-QR; otherwise orth(left half), project the left half out of the right
//                   half (C = Q_l^T A_r, A_r -= Q_l C), orth(right half).
//   Cholesky-QR of a panel P: Gram matrix S = P^T P (split over the rows), Cholesky factor
//   S = R^T R and its inverse in one CTA, P <- P R^-1.  The Cholesky factor has a positive
//   diagonal, so the signs come out as required.  The step is repeated once unless the first
//   factorisation showed the panel to be nearly orthogonal already (see k_chol_inverse).
// Half of the floating-point work is in the two products of the top level and three quarters in
// the top two, which is what lets the matrix unit run close to its peak.
//
// A block projection takes all its coefficients from the same right-hand side (as classical
// Gram-Schmidt does), so one sweep loses orthogonality like cond^2 * 1e-16, with cond the condition
// number of the column-scaled input.  Once the basis tracks the factor the columns of A Q are
// nearly orthogonal and one sweep is accurate to rounding.  The first refresh of a low-rank-plus-
// noise factor is different (cond ~ 1e5): there the whole orthonormalisation is run a second time
// on its own output ("twice is enough"), which restores orthogonality to the rounding level.  The
// second sweep is decided on the device: the first sweep compares the squared norm each column has
// left when its panel is reached with the squared norm it started with, and clears a flag when the
// ratio falls below 1e-8 (a column that kept less than 1e-4 of its length: one sweep then leaves an
// orthogonality error of up to ~1e-16 * 1e4^2); every launch of the second sweep returns at once
// while the flag is set.
// All reductions are done in a fixed order, so the result is bit-reproducible from run to run.
//
// Tensor-core projections.  Once the basis tracks the factor, the two products of a block
// projection no longer need fp64: Q_l, A_r and the coefficients C are split into three bf16 terms
// each (all 24 bits of their fp32 rounding) and the six leading products are accumulated in fp32 on
// the tcgen05 kernel, C = Q_l^T A_r and D = Q_l C, then A_r -= D in fp64, and the whole projection is
// applied twice so that what is left of span(Q_l) is ~1e-7 of the column's length after the
// projection, not before it.  The rounding of D (fp32) remains: ~6e-8 of the column's original
// length in an arbitrary direction, i.e. 6e-8 / s of the projected column when it shrinks to the
// fraction s of its length.  The caller therefore asks for this form only for a basis whose
// previous refresh saw no column shrink below 1e-3 (cond_out), the sweep still measures the
// shrinkage, and it runs the second (fp64) sweep already when a column keeps less than 1e-3 instead
// of 1e-4.  The leaves (Cholesky-QR) and the power product stay in fp64.
#include <algorithm>
#include <cstdlib>
#include <string>
#include <vector>

#include "br_internal.h"

namespace br {
namespace {

constexpr int kB = 128;          // widest panel
// A panel whose every column keeps at least this fraction of its squared norm against the columns
// before it (at least 10 % of its length) needs no second Cholesky-QR pass.
constexpr double kPassRatio = 1e-2;

inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int panel_width(int64_t k) { return k >= 1024 ? 128 : 64; }
inline int gram_splits(int64_t k) { return (int)std::min<int64_t>(64, std::max<int64_t>(1, cdiv(k, 128))); }
inline int proj_splits_max(int64_t k) { return k >= 1024 ? 64 : 1; }
constexpr double kIllRatio = 1e-8;   // squared-norm ratio below which the second sweep runs
constexpr double kTcRatio = 1e-6;    // the same, when the projections ran on the tensor cores; also
                                     // the ratio below which the next refresh must not use them
// sub-buffers of the work area start on 256-byte boundaries
inline int64_t pad32(int64_t doubles) { return (doubles + 31) / 32 * 32; }

// Cholesky factorisation S = R^T R of a bw x bw Gram matrix (bw <= 128) and R^-1, in one CTA.
//
// The matrix lives in registers: thread (ty, tx) of the 32 x 16 grid owns rows ty + 32 a (a < 4)
// and columns tx + 16 b (b < 8), a cyclic distribution that keeps every thread busy while the
// elimination shrinks the active part.  Row c reaches the other threads through shared memory,
// posted by its owners at the end of step c - 1; in step c every thread derives 1 / R_cc from it
// (redundantly, so no thread waits for another inside a step), scales the row and subtracts R_ci
// times it from each of its rows i > c.  The same row operations applied to the identity give
// R^-T; because column j of the Gram matrix is dead once step j is done and column j of R^-T is
// still a unit vector until then, both share one register array: entry (i, j) holds the Gram
// entry while j > c and the entry of R^-T afterwards.  Row c of R^-T is final after step c and is
// written out (as column c of R^-1) straight from the scaled row.
//
// A pivot that underflows 1e-24 of the column's squared norm is clamped and reported as a
// numerically rank-deficient factor.  pivot_c / S_cc is the squared sine of the angle between
// column c and the span of the panel's columns before it.  One Cholesky-QR pass loses orthogonality
// like cond^2 * 1e-16 with cond the condition number of the column-scaled panel; while every column
// keeps at least kPassRatio of its squared norm, cond^2 stays (for other than contrived matrices)
// below ~128 / kPassRatio ~ 1e4 and one pass is accurate far beyond the fp32 result, so *skip_next
// is set and the kernels of the second pass return at once.  norm0 (optional):
// squared norms the panel's columns had before any projection; a column that has lost more than
// 1 - kIllRatio of it marks the input as ill-conditioned by clearing *ill_clear.
__global__ void __launch_bounds__(512)
k_chol_inverse(const double* __restrict__ S, int bw, double* __restrict__ Rinv, int* __restrict__ status,
               int* __restrict__ skip_next, const int* __restrict__ skip_self,
               const double* __restrict__ norm0, int* __restrict__ ill_clear, double ill_ratio,
               int* __restrict__ tc_ok_clear, double* __restrict__ rdiag) {
  if (skip_self && *skip_self) {
    if (skip_next && threadIdx.x == 0) *skip_next = 1;
    return;
  }
  __shared__ double rowS[2][kB];
  __shared__ double diag0[kB], diag0_inv[kB], nrm_floor[kB], tc_floor[kB];
  const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
  if (t < kB) {
    const double n0 = (norm0 && t < bw) ? norm0[t] : 0.0;
    nrm_floor[t] = ill_ratio * n0;
    tc_floor[t] = kTcRatio * n0;
  }
  double Z[4][8];
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int i = ty + 32 * a;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const int j = tx + 16 * b;
      const double v = (i < bw && j < bw) ? S[(int64_t)i * bw + j] : (i == j ? 1.0 : 0.0);
      Z[a][b] = v;
      if (i == j) { diag0[i] = v; diag0_inv[i] = v > 0.0 ? 1.0 / v : 0.0; }
    }
  }
  if (ty == 0) {
#pragma unroll
    for (int b = 0; b < 8; ++b) rowS[0][tx + 16 * b] = Z[0][b];
  }
  __syncthreads();
  double min_ratio = 1.0;    // tracked by thread 0 (every thread sees every pivot)
  bool ill = false, tc_bad = false, any_clamped = false;

  for (int c = 0; c < bw; ++c) {
    const int buf = c & 1;
    const double orig = diag0[c];
    double piv = rowS[buf][c];
    double floor_ = orig * 1e-24;
    if (!(floor_ > 1e-300)) floor_ = 1e-300;
    const bool clamped = !(piv > floor_);
    if (clamped) piv = floor_;
    if (t == 0) {
      if (clamped) { atomicMax(status, (int)BR_WARN_RANK_DEFICIENT); any_clamped = true; }
      min_ratio = fmin(min_ratio, piv * diag0_inv[c]);
      // R_cc^2 of the whole factorisation is the product of this column's pivots over every pass and sweep
      if (rdiag) rdiag[c] *= piv;
      if (orig < nrm_floor[c]) ill = true;
      if (orig < tc_floor[c]) tc_bad = true;
    }
    const double inv_d = rsqrt(piv);
    double rj[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const int j = tx + 16 * b;
      rj[b] = (j == c) ? inv_d : rowS[buf][j] * inv_d;
    }
    // row c of R^-T is final: column c of R^-1 (zero below the diagonal)
    if (ty == 0) {
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        const int j = tx + 16 * b;
        if (j < bw) Rinv[(int64_t)j * bw + c] = (j <= c) ? rj[b] : 0.0;
      }
    }
    double f[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int i = ty + 32 * a;
      f[a] = (i > c) ? rowS[buf][i] * inv_d : 0.0;   // R_ci (row c of R, by symmetry); 0 leaves dead rows alone
#pragma unroll
      for (int b = 0; b < 8; ++b) Z[a][b] = fma(-f[a], rj[b], Z[a][b]);
    }
    // column c turns from a Gram column into a column of R^-T: entry (i, c) = -R_ci / R_cc
    if (tx == (c & 15)) {
      switch (c >> 4) {
#define BR_FIX(B)                                                          \
  case B:                                                                  \
    _Pragma("unroll") for (int a = 0; a < 4; ++a) Z[a][B] = -f[a] * inv_d; \
    break;
        BR_FIX(0) BR_FIX(1) BR_FIX(2) BR_FIX(3) BR_FIX(4) BR_FIX(5) BR_FIX(6) BR_FIX(7)
#undef BR_FIX
      }
    }
    // post row c + 1 for the next step
    if (ty == ((c + 1) & 31)) {
      switch ((c + 1) >> 5) {
#define BR_POST(A)                                                                          \
  case A:                                                                                   \
    _Pragma("unroll") for (int b = 0; b < 8; ++b) rowS[buf ^ 1][tx + 16 * b] = Z[A][b];     \
    break;
        BR_POST(0) BR_POST(1) BR_POST(2) BR_POST(3)
#undef BR_POST
      }
    }
    __syncthreads();
  }
  if (t == 0) {
    if (skip_next) *skip_next = (min_ratio >= kPassRatio) ? 1 : 0;
    if (ill && ill_clear) *ill_clear = 0;
    if (tc_bad && tc_ok_clear) *tc_ok_clear = 0;
    if (any_clamped && tc_ok_clear) tc_ok_clear[1] = 1;      // numerically rank-deficient: noted for the next refresh
  }
}

// flags at the start of a QR: second sweep cancelled, basis well enough conditioned for the
// tensor-core projections next time; and the copy of the latter to its long-lived home at the end
// bit 0: tensor-core projections allowed next time; bit 1: a pivot was clamped (complete the basis next time)
__global__ void k_store_flag(int* dst, const int* src) { *dst = (src[0] ? 1 : 0) | (src[1] ? 2 : 0); }

// part[z][j] = sum over the row chunk z of A[i][j]^2 (rows in order)
constexpr int kNormChunks = 32;
__global__ void __launch_bounds__(256)
k_column_norms_partial(const double* __restrict__ A, int64_t k, int64_t rows_per_chunk, double* __restrict__ part,
                       const int* __restrict__ skip) {
  if (skip && *skip) return;
  const int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (j >= k) return;
  const int64_t r0 = (int64_t)blockIdx.y * rows_per_chunk;
  const int64_t r1 = (r0 + rows_per_chunk < k) ? r0 + rows_per_chunk : k;
  double s0 = 0.0, s1 = 0.0;
  int64_t i = r0;
  for (; i + 1 < r1; i += 2) {
    const double a0 = A[i * k + j], a1 = A[(i + 1) * k + j];
    s0 = fma(a0, a0, s0); s1 = fma(a1, a1, s1);
  }
  if (i < r1) { const double a0 = A[i * k + j]; s0 = fma(a0, a0, s0); }
  part[(int64_t)blockIdx.y * k + j] = s0 + s1;
}
// norm0[j] = sum_z part[z][j] in chunk order; *flag = 1
__global__ void __launch_bounds__(256)
k_column_norms_sum(const double* __restrict__ part, int64_t k, int nchunks, double* __restrict__ norm0,
                   int* __restrict__ flag, double* __restrict__ rdiag, const int* __restrict__ skip) {
  const int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  // sweep-2 cancelled, tensor-core projections allowed next time, no pivot clamped so far
  // (a cancelled factorisation leaves only "sweep 2 cancelled" behind)
  const bool off = skip && *skip;
  if (j == 0) { flag[0] = 1; if (!off) { flag[1] = 1; flag[2] = 0; } }
  if (off || j >= k) return;
  double s = 0.0;
  for (int z = 0; z < nchunks; ++z) s += part[(int64_t)z * k + j];
  norm0[j] = s;
  if (rdiag) rdiag[j] = 1.0;
}

// The rank decision of the oracle's QR, on the squared diagonal of R: the product is rank-deficient when
// some R_jj^2 is at most 1e-24 of the largest (|R_jj| <= 1e-12 max_k |R_kk|), or is not a positive number.
// *run_fix = 0 then lets the completion that is enqueued behind this kernel run (it returns at once
// otherwise), the status word gets BR_WARN_RANK_DEFICIENT, and note[2] tells the next refresh of this
// basis to complete its product up front.
__global__ void __launch_bounds__(256)
k_rank_decide(const double* __restrict__ rdiag, int64_t k, int* __restrict__ skip_fix, int* __restrict__ status,
              int* __restrict__ note) {
  __shared__ double smin[256], smax[256];
  double lo = 1e300, hi = 0.0;
  bool bad = false;
  for (int64_t j = threadIdx.x; j < k; j += blockDim.x) {
    const double v = rdiag[j];
    if (!(v > 0.0)) bad = true;
    lo = fmin(lo, v); hi = fmax(hi, v);
  }
  smin[threadIdx.x] = bad ? 0.0 : lo; smax[threadIdx.x] = hi;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if (threadIdx.x < w) {
      smin[threadIdx.x] = fmin(smin[threadIdx.x], smin[threadIdx.x + w]);
      smax[threadIdx.x] = fmax(smax[threadIdx.x], smax[threadIdx.x + w]);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const bool deficient = !(smin[0] > 1e-24 * smax[0]);
    *skip_fix = deficient ? 0 : 1;
    if (deficient) { atomicMax(status, (int)BR_WARN_RANK_DEFICIENT); if (note) note[2] = 1; }
  }
}

// A <- B (k x k doubles) unless *skip
__global__ void __launch_bounds__(256)
k_copy_unless(double* __restrict__ A, const double* __restrict__ B, int64_t n, const int* __restrict__ skip) {
  if (skip && *skip) return;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) A[i] = B[i];
}

struct ProjNode { int64_t jp, wp, jt, wt; };

// projections of orth(0, k) in the order in which the recursion runs them
// A projection goes to the tensor cores when its coefficient block has at least 2^18 entries (512 x
// 512).  The grouped kernel has no split over K, so such a product has only a handful of output tiles
// and leaves most SMs idle -- to the other lanes of the refresh, which is what makes it pay: in SM-time
// it is several times cheaper than the fp64 product even so (measured on a refresh of 57 bases:
// 397 ms with a threshold of 2^21 and orders from 4096, 352 ms with 2^18 and orders from 2048, 427 ms
// with 2^14).
inline int64_t env_or(const char* name, int64_t dflt, int64_t lo, int64_t hi) {
  if (const char* e = std::getenv(name)) {
    const long long v = std::atoll(e);
    if (v >= lo && v <= hi) return v;
  }
  return dflt;
}
// tuning aids: BR_QR_TC_MIN_NODE (entries of the coefficient block), BR_QR_TC_MIN_ORDER
inline int64_t tc_min_node() { static const int64_t v = env_or("BR_QR_TC_MIN_NODE", (int64_t)1 << 18, 1 << 14, (int64_t)1 << 40); return v; }
inline int64_t tc_min_order() { static const int64_t v = env_or("BR_QR_TC_MIN_ORDER", 2048, 1024, (int64_t)1 << 30); return v; }
inline bool tc_node(int64_t wp, int64_t wt) { return wp * wt >= tc_min_node(); }

void enumerate_nodes(int64_t j0, int64_t w, int64_t b, std::vector<ProjNode>* out) {
  if (w <= b) return;
  const int64_t h = cdiv(w, 2 * b) * b;
  enumerate_nodes(j0, h, b, out);
  if (tc_node(h, w - h)) out->push_back({j0, h, j0 + h, w - h});
  enumerate_nodes(j0 + h, w - h, b, out);
}

}  // namespace

// Plans and scratch of the tensor-core projections for one order k.  Problem 2 i of either plan is
// the coefficient product of node i, problem 2 i + 1 its update product; plan `lead` holds the
// products of the two leading bf16 terms (hi*hi + mid*hi + hi*mid), plan `tail` the next three.
struct QrTc {
  int64_t k = 0;
  std::vector<ProjNode> nodes;
  TcPlan *lead = nullptr, *tail = nullptr;
  __nv_bfloat16 *Q[3] = {}, *A[3] = {}, *C[3] = {};
  float *Cf = nullptr, *Df = nullptr;
  int power_index = -1;       // problem index (in both plans) of the deflated power product
};

namespace {
inline int64_t tc_hmax(int64_t k) { return cdiv(k, 2 * 128) * 128; }
inline size_t al256(size_t x) { return (x + 255) / 256 * 256; }
}  // namespace

int64_t qr_tc_order(const QrTc* t) { return t ? t->k : 0; }
bool qr_tc_eligible(int64_t k) { return k >= tc_min_order() && (k % 8) == 0; }

size_t qr_tc_scratch_bytes(int64_t k) {
  if (!qr_tc_eligible(k)) return 0;
  const size_t h = (size_t)tc_hmax(k), kk = (size_t)k;
  // operand planes and the fp32 result hold a whole k x k matrix (the deflated power product)
  return 6 * al256(kk * kk * 2) + al256(h * h * 4) + 3 * al256(h * h * 2) + al256(kk * kk * 4);
}

void qr_tc_destroy(QrTc* t) {
  if (!t) return;
  tc_plan_destroy(t->lead);
  tc_plan_destroy(t->tail);
  delete t;
}

QrTc* qr_tc_create(int64_t k, char* scratch, int device, cudaStream_t s, const char** err) {
  static thread_local std::string last;
  if (err) *err = nullptr;
  if (!qr_tc_eligible(k) || !tc_supported(device)) return nullptr;
  QrTc* t = new QrTc();
  t->k = k;
  const size_t h = (size_t)tc_hmax(k), kk = (size_t)k;
  size_t off = 0;
  auto take = [&](size_t bytes) { char* p = scratch + off; off += al256(bytes); return p; };
  for (int i = 0; i < 3; ++i) t->Q[i] = reinterpret_cast<__nv_bfloat16*>(take(kk * kk * 2));
  for (int i = 0; i < 3; ++i) t->A[i] = reinterpret_cast<__nv_bfloat16*>(take(kk * kk * 2));
  t->Cf = reinterpret_cast<float*>(take(h * h * 4));
  for (int i = 0; i < 3; ++i) t->C[i] = reinterpret_cast<__nv_bfloat16*>(take(h * h * 2));
  t->Df = reinterpret_cast<float*>(take(kk * kk * 4));
  enumerate_nodes(0, k, 128, &t->nodes);
  std::vector<TcProblem> lead, tail;
  auto opnd = [](const void* p, int64_t ld, int mn) { TcOperand o; o.ptr = p; o.ld = ld; o.mn_major = mn; return o; };
  for (const ProjNode& nd : t->nodes) {
    // coefficients C = Q^T A_r (contraction over the k rows: both operands MN-major)
    TcProblem c; c.Md = nd.wp; c.Nd = nd.wt; c.K = k; c.n_pairs = 3;
    c.epilogue = EPI_AXPBY_F32; c.alpha = 1.f; c.D = t->Cf; c.ldd = nd.wt;
    TcProblem c2 = c;
    const int ia[6] = {0, 1, 0, 2, 0, 1}, ib[6] = {0, 0, 1, 0, 2, 1};      // term pairs, leading three first
    for (int p = 0; p < 3; ++p) {
      c.A[p] = opnd(t->Q[ia[p]], nd.wp, 1); c.B[p] = opnd(t->A[ib[p]], nd.wt, 1);
      c2.A[p] = opnd(t->Q[ia[3 + p]], nd.wp, 1); c2.B[p] = opnd(t->A[ib[3 + p]], nd.wt, 1);
    }
    c.beta = 0.f; c2.beta = 1.f;
    // update D = Q C (Q K-major, C MN-major)
    TcProblem d; d.Md = k; d.Nd = nd.wt; d.K = nd.wp; d.n_pairs = 3;
    d.epilogue = EPI_AXPBY_F32; d.alpha = 1.f; d.D = t->Df; d.ldd = nd.wt;
    TcProblem d2 = d;
    for (int p = 0; p < 3; ++p) {
      d.A[p] = opnd(t->Q[ia[p]], nd.wp, 0); d.B[p] = opnd(t->C[ib[p]], nd.wt, 1);
      d2.A[p] = opnd(t->Q[ia[3 + p]], nd.wp, 0); d2.B[p] = opnd(t->C[ib[3 + p]], nd.wt, 1);
    }
    d.beta = 0.f; d2.beta = 1.f;
    lead.push_back(c); lead.push_back(d);
    tail.push_back(c2); tail.push_back(d2);
  }
  {
    // the power product of the deflated factor: D = F_rest U, F_rest (k x k) K-major, U MN-major
    const int ia[6] = {0, 1, 0, 2, 0, 1}, ib[6] = {0, 0, 1, 0, 2, 1};
    TcProblem p1; p1.Md = k; p1.Nd = k; p1.K = k; p1.n_pairs = 3;
    p1.epilogue = EPI_AXPBY_F32; p1.alpha = 1.f; p1.D = t->Df; p1.ldd = k;
    TcProblem p2 = p1;
    for (int p = 0; p < 3; ++p) {
      p1.A[p] = opnd(t->Q[ia[p]], k, 0); p1.B[p] = opnd(t->A[ib[p]], k, 1);
      p2.A[p] = opnd(t->Q[ia[3 + p]], k, 0); p2.B[p] = opnd(t->A[ib[3 + p]], k, 1);
    }
    p1.beta = 0.f; p2.beta = 1.f;
    t->power_index = (int)lead.size();
    lead.push_back(p1);
    tail.push_back(p2);
  }
  const char* perr = nullptr;
  if (!lead.empty()) {
    t->lead = tc_plan_create(lead.data(), (int)lead.size(), device, s, &perr);
    if (t->lead) t->tail = tc_plan_create(tail.data(), (int)tail.size(), device, s, &perr);
    if (!t->lead || !t->tail) {
      last = perr ? perr : "plan creation failed";
      if (err) *err = last.c_str();
      qr_tc_destroy(t);
      return nullptr;
    }
  }
  return t;
}

cudaError_t qr_tc_project(QrTc* t, int node, double* A, int64_t k, int64_t jp, int64_t wp, int64_t jt,
                          int64_t wt, int* status, cudaStream_t s) {
  if (node < 0 || node >= (int)t->nodes.size()) return cudaErrorInvalidValue;
  const ProjNode& nd = t->nodes[node];
  if (nd.jp != jp || nd.wp != wp || nd.jt != jt || nd.wt != wt || t->k != k) return cudaErrorInvalidValue;
  cudaError_t e;
  if ((e = split3_f64(A + jp, k, k, wp, t->Q[0], t->Q[1], t->Q[2], s)) != cudaSuccess) return e;
  // Twice: whatever error the coefficients of the first pass have leaves that much of span(Q_l) in
  // the column, measured against its length BEFORE the projection; the second pass sees the shrunken
  // column and leaves ~1e-7 of its length AFTER the projection.  Because the second pass removes what
  // the first left inside span(Q_l), the first pass's coefficients need only the three leading
  // products (2^-16); its update Q_l C must be accurate to 2^-24 (its rounding leaves span(Q_l)), so it
  // takes all six.  The second pass is the other way round: coefficients with all six products (they
  // are a small difference of large terms), update with the leading three (C is ~2^-16 of the column
  // by then).  18 products instead of 24.
  for (int pass = 0; pass < 2; ++pass) {
    if ((e = split3_f64(A + jt, k, k, wt, t->A[0], t->A[1], t->A[2], s)) != cudaSuccess) return e;
    if ((e = tc_plan_launch_range(t->lead, 2 * node, 1, 1, 0, 1.f, 0.f, status, s)) != cudaSuccess) return e;
    if (pass == 1 && (e = tc_plan_launch_range(t->tail, 2 * node, 1, 1, 0, 1.f, 0.f, status, s)) != cudaSuccess) return e;
    if ((e = split3_f32(t->Cf, wp * wt, t->C[0], t->C[1], t->C[2], s)) != cudaSuccess) return e;
    if ((e = tc_plan_launch_range(t->lead, 2 * node + 1, 1, 1, 0, 1.f, 0.f, status, s)) != cudaSuccess) return e;
    if (pass == 0 && (e = tc_plan_launch_range(t->tail, 2 * node + 1, 1, 1, 0, 1.f, 0.f, status, s)) != cudaSuccess) return e;
    if ((e = sub_f32_from_f64(A + jt, k, k, wt, t->Df, s)) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// D (fp32, k x k, returned in *out) = Frest U with both operands split into three bf16 terms and the
// six leading products accumulated in fp32.  Frest and U are fp64, row-major with leading dimension k.
cudaError_t qr_tc_power(QrTc* t, const double* Frest, const double* U, int* status, cudaStream_t s, const float** out) {
  const int64_t k = t->k;
  cudaError_t e;
  if ((e = split3_f64(Frest, k, k, k, t->Q[0], t->Q[1], t->Q[2], s)) != cudaSuccess) return e;
  if ((e = split3_f64(U, k, k, k, t->A[0], t->A[1], t->A[2], s)) != cudaSuccess) return e;
  if ((e = tc_plan_launch_range(t->lead, t->power_index, 1, 1, 0, 1.f, 0.f, status, s)) != cudaSuccess) return e;
  if ((e = tc_plan_launch_range(t->tail, t->power_index, 1, 1, 0, 1.f, 0.f, status, s)) != cudaSuccess) return e;
  *out = t->Df;
  return cudaSuccess;
}

namespace {

struct Sweep {
  double* A; int64_t k; int b, sg, sp_max;
  double *gram_part, *S, *Rinv, *norm0, *C, *proj_part;
  double* rdiag = nullptr;    // squared diagonal of R, accumulated over passes and sweeps
  int *skip2, *sweep2_skip;   // sweep2_skip[1] is the "tensor cores allowed next time" flag
  QrTc* tc = nullptr;         // non-null: block projections of the first sweep on the tensor cores
  int node = 0;               // running index of the projection in recursion order
  double ill_ratio = kIllRatio;
  int* status;
  cudaStream_t s;
  const int* skip;        // non-null: every launch of this sweep returns while *skip != 0
  bool first;             // first sweep: watch the column norms
  int64_t launches = 0;
  double flops = 0.0;
  cudaError_t err = cudaSuccess;
};

// Cholesky-QR (at most twice) of the panel of columns [j0, j0 + bw).
void leaf(Sweep& q, int64_t j0, int bw) {
  double* P = q.A + j0;
  const int64_t k = q.k;
  for (int pass = 0; pass < 2 && q.err == cudaSuccess; ++pass) {
    const int* skip = pass ? q.skip2 : q.skip;
    cudaError_t e = dgemm_ex(1, 0, bw, bw, k, 1.0, P, k, P, k, 0.0, q.S, bw, q.sg, q.gram_part, skip, q.s);
    if (e != cudaSuccess) { q.err = e; return; }
    k_chol_inverse<<<1, 512, 0, q.s>>>(q.S, bw, q.Rinv, q.status, pass ? nullptr : q.skip2, skip,
                                       (q.first && !pass) ? q.norm0 + j0 : nullptr, q.sweep2_skip, q.ill_ratio,
                                       q.sweep2_skip + 1, q.rdiag ? q.rdiag + j0 : nullptr);
    // P <- P R^-1 (in place: a CTA reads only the rows it writes, and writes after its last read)
    e = dgemm_ex(0, 0, k, bw, bw, 1.0, P, k, q.Rinv, bw, 0.0, P, k, 1, nullptr, skip, q.s);
    if (e != cudaSuccess) { q.err = e; return; }
    q.launches += 3 + (q.sg > 1 ? 1 : 0);
    if (q.first && !pass) q.flops += 4.0 * (double)k * bw * bw;
  }
}

// A[:, jt : jt + wt] -= Q (Q^T A[:, jt : jt + wt]) with Q = A[:, jp : jp + wp] orthonormal.
void project(Sweep& q, int64_t jp, int64_t wp, int64_t jt, int64_t wt) {
  if (q.err != cudaSuccess) return;
  const int64_t k = q.k;
  if (q.tc && q.first && tc_node(wp, wt)) {
    q.err = qr_tc_project(q.tc, q.node++, q.A, k, jp, wp, jt, wt, q.status, q.s);
    q.launches += 13;
    return;
  }
  const int64_t tiles = cdiv(wp, 128) * cdiv(wt, 128);
  int sp = 1;
  if (tiles < 148) sp = (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(cdiv(296, tiles), q.sp_max), k / 128));
  cudaError_t e = dgemm_ex(1, 0, wp, wt, k, 1.0, q.A + jp, k, q.A + jt, k, 0.0, q.C, wt, sp, q.proj_part, q.skip, q.s);
  if (e == cudaSuccess)
    e = dgemm_ex(0, 0, k, wt, wp, -1.0, q.A + jp, k, q.C, wt, 1.0, q.A + jt, k, 1, nullptr, q.skip, q.s);
  if (e != cudaSuccess) { q.err = e; return; }
  q.launches += 2 + (sp > 1 ? 1 : 0);
  if (q.first) q.flops += 4.0 * (double)k * wp * wt;
}

void orth(Sweep& q, int64_t j0, int64_t w) {
  if (q.err != cudaSuccess) return;
  if (w <= q.b) { leaf(q, j0, (int)w); return; }
  const int64_t h = cdiv(w, 2 * q.b) * q.b;     // left part: a whole number of panels
  orth(q, j0, h);
  project(q, j0, h, j0 + h, w - h);
  orth(q, j0 + h, w - h);
}

inline int64_t proj_part_doubles(int64_t k) {
  const int sp = proj_splits_max(k);
  if (sp <= 1) return 0;
  // a projection is split only while it has fewer than 148 tiles of 128 x 128
  return std::min<int64_t>((int64_t)sp * ((k + 1) / 2) * ((k + 1) / 2), (int64_t)(296 + 148) * 128 * 128);
}

}  // namespace

namespace {
constexpr double kCompletion = 1e-6;
template <typename TQ>
__global__ void __launch_bounds__(256)
k_complete_columns(double* __restrict__ A, const TQ* __restrict__ Q, int64_t k, const double* __restrict__ norm2,
                   int* __restrict__ status, const int* __restrict__ skip) {
  if (skip && *skip) return;
  const int64_t total = k * k;
  if (blockIdx.x == 0 && threadIdx.x == 0) atomicMax(status, (int)BR_WARN_RANK_DEFICIENT);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t c = i % k;
    const double n2 = norm2[c];
    const double d = n2 > 0.0 ? kCompletion * sqrt(n2) : 1.0;
    A[i] = fma(d, (double)Q[i], A[i]);
  }
}
}  // namespace

namespace {
template <typename TQ>
cudaError_t complete_columns(double* A, const TQ* Q, int64_t k, double* work, int* status, const int* skip, cudaStream_t s) {
  // column norms exactly as the factorisation computes them (same kernels, same order)
  double* part = work;                                   // kNormChunks * k doubles at most (see qr_work_doubles)
  const int nchunks = (int)std::min<int64_t>(kNormChunks, std::max<int64_t>(1, k / 4));
  const int64_t rows_per_chunk = cdiv(k, nchunks);
  const int used = (int)cdiv(k, rows_per_chunk);
  double* norm2 = part + (int64_t)used * k;
  int* dummy = reinterpret_cast<int*>(norm2 + k);
  dim3 grid((unsigned)cdiv(k, 256), (unsigned)used);
  k_column_norms_partial<<<grid, 256, 0, s>>>(A, k, rows_per_chunk, part, skip);
  k_column_norms_sum<<<(unsigned)cdiv(k, 256), 256, 0, s>>>(part, k, used, norm2, dummy, nullptr, skip);
  const int64_t blocks = cdiv(k * k, 256);
  k_complete_columns<TQ><<<(unsigned)(blocks < 1184 ? blocks : 1184), 256, 0, s>>>(A, Q, k, norm2, status, skip);
  return cudaGetLastError();
}
}  // namespace

cudaError_t qr_complete_columns(double* A, const float* Q, int64_t k, double* work, int* status, cudaStream_t s) {
  return complete_columns<float>(A, Q, k, work, status, nullptr, s);
}

size_t qr_work_doubles(int64_t k) {
  const int64_t b = std::min<int64_t>(panel_width(k), k);
  return (size_t)(pad32((int64_t)gram_splits(k) * b * b) + 2 * pad32(b * b) + 64 + pad32(k) +
                  pad32(((k + 1) / 2) * ((k + 1) / 2)) + pad32(proj_part_doubles(k)) + pad32(k));
}

namespace {
// One factorisation (two sweeps, the second cancelled on the device unless the first met an ill-conditioned
// input).  flag_base: which of the flag words of the work area this run uses; skip_all: a DEVICE flag that
// turns the whole run into launches that return at once; rdiag: receives the squared diagonal of R.
cudaError_t run_qr(double* A, int64_t k, double* work, int flag_base, int* status, cudaStream_t s, const int* skip_all,
                   QrTc* tc, bool track_rdiag, int64_t* launches, double* flops) {
  Sweep q;
  if (tc && tc->k == k) { q.tc = tc; q.ill_ratio = kTcRatio; }
  q.A = A; q.k = k; q.s = s; q.status = status;
  q.b = (int)std::min<int64_t>(panel_width(k), k);
  q.sg = gram_splits(k);
  q.sp_max = proj_splits_max(k);
  const int64_t b = q.b;
  q.gram_part = work;
  q.S = q.gram_part + pad32((int64_t)q.sg * b * b);
  q.Rinv = q.S + pad32(b * b);
  int* flags = reinterpret_cast<int*>(q.Rinv + pad32(b * b)) + flag_base;      // 64 doubles reserved for flags
  q.skip2 = flags;
  q.sweep2_skip = flags + 1;
  q.norm0 = q.Rinv + pad32(b * b) + 64;
  q.C = q.norm0 + pad32(k);
  q.proj_part = q.C + pad32(((k + 1) / 2) * ((k + 1) / 2));
  q.rdiag = track_rdiag ? q.proj_part + pad32(proj_part_doubles(k)) : nullptr;
  // first sweep, watching how much of its norm each column keeps
  {
    // the partial sums borrow the (still unused) projection buffer: kNormChunks * k <= (k + 1)^2 / 4 for k >= 128
    const int nchunks = (int)std::min<int64_t>(kNormChunks, std::max<int64_t>(1, k / 4));
    const int64_t rows_per_chunk = cdiv(k, nchunks);
    const int used = (int)cdiv(k, rows_per_chunk);
    dim3 grid((unsigned)cdiv(k, 256), (unsigned)used);
    k_column_norms_partial<<<grid, 256, 0, s>>>(A, k, rows_per_chunk, q.C, skip_all);
    k_column_norms_sum<<<(unsigned)cdiv(k, 256), 256, 0, s>>>(q.C, k, used, q.norm0, q.sweep2_skip, q.rdiag, skip_all);
  }
  q.skip = skip_all; q.first = true;
  orth(q, 0, k);
  if (q.err != cudaSuccess) return q.err;
  // second sweep, cancelled on the device unless the first one met an ill-conditioned input
  q.skip = q.sweep2_skip; q.first = false;
  orth(q, 0, k);
  if (q.err != cudaSuccess) return q.err;
  if (launches) *launches += q.launches + 2;
  if (flops) *flops += q.flops;
  return cudaGetLastError();
}
}  // namespace

cudaError_t qr_pos_inplace(double* A, int64_t k, double* work, int* status, cudaStream_t s,
                           int64_t* launches, double* flops, QrTc* tc, int* cond_out, const double* Acopy,
                           const double* Qprev) {
  const bool fix = Acopy != nullptr && Qprev != nullptr;
  cudaError_t e = run_qr(A, k, work, 0, status, s, nullptr, tc, fix, launches, flops);
  if (e != cudaSuccess) return e;
  const int64_t b = std::min<int64_t>(panel_width(k), k);
  int* flags = reinterpret_cast<int*>(work + pad32((int64_t)gram_splits(k) * b * b) + 2 * pad32(b * b));
  if (fix) {
    // The oracle's rule for a rank-deficient product (decided on the diagonal of R, as the oracle decides
    // it): factorise A with 1e-6 ||A_j|| Qprev_j added to every column instead.  Everything is enqueued
    // here and returns at once unless the decision kernel finds the product deficient.
    double* rdiag = work + qr_work_doubles(k) - pad32(k);
    int* skip_fix = flags + 16;
    k_rank_decide<<<1, 256, 0, s>>>(rdiag, k, skip_fix, status, flags + 1);
    const int64_t n = k * k, blocks = cdiv(n, 256);
    k_copy_unless<<<(unsigned)(blocks < 1184 ? blocks : 1184), 256, 0, s>>>(A, Acopy, n, skip_fix);
    if ((e = complete_columns<double>(A, Qprev, k, work, status, skip_fix, s)) != cudaSuccess) return e;
    if ((e = run_qr(A, k, work, 8, status, s, skip_fix, nullptr, false, launches, nullptr)) != cudaSuccess) return e;
    if (launches) *launches += 5;
  }
  if (cond_out) { k_store_flag<<<1, 1, 0, s>>>(cond_out, flags + 2); if (launches) *launches += 1; }
  return cudaGetLastError();
}

}  // namespace br
