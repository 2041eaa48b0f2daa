// fp64-accumulating contractions for the basis refresh (Power(F, Q) of Sec. 3.2): the product
// F Q and the block projections of the QR must be resolved far below the fp32 rounding level
// (F mixes eigenvalues that differ by 1e5, and the small ones are what the trailing basis vectors
// are made of), so they run on the fp64 matrix unit:
//
//   C = alpha * op(A) op(B) + beta * C,  C fp64, A and B fp32 or fp64, all row-major.
//
// 128 x 128 x 16 tiles, 8 warps, each warp a 32 x 64 sub-tile as 4 x 8 mma.sync.m8n8k4.f64
// fragments (64 accumulator doubles per thread), two shared-memory stages with the next tile
// prefetched into registers during the math.  Transposed operands are staged in a second
// shared-memory layout instead of being transposed on the way.  fp32 operands are widened while they are staged,
// so every product is exact and only the fp64 accumulation rounds.  A contraction that is long
// and narrow (Gram matrices, panel projections) is split over K into partial sums that a second
// kernel adds in a fixed order, which keeps the result reproducible from run to run.
#include "br_internal.h"
#include "step_tc.h"

namespace br {
namespace {

constexpr int BM = 128, BN = 128, BK = 16;
// A staged operand tile holds 128 (i) x 16 (kk) doubles in one of two layouts, chosen so that the
// copy from global memory needs no transposition and both the copy and the fragment loads are free
// of bank conflicts:
//   k-major  S[kk * 136 + i]   for an operand whose i index is contiguous in global memory
//   i-major  S[i * 20 + kk]    for an operand whose contraction index is contiguous
constexpr int LDK = 136, LDI = 20;
constexpr int TILE = BM * LDI;            // doubles reserved per operand tile (>= BK * LDK)
constexpr int STAGE = 2 * TILE;           // doubles per stage (A tile + B tile)
constexpr int SMEM_BYTES = 2 * STAGE * (int)sizeof(double);

__device__ __forceinline__ void dmma(double& c0, double& c1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

template <typename T> struct Vec2;
template <> struct Vec2<double> { using type = double2; };
template <> struct Vec2<float> { using type = float2; };

// One operand tile of 128 (i) x 16 (kk) elements, fetched into 8 registers per thread.
//   direct : element (kk, i) at X[(k0 + kk) * ld + i0 + i]   (contraction index is the slow one)
//   scatter: element (i, kk) at X[(i0 + i) * ld + k0 + kk]   (contraction index is contiguous)
// Either way 8 (float: 16) consecutive threads read one contiguous 128-byte (64-byte) run.
// `fast` = the tile is interior and 2-element vector loads are aligned.
template <typename T>
__device__ __forceinline__ void tile_load(double (&r)[8], const T* __restrict__ X, int64_t ld, bool scatter,
                                          bool fast, int64_t i0, int64_t k0, int64_t I, int64_t Kend) {
  const int t = threadIdx.x;
  using V = typename Vec2<T>::type;
  if (!scatter) {
    const int lk = t >> 4, li = (t & 15) * 2;
    const T* row = X + (k0 + lk) * ld + i0 + li;
    if (fast) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const V v = *reinterpret_cast<const V*>(row + 32 * q);
        r[2 * q] = (double)v.x; r[2 * q + 1] = (double)v.y;
      }
    } else {
      const bool kok = (k0 + lk) < Kend;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int64_t i = i0 + li + 32 * q;
        r[2 * q] = (kok && i < I) ? (double)row[32 * q] : 0.0;
        r[2 * q + 1] = (kok && i + 1 < I) ? (double)row[32 * q + 1] : 0.0;
      }
    }
  } else {
    const int li = t >> 3, lk = (t & 7) * 2;      // rows li + 32 q, columns k0 + lk, k0 + lk + 1
    const T* p = X + (i0 + li) * ld + k0 + lk;
    if (fast) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const V v = *reinterpret_cast<const V*>(p + (int64_t)32 * q * ld);
        r[2 * q] = (double)v.x; r[2 * q + 1] = (double)v.y;
      }
    } else {
      const bool k0ok = (k0 + lk) < Kend, k1ok = (k0 + lk + 1) < Kend;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const bool iok = (i0 + li + 32 * q) < I;
        r[2 * q] = (iok && k0ok) ? (double)p[(int64_t)32 * q * ld] : 0.0;
        r[2 * q + 1] = (iok && k1ok) ? (double)p[(int64_t)32 * q * ld + 1] : 0.0;
      }
    }
  }
}

// Registers -> staged tile (k-major for a direct operand, i-major for a scatter operand).
__device__ __forceinline__ void tile_store(double* __restrict__ S, const double (&r)[8], bool scatter) {
  const int t = threadIdx.x;
  if (!scatter) {
    const int lk = t >> 4, li = (t & 15) * 2;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      *reinterpret_cast<double2*>(S + lk * LDK + li + 32 * q) = make_double2(r[2 * q], r[2 * q + 1]);
  } else {
    const int li = t >> 3, lk = (t & 7) * 2;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      *reinterpret_cast<double2*>(S + (li + 32 * q) * LDI + lk) = make_double2(r[2 * q], r[2 * q + 1]);
  }
}

template <typename TA, typename TB>
__global__ void __launch_bounds__(256)
k_dgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const TA* __restrict__ A, int64_t lda,
        const TB* __restrict__ B, int64_t ldb, double beta, double* __restrict__ C, int64_t ldc,
        int vec_a, int vec_b, int vec_c, int64_t k_per_split, double* __restrict__ partial,
        const int* __restrict__ skip) {
  extern __shared__ double sm[];
  if (skip && *skip) return;            // uniform: a device-side flag cancels the whole launch
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
  const int64_t kbeg = (int64_t)blockIdx.z * k_per_split;
  const int64_t kend = (kbeg + k_per_split < K) ? kbeg + k_per_split : K;
  const bool a_scatter = !ta, b_scatter = tb != 0;
  const bool a_int = vec_a && (m0 + BM <= M), b_int = vec_b && (n0 + BN <= N);

  double acc[64];
#pragma unroll
  for (int i = 0; i < 64; ++i) acc[i] = 0.0;
  const int g = lane >> 2, tig = lane & 3;
  const int wm = w & 3, wn = w >> 2;

  double pa[8], pb[8];
  const int64_t nk = (kend - kbeg + BK - 1) / BK;
  if (nk > 0) {
    const bool kfull = kbeg + BK <= kend;
    tile_load<TA>(pa, A, lda, a_scatter, a_int && kfull, m0, kbeg, M, kend);
    tile_load<TB>(pb, B, ldb, b_scatter, b_int && kfull, n0, kbeg, N, kend);
    tile_store(sm, pa, a_scatter);
    tile_store(sm + TILE, pb, b_scatter);
  }
  __syncthreads();
  // fragment addressing: element (i, kk) of a staged tile sits at i * si + kk * sk
  const int a_si = a_scatter ? LDI : 1, a_sk = a_scatter ? 1 : LDK;
  const int b_si = b_scatter ? LDI : 1, b_sk = b_scatter ? 1 : LDK;
  const int a_base = (32 * wm + g) * a_si + tig * a_sk;
  const int b_base = (64 * wn + g) * b_si + tig * b_sk;
  for (int64_t kt = 0; kt < nk; ++kt) {
    const int st = (int)(kt & 1);
    if (kt + 1 < nk) {
      const int64_t k0 = kbeg + (kt + 1) * BK;
      const bool kfull = k0 + BK <= kend;
      tile_load<TA>(pa, A, lda, a_scatter, a_int && kfull, m0, k0, M, kend);
      tile_load<TB>(pb, B, ldb, b_scatter, b_int && kfull, n0, k0, N, kend);
    }
    const double* As = sm + st * STAGE + a_base;
    const double* Bs = sm + st * STAGE + TILE + b_base;
#pragma unroll
    for (int k4 = 0; k4 < BK; k4 += 4) {
      double a[4], b[8];
#pragma unroll
      for (int mi = 0; mi < 4; ++mi) a[mi] = As[8 * mi * a_si + k4 * a_sk];
#pragma unroll
      for (int ni = 0; ni < 8; ++ni) b[ni] = Bs[8 * ni * b_si + k4 * b_sk];
#pragma unroll
      for (int mi = 0; mi < 4; ++mi)
#pragma unroll
        for (int ni = 0; ni < 8; ++ni) dmma(acc[(mi * 8 + ni) * 2], acc[(mi * 8 + ni) * 2 + 1], a[mi], b[ni]);
    }
    if (kt + 1 < nk) {
      double* Sn = sm + (st ^ 1) * STAGE;
      tile_store(Sn, pa, a_scatter);
      tile_store(Sn + TILE, pb, b_scatter);
    }
    __syncthreads();
  }

  // accumulator fragment (mi, ni): rows 32 wm + 8 mi + g, columns 64 wn + 8 ni + 2 tig + {0, 1}
  const bool split = gridDim.z > 1;
  double* out = split ? partial + (int64_t)blockIdx.z * M * N : C;
  const int64_t ldo = split ? N : ldc;
  const bool vec_o = split ? (((N & 1) == 0) && ((reinterpret_cast<uintptr_t>(partial) & 15) == 0)) : (vec_c != 0);
#pragma unroll
  for (int mi = 0; mi < 4; ++mi) {
    const int64_t row = m0 + 32 * wm + 8 * mi + g;
    if (row >= M) continue;
#pragma unroll
    for (int ni = 0; ni < 8; ++ni) {
      const int64_t col = n0 + 64 * wn + 8 * ni + 2 * tig;
      if (col >= N) continue;
      double v0 = acc[(mi * 8 + ni) * 2], v1 = acc[(mi * 8 + ni) * 2 + 1];
      double* p = out + row * ldo + col;
      const bool two = col + 1 < N;
      if (!split) {
        v0 *= alpha; v1 *= alpha;
        if (beta != 0.0) {
          v0 = fma(beta, p[0], v0);
          if (two) v1 = fma(beta, p[1], v1);
        }
      }
      if (two && vec_o) *reinterpret_cast<double2*>(p) = make_double2(v0, v1);
      else { p[0] = v0; if (two) p[1] = v1; }
    }
  }
}

// C = alpha * (sum of the partial products, in split order) + beta * C
__global__ void __launch_bounds__(256)
k_splitk_reduce(const double* __restrict__ partial, int nsplit, int64_t M, int64_t N, double alpha, double beta,
                double* __restrict__ C, int64_t ldc, const int* __restrict__ skip) {
  if (skip && *skip) return;
  const int64_t total = M * N;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    double s = 0.0;
    for (int z = 0; z < nsplit; ++z) s += partial[(int64_t)z * total + i];
    double* p = C + (i / N) * ldc + (i % N);
    s *= alpha;
    if (beta != 0.0) s = fma(beta, *p, s);
    *p = s;
  }
}

inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }

template <typename T> inline bool vec_ok(const T* p, int64_t ld) {
  return ((reinterpret_cast<uintptr_t>(p) % (2 * sizeof(T))) == 0) && ((ld & 1) == 0);
}

template <typename TA, typename TB>
cudaError_t launch(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const TA* A, int64_t lda,
                   const TB* B, int64_t ldb, double beta, double* C, int64_t ldc, int nsplit, double* partial,
                   const int* skip, cudaStream_t s) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  static bool attr_set[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(k_dgemm<TA, TB>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  if (nsplit < 1 || !partial) nsplit = 1;
  int64_t k_per_split = cdiv(cdiv(K, nsplit), BK) * BK;
  if (k_per_split < BK) k_per_split = BK;
  nsplit = (int)cdiv(K > 0 ? K : 1, k_per_split);
  dim3 grid((unsigned)cdiv(N, BN), (unsigned)cdiv(M, BM), (unsigned)nsplit);
  k_dgemm<TA, TB><<<grid, 256, SMEM_BYTES, s>>>(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc,
                                                vec_ok(A, lda) ? 1 : 0, vec_ok(B, ldb) ? 1 : 0,
                                                vec_ok(C, ldc) ? 1 : 0, k_per_split, partial, skip);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (nsplit > 1) {
    const int64_t total = M * N;
    const int64_t blocks = cdiv(total, 256);
    k_splitk_reduce<<<(unsigned)(blocks < 1184 ? blocks : 1184), 256, 0, s>>>(partial, nsplit, M, N, alpha, beta, C, ldc, skip);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace

cudaError_t sdgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const float* A,
                   int64_t lda, const float* B, int64_t ldb, double beta, double* C, int64_t ldc,
                   cudaStream_t s) {
  return launch<float, float>(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, 1, nullptr, nullptr, s);
}

cudaError_t fdgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const float* A,
                   int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                   cudaStream_t s) {
  return launch<float, double>(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, 1, nullptr, nullptr, s);
}

cudaError_t dgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const double* A,
                  int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                  cudaStream_t s) {
  return launch<double, double>(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, 1, nullptr, nullptr, s);
}

cudaError_t dgemm_ex(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const double* A,
                     int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                     int nsplit, double* partial, const int* skip, cudaStream_t s) {
  return launch<double, double>(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, nsplit, partial, skip, s);
}

}  // namespace br
