// SIMT (FFMA) contractions: the accurate fp32 path.  Used for BR_GEMM_FP32 and for layers whose
// shapes the tensor-core tiles do not take.  (The fp64 contractions of the basis refresh live in
// dgemm.cu.)
//
// C = alpha * op(A) op(B) + beta * C, all row-major.  op(A) is M x K, op(B) is K x N.
#include "br_internal.h"
#include "step_tc.h"

namespace br {
namespace {

template <typename TA, typename TB, typename TC, int BM, int BN, int BK, int TM, int TN>
__global__ void __launch_bounds__((BM / TM) * (BN / TN))
k_gemm(int ta, int tb, int64_t M, int64_t N, int64_t K, TC alpha, const TA* __restrict__ A,
       int64_t lda, const TB* __restrict__ B, int64_t ldb, TC beta, TC* __restrict__ C,
       int64_t ldc) {
  constexpr int NT = (BM / TM) * (BN / TN);
  constexpr int PAD = 4;
  __shared__ TC As[BK][BM + PAD];
  __shared__ TC Bs[BK][BN + PAD];

  const int t = threadIdx.x;
  const int tx = t % (BN / TN), ty = t / (BN / TN);
  const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;

  TC acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = TC(0);

  for (int64_t k0 = 0; k0 < K; k0 += BK) {
    // ---- stage op(A)[m0:m0+BM, k0:k0+BK] as As[kk][i] --------------------------------------
#pragma unroll 1
    for (int idx = t; idx < BM * BK; idx += NT) {
      int i, kk;
      if (ta) { i = idx % BM; kk = idx / BM; } else { kk = idx % BK; i = idx / BK; }
      const int64_t gm = m0 + i, gk = k0 + kk;
      TC v = TC(0);
      if (gm < M && gk < K) v = (TC)(ta ? A[gk * lda + gm] : A[gm * lda + gk]);
      As[kk][i] = v;
    }
    // ---- stage op(B)[k0:k0+BK, n0:n0+BN] as Bs[kk][j] --------------------------------------
#pragma unroll 1
    for (int idx = t; idx < BN * BK; idx += NT) {
      int j, kk;
      if (tb) { kk = idx % BK; j = idx / BK; } else { j = idx % BN; kk = idx / BN; }
      const int64_t gn = n0 + j, gk = k0 + kk;
      TC v = TC(0);
      if (gn < N && gk < K) v = (TC)(tb ? B[gn * ldb + gk] : B[gk * ldb + gn]);
      Bs[kk][j] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      TC a[TM], b[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
      for (int j = 0; j < TN; ++j) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t gm = m0 + ty * TM + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int64_t gn = n0 + tx * TN + j;
      if (gn >= N) continue;
      TC* p = C + gm * ldc + gn;
      TC v = alpha * acc[i][j];
      if (beta != TC(0)) v = fma(beta, *p, v);
      *p = v;
    }
  }
}

template <typename TA, typename TB, typename TC>
cudaError_t launch(int ta, int tb, int64_t M, int64_t N, int64_t K, TC alpha, const TA* A,
                   int64_t lda, const TB* B, int64_t ldb, TC beta, TC* C, int64_t ldc,
                   cudaStream_t s) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  const int64_t tiles_big = ((M + 127) / 128) * ((N + 127) / 128);
  if (tiles_big >= 148) {
    dim3 grid((unsigned)((N + 127) / 128), (unsigned)((M + 127) / 128));
    k_gemm<TA, TB, TC, 128, 128, 8, 8, 8><<<grid, 256, 0, s>>>(ta, tb, M, N, K, alpha, A, lda, B, ldb,
                                                              beta, C, ldc);
  } else {
    dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64));
    k_gemm<TA, TB, TC, 64, 64, 16, 4, 4><<<grid, 256, 0, s>>>(ta, tb, M, N, K, alpha, A, lda, B, ldb,
                                                             beta, C, ldc);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t sgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, float alpha, const float* A,
                  int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                  cudaStream_t s) {
  return launch<float, float, float>(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, s);
}

}  // namespace br
