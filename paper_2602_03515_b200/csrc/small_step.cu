// One rotated-Adam update of a small weight matrix (both dimensions at most 128) in a single launch of
// a single CTA: Alg. 1 (momentum, rotation, second moment, weight update) and the factor EMAs of Alg. 2, with every operand staged in
// shared memory and fp32 FFMA dot products.  A matrix of this size is bound by launch latency, not by
// arithmetic: the general fp32 path takes about fifteen launches per update (momentum EMA, two factor
// products, four rotations, the element-wise second-moment step, two back rotations, copies), this
// kernel one.  The refresh of the bases (Alg. 1 (periodic refresh)) is not part of it: a call on which a refresh
// is due goes through the general path.
#include "br_internal.h"

namespace br {
namespace {

constexpr int kThreads = 512;

struct SmallArgs {
  int m, n;
  int left, right;          // which sides are rotated
  int g_is_bf16;
  int accumulate;           // 1: update L and R in this call
  const void* G;
  const float* gscale;      // clipping factor of the gradient's call, or null
  float *M, *V2, *U, *V, *L, *R, *W;
  float lr, beta1, beta2, eps, decay, beta_factor;
};

__device__ __forceinline__ float load_g(const void* G, int g_is_bf16, int i) {
  return g_is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(G)[i]) : reinterpret_cast<const float*>(G)[i];
}

__global__ void __launch_bounds__(kThreads) k_small_step(SmallArgs a) {
  extern __shared__ float sm[];
  const int m = a.m, n = a.n, mn = m * n;
  // rows are padded by one word: a column walk (threads that differ in the row index) then touches
  // 32 different banks instead of one
  const int ln = n + 1, lm = m + 1;
  float* sG = sm;                 // G, later X
  float* sM = sG + m * ln;        // M, later Y
  float* sT1 = sM + m * ln;       // first-side product of G
  float* sT2 = sT1 + m * ln;      // first-side product of M
  float* sU = sT2 + m * ln;       // m x m (left side rotated)
  float* sV = sU + (a.left ? m * lm : 0);
  const int t = threadIdx.x;
  const float gs = a.gscale ? *a.gscale : 1.0f;
  // Alg. 1 (momentum update): M <- beta1 M + (1 - beta1) G
  for (int i = t; i < mn; i += kThreads) {
    const float g = gs * load_g(a.G, a.g_is_bf16, i);
    const float mo = a.beta1 * a.M[i] + (1.0f - a.beta1) * g;
    const int r = i / n, c = i % n;
    sG[r * ln + c] = g; sM[r * ln + c] = mo; a.M[i] = mo;
  }
  if (a.left) for (int i = t; i < m * m; i += kThreads) sU[(i / m) * lm + i % m] = a.U[i];
  if (a.right) for (int i = t; i < n * n; i += kThreads) sV[(i / n) * ln + i % n] = a.V[i];
  __syncthreads();
  // Alg. 2: L <- b L + (1 - b) G G^T ; R <- b R + (1 - b) G^T G
  if (a.accumulate) {
    const float b = a.beta_factor, ob = 1.0f - a.beta_factor;
    if (a.L)
      for (int e = t; e < m * m; e += kThreads) {
        const int i = e / m, j = e % m;
        float s = 0.f;
        for (int k = 0; k < n; ++k) s = fmaf(sG[i * ln + k], sG[j * ln + k], s);
        a.L[e] = b * a.L[e] + ob * s;
      }
    if (a.R)
      for (int e = t; e < n * n; e += kThreads) {
        const int i = e / n, j = e % n;
        float s = 0.f;
        for (int k = 0; k < m; ++k) s = fmaf(sG[k * ln + i], sG[k * ln + j], s);
        a.R[e] = b * a.R[e] + ob * s;
      }
  }
  // Alg. 1 (rotation of G and M), first side: T1 = U^T G, T2 = U^T M (or the matrices themselves)
  for (int e = t; e < mn; e += kThreads) {
    const int i = e / n, j = e % n;
    float s1 = sG[i * ln + j], s2 = sM[i * ln + j];
    if (a.left) {
      s1 = 0.f; s2 = 0.f;
      for (int k = 0; k < m; ++k) { const float u = sU[k * lm + i]; s1 = fmaf(u, sG[k * ln + j], s1); s2 = fmaf(u, sM[k * ln + j], s2); }
    }
    sT1[i * ln + j] = s1; sT2[i * ln + j] = s2;
  }
  __syncthreads();
  // second side: G~ = T1 V, M~ = T2 V; then the second moment and the scaling: V~ <- beta2 V~ + (1 - beta2) G~^2, X = M~ / sqrt(V~ + eps)
  for (int e = t; e < mn; e += kThreads) {
    const int i = e / n, j = e % n;
    float gt = sT1[i * ln + j], mt = sT2[i * ln + j];
    if (a.right) {
      gt = 0.f; mt = 0.f;
      for (int k = 0; k < n; ++k) { const float v = sV[k * ln + j]; gt = fmaf(sT1[i * ln + k], v, gt); mt = fmaf(sT2[i * ln + k], v, mt); }
    }
    const float v2 = a.beta2 * a.V2[e] + (1.0f - a.beta2) * gt * gt;
    a.V2[e] = v2;
    sG[i * ln + j] = mt / sqrtf(v2 + a.eps);        // X (G is not needed any more)
  }
  __syncthreads();
  // weight update: W <- decay W - eta U X V^T
  for (int e = t; e < mn; e += kThreads) {
    const int i = e / n, j = e % n;
    float y = sG[i * ln + j];
    if (a.left) {
      y = 0.f;
      for (int k = 0; k < m; ++k) y = fmaf(sU[i * lm + k], sG[k * ln + j], y);
    }
    sM[i * ln + j] = y;                     // Y = U X
  }
  __syncthreads();
  for (int e = t; e < mn; e += kThreads) {
    const int i = e / n, j = e % n;
    float d = sM[i * ln + j];
    if (a.right) {
      d = 0.f;
      for (int k = 0; k < n; ++k) d = fmaf(sM[i * ln + k], sV[j * ln + k], d);
    }
    a.W[e] = a.decay * a.W[e] - a.lr * d;
  }
}

size_t small_bytes(int64_t m, int64_t n, bool left, bool right) {
  return sizeof(float) * (size_t)(4 * m * (n + 1) + (left ? m * (m + 1) : 0) + (right ? n * (n + 1) : 0));
}

}  // namespace

bool small_step_eligible(int64_t m, int64_t n, bool left, bool right) {
  return (left || right) && m <= 128 && n <= 128 && small_bytes(m, n, left, right) <= 160 * 1024;
}

cudaError_t small_step(int64_t m, int64_t n, bool left, bool right, const void* G, int g_is_bf16, const float* gscale,
                       float* M, float* V2, float* U, float* V, float* L, float* R, float* W, int accumulate, float lr,
                       float beta1, float beta2, float eps, float weight_decay, float beta_factor, cudaStream_t s) {
  SmallArgs a;
  a.m = (int)m; a.n = (int)n; a.left = left; a.right = right; a.g_is_bf16 = g_is_bf16; a.accumulate = accumulate;
  a.G = G; a.gscale = gscale; a.M = M; a.V2 = V2; a.U = U; a.V = V; a.L = L; a.R = R; a.W = W;
  a.lr = lr; a.beta1 = beta1; a.beta2 = beta2; a.eps = eps; a.decay = 1.0f - lr * weight_decay; a.beta_factor = beta_factor;
  const size_t bytes = small_bytes(m, n, left, right);
  static bool attr_set[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(k_small_step, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  k_small_step<<<1, kThreads, bytes, s>>>(a);
  return cudaGetLastError();
}

}  // namespace br
