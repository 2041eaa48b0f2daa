// Fused element-wise kernels of the rotated Adam step.  All are HBM-bound: one pass over the
// data, 128-bit accesses on the aligned body, grid-stride loops on a grid sized as a multiple of
// the SM count.
#include "br_internal.h"

namespace br {

namespace {

constexpr int kThreads = 256;

template <int NSEG>
struct ClipSegs {                 // passed by value: one launch covers up to NSEG gradients
  const void* ptr[NSEG];
  long long begin[NSEG + 1];      // element offsets in the concatenation
  int bf16[NSEG];
};

inline int grid_for(int64_t n_vec) {
  // 148 SMs on a B200, 8 resident CTAs of 256 threads each.
  int64_t want = (n_vec + kThreads - 1) / kThreads;
  int64_t cap = 148 * 8;
  if (want < 1) want = 1;
  return (int)(want < cap ? want : cap);
}

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }

__device__ __forceinline__ float4 ld4_bf16(const __nv_bfloat16* p) {
  uint2 raw = *reinterpret_cast<const uint2*>(p);
  float4 r;
  r.x = __uint_as_float(raw.x << 16);
  r.y = __uint_as_float(raw.x & 0xFFFF0000u);
  r.z = __uint_as_float(raw.y << 16);
  r.w = __uint_as_float(raw.y & 0xFFFF0000u);
  return r;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ void st4_bf16(__nv_bfloat16* p, float4 v) {
  uint2 raw;
  raw.x = pack_bf16(v.x, v.y);
  raw.y = pack_bf16(v.z, v.w);
  *reinterpret_cast<uint2*>(p) = raw;
}

__device__ __forceinline__ float bf16_round(float x) {
  return __bfloat162float(__float2bfloat16_rn(x));
}

template <bool G_BF16>
__device__ __forceinline__ float4 load_grad4(const void* G, int64_t i) {
  if (G_BF16) return ld4_bf16(reinterpret_cast<const __nv_bfloat16*>(G) + i);
  return ld4(reinterpret_cast<const float*>(G) + i);
}
template <bool G_BF16>
__device__ __forceinline__ float load_grad1(const void* G, int64_t i) {
  if (G_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(G)[i]);
  return reinterpret_cast<const float*>(G)[i];
}

__global__ void k_set_identity(float* Q, int64_t k) {
  int64_t n = k * k;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    Q[i] = (i / k == i % k) ? 1.0f : 0.0f;
  }
}

template <bool G_BF16>
__global__ void __launch_bounds__(kThreads)
k_ema_momentum(float* __restrict__ M, const void* __restrict__ G, int64_t numel, float beta1,
               float* __restrict__ Gf32, __nv_bfloat16* __restrict__ Mh,
               __nv_bfloat16* __restrict__ Ml, const float* __restrict__ gscale) {
  const float gs = gscale ? *gscale : 1.0f;     // clipping factor of the call this gradient came with
  const float omb = 1.0f - beta1;
  const int64_t nvec = numel >> 2;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const int64_t i = v << 2;
    float4 g = load_grad4<G_BF16>(G, i);
    g.x *= gs; g.y *= gs; g.z *= gs; g.w *= gs;
    float4 m = ld4(M + i);
    m.x = beta1 * m.x + omb * g.x;
    m.y = beta1 * m.y + omb * g.y;
    m.z = beta1 * m.z + omb * g.z;
    m.w = beta1 * m.w + omb * g.w;
    st4(M + i, m);
    if (Gf32) st4(Gf32 + i, g);
    if (Mh) {
      float4 h = make_float4(bf16_round(m.x), bf16_round(m.y), bf16_round(m.z), bf16_round(m.w));
      st4_bf16(Mh + i, h);
      if (Ml) st4_bf16(Ml + i, make_float4(m.x - h.x, m.y - h.y, m.z - h.z, m.w - h.w));
    }
  }
  // ragged tail (numel not a multiple of 4)
  for (int64_t i = (nvec << 2) + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel;
       i += stride) {
    float g = gs * load_grad1<G_BF16>(G, i);
    float m = beta1 * M[i] + omb * g;
    M[i] = m;
    if (Gf32) Gf32[i] = g;
    if (Mh) {
      float h = bf16_round(m);
      Mh[i] = __float2bfloat16_rn(m);
      if (Ml) Ml[i] = __float2bfloat16_rn(m - h);
    }
  }
}

template <bool G_BF16>
__global__ void __launch_bounds__(kThreads)
k_plain_adam(float* __restrict__ W, float* __restrict__ M, float* __restrict__ V,
             const void* __restrict__ G, int64_t numel, float lr, float beta1, float beta2,
             float eps, float decay, const float* __restrict__ gscale) {
  const float gs = gscale ? *gscale : 1.0f;
  const float omb1 = 1.0f - beta1, omb2 = 1.0f - beta2;
  const int64_t nvec = numel >> 2;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const int64_t i = v << 2;
    float4 g = load_grad4<G_BF16>(G, i);
    g.x *= gs; g.y *= gs; g.z *= gs; g.w *= gs;
    float4 m = ld4(M + i), s = ld4(V + i), w = ld4(W + i);
#define BR_ADAM1(c)                                   \
  m.c = beta1 * m.c + omb1 * g.c;                     \
  s.c = beta2 * s.c + omb2 * g.c * g.c;               \
  w.c = decay * w.c - lr * (m.c / sqrtf(s.c + eps));
    BR_ADAM1(x) BR_ADAM1(y) BR_ADAM1(z) BR_ADAM1(w)
#undef BR_ADAM1
    st4(M + i, m);
    st4(V + i, s);
    st4(W + i, w);
  }
  for (int64_t i = (nvec << 2) + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel;
       i += stride) {
    float g = gs * load_grad1<G_BF16>(G, i);
    float m = beta1 * M[i] + omb1 * g;
    float s = beta2 * V[i] + omb2 * g * g;
    M[i] = m;
    V[i] = s;
    W[i] = decay * W[i] - lr * (m / sqrtf(s + eps));
  }
}

__global__ void __launch_bounds__(kThreads)
k_second_moment_scale(float* __restrict__ V2, const float* __restrict__ Gt, float* __restrict__ Mt,
                      int64_t numel, float beta2, float eps) {
  const float omb2 = 1.0f - beta2;
  const int64_t nvec = numel >> 2;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const int64_t i = v << 2;
    float4 g = ld4(Gt + i), s = ld4(V2 + i), m = ld4(Mt + i);
    s.x = beta2 * s.x + omb2 * g.x * g.x;  m.x = m.x / sqrtf(s.x + eps);
    s.y = beta2 * s.y + omb2 * g.y * g.y;  m.y = m.y / sqrtf(s.y + eps);
    s.z = beta2 * s.z + omb2 * g.z * g.z;  m.z = m.z / sqrtf(s.z + eps);
    s.w = beta2 * s.w + omb2 * g.w * g.w;  m.w = m.w / sqrtf(s.w + eps);
    st4(V2 + i, s);
    st4(Mt + i, m);
  }
  for (int64_t i = (nvec << 2) + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel;
       i += stride) {
    float g = Gt[i];
    float s = beta2 * V2[i] + omb2 * g * g;
    V2[i] = s;
    Mt[i] = Mt[i] / sqrtf(s + eps);
  }
}

__global__ void __launch_bounds__(kThreads)
k_split_bf16(const float* __restrict__ X, __nv_bfloat16* __restrict__ hi,
             __nv_bfloat16* __restrict__ lo, int64_t numel) {
  const int64_t nvec = numel >> 2;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const int64_t i = v << 2;
    float4 x = ld4(X + i);
    float4 h = make_float4(bf16_round(x.x), bf16_round(x.y), bf16_round(x.z), bf16_round(x.w));
    st4_bf16(hi + i, h);
    if (lo) st4_bf16(lo + i, make_float4(x.x - h.x, x.y - h.y, x.z - h.z, x.w - h.w));
  }
  for (int64_t i = (nvec << 2) + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel;
       i += stride) {
    float x = X[i], h = bf16_round(x);
    hi[i] = __float2bfloat16_rn(x);
    if (lo) lo[i] = __float2bfloat16_rn(x - h);
  }
}

__global__ void __launch_bounds__(kThreads)
k_widen_bf16(const __nv_bfloat16* __restrict__ X, float* __restrict__ out, int64_t numel) {
  const int64_t nvec = numel >> 2;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const int64_t i = v << 2;
    st4(out + i, ld4_bf16(X + i));
  }
  for (int64_t i = (nvec << 2) + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel;
       i += stride)
    out[i] = __bfloat162float(X[i]);
}

// out <- beta1 M + (1-beta1) G, M untouched (M_t for a refresh that reads the momentum)
template <bool G_BF16>
__global__ void __launch_bounds__(kThreads)
k_ema_out(float* __restrict__ out, const float* __restrict__ M, const void* __restrict__ G, int64_t numel,
          float beta1, const float* __restrict__ gscale) {
  const float omb = (1.0f - beta1) * (gscale ? *gscale : 1.0f);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t nvec = numel >> 2;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const int64_t i = v << 2;
    const float4 g = load_grad4<G_BF16>(G, i);
    float4 m = ld4(M + i);
    m.x = beta1 * m.x + omb * g.x; m.y = beta1 * m.y + omb * g.y;
    m.z = beta1 * m.z + omb * g.z; m.w = beta1 * m.w + omb * g.w;
    st4(out + i, m);
  }
  for (int64_t i = (nvec << 2) + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel; i += stride)
    out[i] = beta1 * M[i] + omb * load_grad1<G_BF16>(G, i);
}

// Global-norm clipping factor of one call (App. D.2): sum of squares over all layers' gradients in a
// fixed order (each CTA a contiguous share of the concatenated gradients, tree inside the CTA, then one
// thread over the CTAs), then factor = min(1, clip / norm).
template <int NSEG>
__global__ void __launch_bounds__(kThreads)
k_clip_partial(ClipSegs<NSEG> segs, int nseg, double* __restrict__ part) {
  __shared__ double sh[kThreads];
  const long long total = segs.begin[nseg];
  const long long chunk = (total + gridDim.x - 1) / gridDim.x;
  const long long lo = (long long)blockIdx.x * chunk;
  const long long hi = lo + chunk < total ? lo + chunk : total;
  double acc = 0.0;
  int sg = 0;
  while (sg < nseg && segs.begin[sg + 1] <= lo) ++sg;
  for (; sg < nseg && segs.begin[sg] < hi; ++sg) {
    const long long a = (lo > segs.begin[sg] ? lo : segs.begin[sg]) - segs.begin[sg];
    const long long b = (hi < segs.begin[sg + 1] ? hi : segs.begin[sg + 1]) - segs.begin[sg];
    if (segs.bf16[sg]) {
      const __nv_bfloat16* g = reinterpret_cast<const __nv_bfloat16*>(segs.ptr[sg]);
      for (long long i = a + threadIdx.x; i < b; i += kThreads) { const float v = __bfloat162float(g[i]); acc = fma((double)v, (double)v, acc); }
    } else {
      const float* g = reinterpret_cast<const float*>(segs.ptr[sg]);
      for (long long i = a + threadIdx.x; i < b; i += kThreads) { const float v = g[i]; acc = fma((double)v, (double)v, acc); }
    }
  }
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int w = kThreads / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) part[blockIdx.x] = sh[0];
}
__global__ void k_clip_final(const double* __restrict__ part, int n, float clip, float* __restrict__ out) {
  double s = 0.0;
  for (int i = 0; i < n; ++i) s += part[i];
  const double nrm = sqrt(s);
  *out = (nrm > (double)clip) ? (float)((double)clip / nrm) : 1.0f;
}

// x (rounded to fp32) = p1 + p2 + p3 with three bf16 terms: all 24 significant bits survive.
__device__ __forceinline__ void split3(float f, __nv_bfloat16& p1, __nv_bfloat16& p2, __nv_bfloat16& p3) {
  const float h1 = bf16_round(f);
  const float r1 = f - h1;
  const float h2 = bf16_round(r1);
  const float r2 = r1 - h2;
  p1 = __float2bfloat16_rn(h1); p2 = __float2bfloat16_rn(h2); p3 = __float2bfloat16_rn(r2);
}

// X: rows x cols block of a row-major fp64 matrix with leading dimension ld -> three compact
// (ld = cols) bf16 planes
__global__ void __launch_bounds__(kThreads)
k_split3_f64(const double* __restrict__ X, int64_t ld, int64_t rows, int64_t cols, __nv_bfloat16* __restrict__ p1,
             __nv_bfloat16* __restrict__ p2, __nv_bfloat16* __restrict__ p3) {
  const int64_t total = rows * cols;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / cols, c = i - r * cols;
    split3((float)X[r * ld + c], p1[i], p2[i], p3[i]);
  }
}

__global__ void __launch_bounds__(kThreads)
k_split3_f32(const float* __restrict__ X, int64_t numel, __nv_bfloat16* __restrict__ p1,
             __nv_bfloat16* __restrict__ p2, __nv_bfloat16* __restrict__ p3) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel; i += (int64_t)gridDim.x * blockDim.x)
    split3(X[i], p1[i], p2[i], p3[i]);
}

// A (fp64, leading dimension ld) -= D (fp32, compact rows x cols)
__global__ void __launch_bounds__(kThreads)
k_sub_f32_from_f64(double* __restrict__ A, int64_t ld, int64_t rows, int64_t cols, const float* __restrict__ D) {
  const int64_t total = rows * cols;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / cols, c = i - r * cols;
    A[r * ld + c] -= (double)D[i];
  }
}

__global__ void __launch_bounds__(kThreads)
k_f32_to_f64(const float* __restrict__ X, double* __restrict__ out, int64_t numel) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel; i += stride)
    out[i] = (double)X[i];
}

__global__ void __launch_bounds__(kThreads)
k_f64_to_f32(const double* __restrict__ X, float* __restrict__ out, int64_t numel) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < numel; i += stride)
    out[i] = (float)X[i];
}

}  // namespace

cudaError_t set_identity(float* Q, int64_t k, cudaStream_t s) {
  k_set_identity<<<grid_for(k * k), kThreads, 0, s>>>(Q, k);
  return cudaGetLastError();
}

cudaError_t ema_momentum(float* M, const void* G, int g_is_bf16, int64_t numel, float beta1,
                         float* Gf32, __nv_bfloat16* Mh, __nv_bfloat16* Ml, const float* gscale, cudaStream_t s) {
  int grid = grid_for((numel + 3) / 4);
  if (g_is_bf16)
    k_ema_momentum<true><<<grid, kThreads, 0, s>>>(M, G, numel, beta1, Gf32, Mh, Ml, gscale);
  else
    k_ema_momentum<false><<<grid, kThreads, 0, s>>>(M, G, numel, beta1, Gf32, Mh, Ml, gscale);
  return cudaGetLastError();
}

cudaError_t plain_adam(float* W, float* M, float* V, const void* G, int g_is_bf16, int64_t numel,
                       float lr, float beta1, float beta2, float eps, float wd, const float* gscale, cudaStream_t s) {
  int grid = grid_for((numel + 3) / 4);
  float decay = 1.0f - lr * wd;
  if (g_is_bf16)
    k_plain_adam<true><<<grid, kThreads, 0, s>>>(W, M, V, G, numel, lr, beta1, beta2, eps, decay, gscale);
  else
    k_plain_adam<false><<<grid, kThreads, 0, s>>>(W, M, V, G, numel, lr, beta1, beta2, eps, decay, gscale);
  return cudaGetLastError();
}

cudaError_t second_moment_scale(float* V2, const float* Gt, float* Mt, int64_t numel, float beta2,
                                float eps, cudaStream_t s) {
  k_second_moment_scale<<<grid_for((numel + 3) / 4), kThreads, 0, s>>>(V2, Gt, Mt, numel, beta2, eps);
  return cudaGetLastError();
}

cudaError_t split_bf16(const float* X, __nv_bfloat16* hi, __nv_bfloat16* lo, int64_t numel,
                       cudaStream_t s) {
  k_split_bf16<<<grid_for((numel + 3) / 4), kThreads, 0, s>>>(X, hi, lo, numel);
  return cudaGetLastError();
}

cudaError_t widen_bf16(const __nv_bfloat16* X, float* out, int64_t numel, cudaStream_t s) {
  k_widen_bf16<<<grid_for((numel + 3) / 4), kThreads, 0, s>>>(X, out, numel);
  return cudaGetLastError();
}

cudaError_t ema_out(float* out, const float* M, const void* G, int g_is_bf16, int64_t numel, float beta1,
                    const float* gscale, cudaStream_t s) {
  const int grid = grid_for((numel + 3) / 4);
  if (g_is_bf16) k_ema_out<true><<<grid, kThreads, 0, s>>>(out, M, G, numel, beta1, gscale);
  else k_ema_out<false><<<grid, kThreads, 0, s>>>(out, M, G, numel, beta1, gscale);
  return cudaGetLastError();
}

cudaError_t clip_factor(const void* const* grads, const int64_t* numel, const int* is_bf16, int n, float clip,
                        double* part, float* out, cudaStream_t s) {
  constexpr int NSEG = 64, GRID = 296;
  int launches = 0;
  for (int first = 0; first < n; first += NSEG, ++launches) {
    ClipSegs<NSEG> segs;
    const int cnt = (n - first < NSEG) ? n - first : NSEG;
    segs.begin[0] = 0;
    for (int i = 0; i < cnt; ++i) {
      segs.ptr[i] = grads[first + i];
      segs.bf16[i] = is_bf16[first + i];
      segs.begin[i + 1] = segs.begin[i] + numel[first + i];
    }
    k_clip_partial<NSEG><<<GRID, kThreads, 0, s>>>(segs, cnt, part + (size_t)launches * GRID);
  }
  k_clip_final<<<1, 1, 0, s>>>(part, launches * GRID, clip, out);
  return cudaGetLastError();
}

cudaError_t split3_f64(const double* X, int64_t ld, int64_t rows, int64_t cols, __nv_bfloat16* p1,
                       __nv_bfloat16* p2, __nv_bfloat16* p3, cudaStream_t s) {
  k_split3_f64<<<grid_for(rows * cols), kThreads, 0, s>>>(X, ld, rows, cols, p1, p2, p3);
  return cudaGetLastError();
}

cudaError_t split3_f32(const float* X, int64_t numel, __nv_bfloat16* p1, __nv_bfloat16* p2, __nv_bfloat16* p3,
                       cudaStream_t s) {
  k_split3_f32<<<grid_for(numel), kThreads, 0, s>>>(X, numel, p1, p2, p3);
  return cudaGetLastError();
}

cudaError_t sub_f32_from_f64(double* A, int64_t ld, int64_t rows, int64_t cols, const float* D, cudaStream_t s) {
  k_sub_f32_from_f64<<<grid_for(rows * cols), kThreads, 0, s>>>(A, ld, rows, cols, D);
  return cudaGetLastError();
}

cudaError_t f32_to_f64(const float* X, double* out, int64_t numel, cudaStream_t s) {
  k_f32_to_f64<<<grid_for(numel), kThreads, 0, s>>>(X, out, numel);
  return cudaGetLastError();
}

cudaError_t f64_to_f32(const double* X, float* out, int64_t numel, cudaStream_t s) {
  k_f64_to_f32<<<grid_for(numel), kThreads, 0, s>>>(X, out, numel);
  return cudaGetLastError();
}

// ---- debug canaries: 256-byte guard words behind every piece of the handle's slab ----
namespace {
constexpr unsigned int kGuardWord = 0xC5C5C5C5u;
__global__ void k_guard_fill(char* slab, const unsigned long long* offs, int n) {
  const int g = blockIdx.x;
  if (g < n) reinterpret_cast<unsigned int*>(slab + offs[g])[threadIdx.x] = kGuardWord;
}
__global__ void k_guard_check(const char* slab, const unsigned long long* offs, int n, int* first_bad) {
  const int g = blockIdx.x;
  if (g < n && reinterpret_cast<const unsigned int*>(slab + offs[g])[threadIdx.x] != kGuardWord) atomicMin(first_bad, g);
}
}  // namespace

cudaError_t guard_fill(char* slab, const unsigned long long* offs, int n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  k_guard_fill<<<n, 64, 0, s>>>(slab, offs, n);
  return cudaGetLastError();
}
cudaError_t guard_check(const char* slab, const unsigned long long* offs, int n, int* first_bad, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  k_guard_check<<<n, 64, 0, s>>>(slab, offs, n, first_bad);
  return cudaGetLastError();
}

}  // namespace br
