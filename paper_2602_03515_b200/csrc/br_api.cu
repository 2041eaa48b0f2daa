// Host side of libbr: handle, validation, integer state (calls, t, ring slots, refresh schedule),
// memory layout and the launch plan of one delayed rotated-Adam step.  See include/br.h for the
// contract of every entry point.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <string>
#include <vector>

#include "br_internal.h"
#include "step_tc.h"

using namespace br;

namespace {

thread_local std::string g_create_error;

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

}  // namespace

namespace br {

std::string format(const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  return std::string(buf);
}

size_t dtype_size(int dt) { return dt == BR_BF16 ? 2 : 4; }

// Which sides carry a rotation: unilateral rotates the smaller dimension (Sec. 3.2), ties left.
void rotated_sides(int64_t m, int64_t n, int geom, bool* left, bool* right) {
  *left = *right = false;
  if (geom == BR_GEOM_BILATERAL) { *left = *right = true; }
  else if (geom == BR_GEOM_UNILATERAL) { *left = (m <= n); *right = (m > n); }
}

}  // namespace br

// ---------------------------------------------------------------------------------------------
// Validation and memory layout (host only)
// ---------------------------------------------------------------------------------------------
namespace {

br_status validate(const br_layer_desc* layers, int n_layers, const br_hparams* hp, std::string* err) {
  if (!layers || !hp || n_layers <= 0) { *err = "NULL layers/hparams or n_layers <= 0"; return BR_ERR_INVALID; }
  if (!(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f) ||
      !(hp->eps >= 0.f) || !(hp->beta_factor < 1.f) || !std::isfinite(hp->lr) || !(hp->weight_decay >= 0.f)) {
    *err = "hyper-parameter out of range"; return BR_ERR_INVALID;
  }
  if (!(hp->clip_norm >= 0.f) || !std::isfinite(hp->clip_norm)) { *err = "clip_norm must be finite and >= 0"; return BR_ERR_INVALID; }
  if (hp->freq < 1 || hp->power_iters < 1) { *err = "freq and power_iters must be >= 1"; return BR_ERR_INVALID; }
  if (hp->accum != BR_ACCUM_EVERY_STEP && hp->accum != BR_ACCUM_ON_REFRESH) { *err = "bad accum mode"; return BR_ERR_INVALID; }
  if (hp->gemm_prec != BR_GEMM_FP32 && hp->gemm_prec != BR_GEMM_BF16) { *err = "bad gemm_prec"; return BR_ERR_INVALID; }
  if (hp->flags & ~(uint32_t)BR_FLAG_DEBUG_CANARY) { *err = "unknown bit in flags"; return BR_ERR_INVALID; }
  for (int i = 0; i < n_layers; ++i) {
    const br_layer_desc& d = layers[i];
    if (d.m < 1 || d.n < 1 || d.m > (1 << 20) || d.n > (1 << 20)) { *err = format("layer %d: bad shape %lld x %lld", i, (long long)d.m, (long long)d.n); return BR_ERR_SHAPE; }
    if (d.geom < BR_GEOM_NONE || d.geom > BR_GEOM_BILATERAL) { *err = format("layer %d: bad geometry", i); return BR_ERR_INVALID; }
    if (d.geom != BR_GEOM_NONE && d.src != BR_SRC_FIRST && d.src != BR_SRC_SECOND) { *err = format("layer %d: bad source", i); return BR_ERR_INVALID; }
    if (d.grad_dtype != BR_F32 && d.grad_dtype != BR_BF16) { *err = format("layer %d: bad grad dtype", i); return BR_ERR_DTYPE; }
    if (d.tau_max < 0) { *err = format("layer %d: tau_max < 0", i); return BR_ERR_TAU; }
  }
  return BR_OK;
}

struct Sizes {
  size_t total = 0, overhead = 0;
};

}  // namespace

// ---------------------------------------------------------------------------------------------
// Handle
// ---------------------------------------------------------------------------------------------
struct br_handle {
  int device = 0;
  cudaStream_t stream = nullptr;
  br_allocator alloc{};
  br_hparams hp{};
  std::vector<Layer> layers;
  int64_t calls = 0;
  char* slab = nullptr;
  size_t slab_bytes = 0;
  int* d_status = nullptr;
  // scratch of the SIMT path (one layer at a time)
  float *sG = nullptr, *sT = nullptr, *sGt = nullptr, *sMt = nullptr;
  // The refresh runs independent Power() applications (one per layer and side) on a few lanes at
  // once: lane 0 is the handle's own stream, the others are internal streams that wait for the
  // handle's stream before they start and that the handle's stream waits for when they are done.
  // The orthonormalisation is a chain of short dependent launches between large products; with
  // several chains in flight the short ones fill the gaps of the others.
  struct Lane {
    cudaStream_t stream = nullptr;
    cudaEvent_t done = nullptr;
    double *rA = nullptr, *rF = nullptr, *rQ = nullptr, *rZ = nullptr, *rWork = nullptr;
    char* tcq_scratch = nullptr;          // scratch of the tensor-core projections (largest eligible order)
    std::vector<QrTc*> tcq;               // their plans, one per distinct eligible order
    int64_t cap_k = 0;                    // largest order this lane's buffers hold
    // The orthonormalisation of one basis is several hundred dependent launches whose arguments
    // depend only on the lane (its buffers) and on the order: it is captured into a CUDA graph the
    // first time and replayed afterwards, one launch per basis.  Key: 2 * order + (tensor-core form).
    struct QrGraph { cudaGraphExec_t exec = nullptr; int64_t launches = 0; double flops = 0.0; };
    std::map<int64_t, QrGraph> qr_graphs;
    int* cond = nullptr;                  // conditioning note of the lane's current job (device)
  };
  bool use_graphs = true;                 // cleared when a capture fails (BR_REFRESH_GRAPHS=0 switches it off)
  // Up to three lanes hold the largest order; up to five more hold only the small orders (at most
  // 1/sqrt(2) of the largest, S = 2nd), whose refresh is a chain of short launches that leaves most of
  // the GPU idle: eight streams in all, the default number of hardware queues.
  static constexpr int kBigLanes = 3;       // default number of full-size lanes (BR_REFRESH_LANES: 1..6)
  static constexpr int kMaxBigLanes = 6;
  static constexpr int kMaxLanes = 8;       // lanes of both kinds
  Lane lanes[kMaxLanes];
  int n_lanes = 1;
  cudaEvent_t ev_begin = nullptr;
  // The gradients of a call are stored in the ring on a side stream, chunk by chunk, as soon as the
  // launches that read the slots they overwrite are enqueued, so that the copies run beside the rest of
  // the step; the step's stream waits for them before br_step returns control of it.
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_consumed = nullptr, ev_copied = nullptr;
  // Conditioning notes of the last refresh, per layer and side (index 2 * layer + (right side)):
  // written on the device by the refresh, copied to pinned host memory after every batch, read by
  // the host before the next one (which then decides where the block projections run).
  // global-norm clipping: factor of each of the last calls (slot (call - 1) mod clip_slots)
  float* d_clip = nullptr;
  int clip_slots = 0;
  double* d_clip_part = nullptr;
  int* d_cond = nullptr;
  int* h_cond = nullptr;
  std::vector<int> cond_known;
  cudaEvent_t ev_cond = nullptr;
  bool cond_pending = false;
  size_t tcq_bytes = 0;
  // tensor-core path
  TcStep* tc = nullptr;
  // debug canaries (BR_FLAG_DEBUG_CANARY): offsets of the guards in the slab, on the host and on the device
  std::vector<unsigned long long> guard_offsets;
  unsigned long long* d_guard_offsets = nullptr;
  LaunchStats stats;
  std::string err;
};

namespace {

br_status step_enqueue(br_handle* h, const void* const* grads, int tau);
void release(br_handle* h);

struct Bump {
  size_t off = 0;
  char* base = nullptr;
  size_t guard = 0;                                   // debug canaries: bytes of guard behind every piece
  std::vector<unsigned long long>* guards = nullptr;  // their offsets (collected in the pass that has a base)
  template <typename T> T* take(size_t count) {
    size_t o = off;
    off = align_up(off + count * sizeof(T));
    if (guard) {
      if (guards && base) guards->push_back((unsigned long long)off);
      off += guard;
    }
    return base ? reinterpret_cast<T*>(base + o) : nullptr;
  }
};

// Lays out every buffer of the handle in one slab.  With base == nullptr only sizes are computed.
void layout(br_handle* h, Bump& b, Sizes* sz) {
  const br_hparams& hp = h->hp;
  if (hp.flags & BR_FLAG_DEBUG_CANARY) { b.guard = kAlign; b.guards = &h->guard_offsets; h->guard_offsets.clear(); }
  size_t max_numel = 0, max_k = 0, max_z = 0, n_sides = 0;
  bool any_simt = false;
  for (Layer& L : h->layers) {
    const size_t mn = (size_t)L.d.m * L.d.n;
    L.M = b.take<float>(mn);
    if (L.use_tc && L.d.src == BR_SRC_FIRST) L.Morig = b.take<float>(mn);
    L.V2 = b.take<float>(mn);
    const bool second = L.d.src == BR_SRC_SECOND;
    if (L.left) { L.U = b.take<float>((size_t)L.d.m * L.d.m); sz->overhead += 4 * (size_t)L.d.m * L.d.m; }
    if (L.right) { L.V = b.take<float>((size_t)L.d.n * L.d.n); sz->overhead += 4 * (size_t)L.d.n * L.d.n; }
    if (L.left && second) { L.L = b.take<float>((size_t)L.d.m * L.d.m); sz->overhead += 4 * (size_t)L.d.m * L.d.m; }
    if (L.right && second) { L.R = b.take<float>((size_t)L.d.n * L.d.n); sz->overhead += 4 * (size_t)L.d.n * L.d.n; }
    if (L.use_tc) {
      if (L.left) { L.Uh = b.take<__nv_bfloat16>((size_t)L.d.m * L.d.m); L.Ul = b.take<__nv_bfloat16>((size_t)L.d.m * L.d.m); }
      if (L.right) { L.Vh = b.take<__nv_bfloat16>((size_t)L.d.n * L.d.n); L.Vl = b.take<__nv_bfloat16>((size_t)L.d.n * L.d.n); }
    }
    // a tensor-core layer reads its gradient through a tensor map over the ring, so it keeps
    // one slot even without delay
    L.ring_slots = L.d.tau_max > 0 ? L.d.tau_max : (L.use_tc ? 1 : 0);
    if (L.ring_slots > 0) {
      L.slot_stride = align_up(mn * dtype_size(L.d.grad_dtype));
      L.ring = b.take<char>(L.slot_stride * (size_t)L.ring_slots);
    }
    if (L.d.geom != BR_GEOM_NONE) {
      if (!L.use_tc) { any_simt = true; max_numel = std::max(max_numel, mn); }
      if (L.left) { max_k = std::max(max_k, (size_t)L.d.m); ++n_sides; }
      if (L.right) { max_k = std::max(max_k, (size_t)L.d.n); ++n_sides; }
      if (!second) max_z = std::max(max_z, mn);
    }
  }
  if (any_simt) {
    h->sG = b.take<float>(max_numel);
    h->sT = b.take<float>(max_numel);
    h->sGt = b.take<float>(max_numel);
    h->sMt = b.take<float>(max_numel);
  }
  h->tcq_bytes = 0;
  for (const Layer& L : h->layers) {
    if (!L.use_tc) continue;
    if (L.left) h->tcq_bytes = std::max(h->tcq_bytes, qr_tc_scratch_bytes(L.d.m));
    if (L.right) h->tcq_bytes = std::max(h->tcq_bytes, qr_tc_scratch_bytes(L.d.n));
  }
  if (max_k) {
    int want_big = br_handle::kBigLanes;
    // tuning aid: BR_REFRESH_LANES=1..6 sets the number of concurrent full-size refresh lanes
    if (const char* env = std::getenv("BR_REFRESH_LANES")) {
      const int v = std::atoi(env);
      if (v >= 1 && v <= br_handle::kMaxBigLanes) want_big = v;
    }
    int n_big = (int)std::min<size_t>((size_t)want_big, std::max<size_t>(1, n_sides));
    // the small class: orders of S = 2nd sides of at most max_k / sqrt(2)
    size_t small_k = 0, n_small_sides = 0;
    std::vector<size_t> orders;
    for (const Layer& L : h->layers) {
      if (L.d.geom == BR_GEOM_NONE) continue;
      for (size_t k : {L.left ? (size_t)L.d.m : (size_t)0, L.right ? (size_t)L.d.n : (size_t)0}) {
        if (!k) continue;
        orders.push_back(k);
        if (L.d.src == BR_SRC_SECOND && 2 * k * k <= max_k * max_k) { small_k = std::max(small_k, k); ++n_small_sides; }
      }
    }
    int n_small = (int)std::min<size_t>((size_t)(br_handle::kMaxLanes - n_big), n_small_sides);
    if ((int)n_sides <= n_big) n_small = 0;
    // tuning aid: BR_REFRESH_SMALL_LANES=0..5 caps the number of small-order lanes
    if (const char* env = std::getenv("BR_REFRESH_SMALL_LANES")) {
      const int v = std::atoi(env);
      if (v >= 0 && v < n_small) n_small = v;
    }
    h->n_lanes = n_big + n_small;
    for (int i = 0; i < h->n_lanes; ++i) {
      br_handle::Lane& ln = h->lanes[i];
      const bool big = i < n_big;
      const size_t cap = big ? max_k : small_k;
      ln.cap_k = (int64_t)cap;
      ln.rA = b.take<double>(cap * cap);
      ln.rF = b.take<double>(cap * cap);
      ln.rQ = b.take<double>(cap * cap);
      size_t work = 1056;                                  // (also 1025 doubles of norm scratch)
      for (size_t k : orders) if (k <= cap) work = std::max(work, qr_work_doubles((int64_t)k));
      ln.rWork = b.take<double>(work);
      ln.cond = b.take<int>(64);
      if (big && max_z) ln.rZ = b.take<double>(max_z);
      {
        // scratch of the tensor-core projections for the largest eligible order this lane can hold
        size_t tb = 0;
        for (const Layer& L : h->layers) {
          if (!L.use_tc) continue;
          if (L.left && (size_t)L.d.m <= cap) tb = std::max(tb, qr_tc_scratch_bytes(L.d.m));
          if (L.right && (size_t)L.d.n <= cap) tb = std::max(tb, qr_tc_scratch_bytes(L.d.n));
        }
        if (tb) ln.tcq_scratch = b.take<char>(tb);
      }
    }
  }
  h->d_cond = b.take<int>(2 * h->layers.size() + 2);
  if (hp.clip_norm > 0.f) {
    int tmax = 0;
    for (const Layer& L : h->layers) tmax = std::max(tmax, (int)L.d.tau_max);
    h->clip_slots = tmax + 1;
    h->d_clip = b.take<float>((size_t)h->clip_slots);
    h->d_clip_part = b.take<double>(296 * ((h->layers.size() + 63) / 64));
  }
  h->d_status = b.take<int>(64);
  (void)hp;
  sz->total = b.off;
}

void init_layers(br_handle* h, const br_layer_desc* layers, int n_layers) {
  h->layers.resize(n_layers);
  for (int i = 0; i < n_layers; ++i) {
    Layer& L = h->layers[i];
    L = Layer{};
    L.d = layers[i];
    rotated_sides(L.d.m, L.d.n, L.d.geom, &L.left, &L.right);
    L.freq = L.d.freq > 0 ? L.d.freq : h->hp.freq;
    L.use_tc = h->hp.gemm_prec == BR_GEMM_BF16 && L.d.geom != BR_GEOM_NONE &&
               (L.d.m % 8 == 0) && (L.d.n % 8 == 0) && L.d.grad_dtype == BR_BF16;
  }
}

#define BR_CUDA(h, expr)                                                              \
  do {                                                                                \
    cudaError_t e__ = (h)->stats.inject() ? cudaErrorLaunchFailure : (expr);          \
    if (e__ != cudaSuccess) {                                                         \
      (h)->err = format("%s failed: %s", #expr, cudaGetErrorString(e__));             \
      return BR_ERR_CUDA;                                                             \
    }                                                                                 \
  } while (0)

inline void count(br_handle* h, int n = 1) { h->stats.launches += n; }

const void* ring_slot_ptr(const Layer& L, int64_t slot) {
  return L.ring + (size_t)slot * L.slot_stride;
}

// ---- the power product F Q of a tracking basis, mostly on the tensor cores -------------------------
// F Q in fp32-level arithmetic is useless as it stands: the small eigen-directions of F come out of
// a cancellation against eigenvalues up to 1e5 times larger.  But once the basis tracks the factor
// its leading columns U_s (one panel of r = 128) span the dominant directions, and
//   F = F_rest + P F + F P - P F P,   P = U_s U_s^T,   F_rest = (I - P) F (I - P)
// holds for ANY matrix P (it is plain algebra), with F_rest free of the large eigenvalues.  So
//   F Q = F_rest Q + B (U_s^T Q) + U_s (B^T Q - Lam U_s^T Q),   B = F U_s,  Lam = U_s^T B  (F symmetric)
// where the rank-r terms (14 k^2 r flop) and F_rest itself are computed on the fp64 matrix unit
// and only F_rest Q (2 k^3 flop) runs on the tensor cores, on three-term bf16 splits: its error is
// ~2e-7 ||F_rest|| per column, a relative 2e-7 of the small columns instead of 2e-7 * 1e5.
// On entry ln.rF and ln.rQ hold F and Q widened to fp64; on exit ln.rA holds F Q (rF is overwritten).
br_status deflated_power(br_handle* h, br_handle::Lane& ln, QrTc* tcq, int64_t k, cudaStream_t s) {
  const int64_t r = 128, r2 = 2 * r;
  double* w = ln.rWork;                               // the QR work area is free until the QR starts
  double* W1 = w;              w += k * r2;           // k x 2r: [U_s | T1]
  double* W2 = w;              w += k * r2;           // k x 2r: [B | U_s]
  double* C1 = w;              w += r * k;            // r x k
  double* C2 = w;              w += r * k;            // r x k, directly below C1: [C1; C2] is 2r x k
  double* Lam = w;             w += r * r;            // r x r
  double* part = w;                                   // split-K partial sums (at most 54 * r * r, 4 * r * k doubles)
  const int sp_small = (int)std::min<int64_t>(54, std::max<int64_t>(1, k / 128));
  double* F = ln.rF;
  double* Q = ln.rQ;
  const double* Us = Q;                               // first r columns of Q, leading dimension k
  double* B = W2;                                     // leading dimension 2r
  double* T1 = W1 + r;                                // leading dimension 2r
  const size_t rb = sizeof(double) * r, pk = sizeof(double) * k, p2 = sizeof(double) * r2;
  // B = F U_s ; Lam = U_s^T B ; C1 = U_s^T Q ; C2 = B^T Q
  BR_CUDA(h, dgemm(0, 0, k, r, k, 1.0, F, k, Us, k, 0.0, B, r2, s));
  BR_CUDA(h, dgemm_ex(1, 0, r, r, k, 1.0, Us, k, B, r2, 0.0, Lam, r, sp_small, part, nullptr, s));
  BR_CUDA(h, dgemm_ex(1, 0, r, k, k, 1.0, Us, k, Q, k, 0.0, C1, k, 4, part, nullptr, s));
  BR_CUDA(h, dgemm_ex(1, 0, r, k, k, 1.0, B, r2, Q, k, 0.0, C2, k, 4, part, nullptr, s));
  // the two rank-r corrections as one rank-2r product each: W1 = [U_s | T1], W2 = [B | U_s], T1 = B - U_s Lam
  BR_CUDA(h, cudaMemcpy2DAsync(W1, p2, Us, pk, rb, (size_t)k, cudaMemcpyDeviceToDevice, s));
  BR_CUDA(h, cudaMemcpy2DAsync(W2 + r, p2, Us, pk, rb, (size_t)k, cudaMemcpyDeviceToDevice, s));
  BR_CUDA(h, cudaMemcpy2DAsync(T1, p2, B, p2, rb, (size_t)k, cudaMemcpyDeviceToDevice, s));
  BR_CUDA(h, dgemm(0, 0, k, r, r, -1.0, Us, k, Lam, r, 1.0, T1, r2, s));
  // F_rest = F - U_s B^T - T1 U_s^T = F - W1 W2^T
  BR_CUDA(h, dgemm(0, 1, k, k, r2, -1.0, W1, r2, W2, r2, 1.0, F, k, s));
  // F_rest Q on the tensor cores
  const float* Af = nullptr;
  BR_CUDA(h, qr_tc_power(tcq, F, Q, h->d_status, s, &Af));
  // C2 <- C2 - Lam C1 ; A = F_rest Q + B C1 + U_s C2 = F_rest Q + W2 [C1; C2]
  BR_CUDA(h, dgemm(0, 0, r, k, r, -1.0, Lam, r, C1, k, 1.0, C2, k, s));
  BR_CUDA(h, f32_to_f64(Af, ln.rA, k * k, s));
  BR_CUDA(h, dgemm(0, 0, k, k, r2, 1.0, W2, r2, C1, k, 1.0, ln.rA, k, s));
  count(h, 20);
  h->stats.gemm_flops += 14.0 * k * k * r;
  return BR_OK;
}

// A <- qr(A).Q for the product in the lane's buffer; the conditioning note goes to d_cond[ci].
br_status orthonormalise(br_handle* h, br_handle::Lane& ln, int64_t k, QrTc* tcq, int ci, cudaStream_t s) {
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess) { cudaGetLastError(); capturing = cudaStreamCaptureStatusActive; }
  if (h->use_graphs && capturing == cudaStreamCaptureStatusNone) {
    const int64_t key = 2 * k + (tcq ? 1 : 0);
    auto it = ln.qr_graphs.find(key);
    if (it == ln.qr_graphs.end()) {
      br_handle::Lane::QrGraph g;
      cudaGraph_t graph = nullptr;
      cudaError_t e = cudaStreamBeginCapture(s, cudaStreamCaptureModeRelaxed);
      if (e == cudaSuccess) {
        // (the completion of a rank-deficient product is part of the chain as launches that a device flag
        // cancels; as the body of a conditional graph node it made a refresh of 57 bases slower, 354 ms
        // against 324, although a full-rank product then launches nothing of it)
        const cudaError_t qe = qr_pos_inplace(ln.rA, k, ln.rWork, h->d_status, s, &g.launches, &g.flops, tcq, ln.cond, ln.rF, ln.rQ);
        e = cudaStreamEndCapture(s, &graph);          // always ends the capture, also after a failed launch
        if (e == cudaSuccess && qe != cudaSuccess) e = qe;
        if (e == cudaSuccess && graph) e = cudaGraphInstantiate(&g.exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
      }
      if (e != cudaSuccess || !g.exec) {
        cudaGetLastError();
        h->use_graphs = false;                         // nothing was enqueued: run it directly below
      } else {
        it = ln.qr_graphs.emplace(key, g).first;
      }
    }
    if (h->use_graphs) {
      BR_CUDA(h, cudaGraphLaunch(it->second.exec, s));
      h->stats.launches += it->second.launches;
      h->stats.gemm_flops += it->second.flops;
      BR_CUDA(h, cudaMemcpyAsync(h->d_cond + ci, ln.cond, sizeof(int), cudaMemcpyDeviceToDevice, s));
      return BR_OK;
    }
  }
  BR_CUDA(h, qr_pos_inplace(ln.rA, k, ln.rWork, h->d_status, s, &h->stats.launches, &h->stats.gemm_flops, tcq,
                            h->d_cond + ci, ln.rF, ln.rQ));
  return BR_OK;
}

// ---- refresh of one side: Q <- qr(F Q).Q in fp64, F = L | R (S=2nd) or M M^T | M^T M (S=1st) ----
br_status refresh_side(br_handle* h, Layer& L, bool left_side, br_handle::Lane& ln) {
  cudaStream_t s = ln.stream;
  const int64_t m = L.d.m, n = L.d.n;
  const int64_t k = left_side ? m : n;
  float* Q = left_side ? L.U : L.V;
  // S = 1st reads the momentum in the original space: the state buffer itself on the fp32 path, the
  // copy the caller prepared on the tensor-core path (whose state is the rotated momentum)
  const float* Mo = L.Morig ? L.Morig : L.M;
  const int ci = 2 * (int)(&L - h->layers.data()) + (left_side ? 0 : 1);
  // the tensor-core forms (power product, block projections) only for a basis whose last refresh
  // found it tracking the factor, and only where the product is known to have full rank
  const int64_t other = left_side ? n : m;
  const bool short_of_rank = (L.d.src == BR_SRC_FIRST) ? (k > other)
                                                       : (L.n_accum < (k + other - 1) / other);
  const bool complete = short_of_rank;
  QrTc* tcq = nullptr;
  if (L.use_tc && (h->cond_known[ci] & 1) && !complete)
    for (QrTc* t : ln.tcq) if (qr_tc_order(t) == k) tcq = t;
  for (int it = 0; it < h->hp.power_iters; ++it) {
    if (L.d.src == BR_SRC_SECOND) {
      const float* F = left_side ? L.L : L.R;
      // widen once, then fp64 products (the products of fp32 values are exact either way)
      BR_CUDA(h, f32_to_f64(F, ln.rF, k * k, s));
      BR_CUDA(h, f32_to_f64(Q, ln.rQ, k * k, s));
      count(h, 2);
      if (tcq) {
        br_status st = deflated_power(h, ln, tcq, k, s);
        if (st != BR_OK) return st;
      } else {
        BR_CUDA(h, dgemm(0, 0, k, k, k, 1.0, ln.rF, k, ln.rQ, k, 0.0, ln.rA, k, s));
        count(h); h->stats.gemm_flops += 2.0 * k * k * k;
      }
    } else if (left_side) {
      // (M M^T) U = M (M^T U)
      BR_CUDA(h, f32_to_f64(Q, ln.rQ, k * k, s));          // the current basis, for the completion of a deficient product
      count(h);
      BR_CUDA(h, sdgemm(1, 0, n, m, m, 1.0, Mo, n, Q, m, 0.0, ln.rZ, m, s));
      BR_CUDA(h, fdgemm(0, 0, m, m, n, 1.0, Mo, n, ln.rZ, m, 0.0, ln.rA, m, s));
      count(h, 2); h->stats.gemm_flops += 4.0 * m * m * n;
    } else {
      // (M^T M) V = M^T (M V)
      BR_CUDA(h, f32_to_f64(Q, ln.rQ, k * k, s));
      count(h);
      BR_CUDA(h, sdgemm(0, 0, m, n, n, 1.0, Mo, n, Q, n, 0.0, ln.rZ, n, s));
      BR_CUDA(h, fdgemm(1, 0, n, n, m, 1.0, Mo, n, ln.rZ, n, 0.0, ln.rA, n, s));
      count(h, 2); h->stats.gemm_flops += 4.0 * n * n * m;
    }
    // A rank-deficient product has no unique Q factor.  Which products are is known on the host: with
    // S = 1st, M M^T (M^T M) has rank <= min(m, n), short of the larger side; with S = 2nd, a factor that
    // has accumulated a gradients has rank <= a * (the other dimension).  The directions outside the
    // range of F Q are then completed from the current basis: what is orthonormalised is F Q with
    // 1e-6 ||(F Q)_j|| Q_j added to every column j (full rank whenever Q is).
    if (complete) {
      BR_CUDA(h, qr_complete_columns(ln.rA, Q, k, ln.rWork, h->d_status, s));
      count(h, 3);
    }
    // A product that is rank-deficient only numerically (gradients confined to a subspace) shows in the
    // factorisation itself: the orthonormalisation then repeats it, in the same call, on the completed
    // product, for which it needs the product once more (the factor's buffer is free by now) and the
    // current basis (ln.rQ).
    BR_CUDA(h, cudaMemcpyAsync(ln.rF, ln.rA, sizeof(double) * (size_t)k * (size_t)k, cudaMemcpyDeviceToDevice, s));
    {
      br_status st = orthonormalise(h, ln, k, tcq, ci, s);
      if (st != BR_OK) return st;
    }
    BR_CUDA(h, f64_to_f32(ln.rA, Q, k * k, s));
    count(h);
  }
  if (L.use_tc) {
    BR_CUDA(h, split_bf16(Q, left_side ? L.Uh : L.Vh, left_side ? L.Ul : L.Vl, k * k, s));
    count(h);
  }
  return BR_OK;
}

// Refresh the bases of the given layers: every (layer, side) is an independent job; jobs are
// dealt to the lanes largest first, each to the lane with the least work so far.
br_status refresh_layers(br_handle* h, const int* ids, int n_ids) {
  struct Job { int layer; bool left; double cost; int64_t k; bool needs_z; };
  std::vector<Job> jobs;
  // time of one job when it runs alone (ms, measured: 11 at order 2560, 45 at order 6912): a cubic
  // term for the products and a linear one for the chain of panel factorisations
  auto cost = [](double k) { return 5.4e-11 * k * k * k + 3.9e-3 * k; };
  for (int j = 0; j < n_ids; ++j) {
    const Layer& L = h->layers[ids[j]];
    const bool z = L.d.src != BR_SRC_SECOND;
    if (L.left) jobs.push_back({ids[j], true, cost((double)L.d.m), L.d.m, z});
    if (L.right) jobs.push_back({ids[j], false, cost((double)L.d.n), L.d.n, z});
  }
  if (jobs.empty()) return BR_OK;
  if (h->cond_pending) {
    // the notes of the previous batch: long since on the host unless the two refreshes are back to back
    BR_CUDA(h, cudaEventSynchronize(h->ev_cond));
    for (size_t i = 0; i < h->cond_known.size(); ++i) h->cond_known[i] = h->h_cond[i];
    h->cond_pending = false;
  }
  std::stable_sort(jobs.begin(), jobs.end(), [](const Job& a, const Job& b) { return a.cost > b.cost; });
  // each job to the least loaded lane that can hold it (lane 0 holds everything)
  const int nl = h->n_lanes;
  std::vector<std::vector<Job>> per_lane(nl);
  std::vector<double> load(nl, 0.0);
  for (const Job& jb : jobs) {
    int best = 0;
    for (int i = 1; i < nl; ++i) {
      const br_handle::Lane& ln = h->lanes[i];
      if (ln.cap_k < jb.k || (jb.needs_z && !ln.rZ)) continue;
      if (load[i] < load[best]) best = i;
    }
    per_lane[best].push_back(jb);
    load[best] += jb.cost;
  }
  const double f0 = h->stats.gemm_flops;
  const int span = h->stats.prof.begin(PROF_REFRESH, h->stream);
  if (nl > 1) {
    BR_CUDA(h, cudaEventRecord(h->ev_begin, h->stream));
    for (int i = 1; i < nl; ++i) BR_CUDA(h, cudaStreamWaitEvent(h->lanes[i].stream, h->ev_begin, 0));
  }
  // interleave the enqueueing so that every lane has work early
  size_t longest = 0;
  for (auto& v : per_lane) longest = std::max(longest, v.size());
  br_status failed = BR_OK;
  for (size_t r = 0; r < longest && failed == BR_OK; ++r)
    for (int i = 0; i < nl && failed == BR_OK; ++i) {
      if (r >= per_lane[i].size()) continue;
      const Job& jb = per_lane[i][r];
      failed = refresh_side(h, h->layers[jb.layer], jb.left, h->lanes[i]);
    }
  // the lanes forked from the handle's stream: join them again whatever happened above, so that
  // nothing of this call is still running on an internal stream once the handle's stream has passed it
  for (int i = 1; i < nl; ++i) {
    cudaError_t je = cudaEventRecord(h->lanes[i].done, h->lanes[i].stream);
    if (je == cudaSuccess) je = cudaStreamWaitEvent(h->stream, h->lanes[i].done, 0);
    if (je != cudaSuccess && failed == BR_OK) {
      h->err = format("joining a refresh lane failed: %s", cudaGetErrorString(je));
      failed = BR_ERR_CUDA;
    }
  }
  if (failed != BR_OK) return failed;
  h->stats.prof.end(span, h->stream, h->stats.gemm_flops - f0);
  BR_CUDA(h, cudaMemcpyAsync(h->h_cond, h->d_cond, sizeof(int) * h->cond_known.size(), cudaMemcpyDeviceToHost, h->stream));
  BR_CUDA(h, cudaEventRecord(h->ev_cond, h->stream));
  h->cond_pending = true;
  for (int j = 0; j < n_ids; ++j) {
    Layer& L = h->layers[ids[j]];
    if (L.left || L.right) L.refresh_count += 1;
  }
  return BR_OK;
}

br_status refresh_layer(br_handle* h, Layer& L) {
  const int id = (int)(&L - h->layers.data());
  return refresh_layers(h, &id, 1);
}

// L <- beta L + (1-beta) G G^T ; R <- beta R + (1-beta) G^T G   (Alg. 2), fp32 FFMA
br_status accumulate_factors_simt(br_handle* h, Layer& L, const float* G) {
  const float beta = h->hp.beta_factor < 0.f ? h->hp.beta2 : h->hp.beta_factor;
  const int64_t m = L.d.m, n = L.d.n;
  if (L.L) {
    BR_CUDA(h, sgemm(0, 1, m, m, n, 1.0f - beta, G, n, G, n, beta, L.L, m, h->stream));
    count(h); h->stats.gemm_flops += 2.0 * m * m * n;
  }
  if (L.R) {
    BR_CUDA(h, sgemm(1, 0, n, n, m, 1.0f - beta, G, n, G, n, beta, L.R, n, h->stream));
    count(h); h->stats.gemm_flops += 2.0 * n * n * m;
  }
  L.n_accum += 1;
  return BR_OK;
}

// out = U^T X V with the identity on an unrotated side; tmp is scratch
br_status rotate_simt(br_handle* h, Layer& L, const float* X, float* tmp, float* out) {
  const int64_t m = L.d.m, n = L.d.n;
  cudaStream_t s = h->stream;
  if (L.left && L.right) {
    BR_CUDA(h, sgemm(1, 0, m, n, m, 1.f, L.U, m, X, n, 0.f, tmp, n, s));
    BR_CUDA(h, sgemm(0, 0, m, n, n, 1.f, tmp, n, L.V, n, 0.f, out, n, s));
    count(h, 2); h->stats.gemm_flops += 2.0 * m * n * (m + n);
  } else if (L.left) {
    BR_CUDA(h, sgemm(1, 0, m, n, m, 1.f, L.U, m, X, n, 0.f, out, n, s));
    count(h); h->stats.gemm_flops += 2.0 * m * n * m;
  } else {
    BR_CUDA(h, sgemm(0, 0, m, n, n, 1.f, X, n, L.V, n, 0.f, out, n, s));
    count(h); h->stats.gemm_flops += 2.0 * m * n * n;
  }
  return BR_OK;
}

// out = U X V^T with the identity on an unrotated side; tmp is scratch
br_status rotate_back_simt(br_handle* h, Layer& L, const float* X, float* tmp, float* out) {
  const int64_t m = L.d.m, n = L.d.n;
  cudaStream_t s = h->stream;
  if (L.left && L.right) {
    BR_CUDA(h, sgemm(0, 0, m, n, m, 1.f, L.U, m, X, n, 0.f, tmp, n, s));
    BR_CUDA(h, sgemm(0, 1, m, n, n, 1.f, tmp, n, L.V, n, 0.f, out, n, s));
    count(h, 2);
  } else if (L.left) {
    BR_CUDA(h, sgemm(0, 0, m, n, m, 1.f, L.U, m, X, n, 0.f, out, n, s));
    count(h);
  } else {
    BR_CUDA(h, sgemm(0, 1, m, n, n, 1.f, X, n, L.V, n, 0.f, out, n, s));
    count(h);
  }
  return BR_OK;
}

// Temporary device memory for the state accessors (synchronising calls; not used by br_step).
float* tmp_alloc(br_handle* h, size_t bytes) {
  void* p = nullptr;
  if (h->alloc.alloc) return static_cast<float*>(h->alloc.alloc(bytes, h->alloc.ctx));
  if (cudaMalloc(&p, bytes) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
  return static_cast<float*>(p);
}
void tmp_free(br_handle* h, void* p) {
  if (!p) return;
  if (h->alloc.alloc) h->alloc.free(p, h->alloc.ctx); else cudaFree(p);
}

// One update of one layer on the accurate (fp32 FFMA) path.  G: the gradient to apply.
br_status update_layer_simt(br_handle* h, Layer& L, const void* G, const float* gscale) {
  const br_hparams& hp = h->hp;
  cudaStream_t s = h->stream;
  const int64_t m = L.d.m, n = L.d.n, mn = m * n;
  const int bf = L.d.grad_dtype == BR_BF16;
  br_status st;
  // Alg. 1 (momentum update) (and widen a bf16 gradient once)
  // (a clipped gradient is materialised in fp32 too: everything below works on the scaled values)
  const bool copy = bf || gscale != nullptr;
  BR_CUDA(h, ema_momentum(L.M, G, bf, mn, hp.beta1, copy ? h->sG : nullptr, nullptr, nullptr, gscale, s));
  count(h);
  const float* G32 = copy ? h->sG : reinterpret_cast<const float*>(G);
  const bool second = L.d.src == BR_SRC_SECOND;
  if (second && hp.accum == BR_ACCUM_EVERY_STEP && (st = accumulate_factors_simt(h, L, G32)) != BR_OK) return st;
  // Alg. 1 (periodic refresh)
  if (L.t % L.freq == 0) {
    if (second && hp.accum == BR_ACCUM_ON_REFRESH && (st = accumulate_factors_simt(h, L, G32)) != BR_OK) return st;
    if ((st = refresh_layer(h, L)) != BR_OK) return st;
  }
  // Alg. 1 (rotation of G and M)
  if ((st = rotate_simt(h, L, G32, h->sT, h->sGt)) != BR_OK) return st;
  if ((st = rotate_simt(h, L, L.M, h->sT, h->sMt)) != BR_OK) return st;
  // second-moment update and scaling, element-wise part: X overwrites sMt
  BR_CUDA(h, second_moment_scale(L.V2, h->sGt, h->sMt, mn, hp.beta2, hp.eps, s));
  count(h);
  // weight update: W <- (1 - eta lambda) W - eta U X V^T
  const float decay = 1.0f - hp.lr * hp.weight_decay;
  float* W = L.d.weight;
  if (L.left && L.right) {
    BR_CUDA(h, sgemm(0, 0, m, n, m, 1.f, L.U, m, h->sMt, n, 0.f, h->sT, n, s));
    BR_CUDA(h, sgemm(0, 1, m, n, n, -hp.lr, h->sT, n, L.V, n, decay, W, n, s));
    count(h, 2); h->stats.gemm_flops += 2.0 * m * n * (m + n);
  } else if (L.left) {
    BR_CUDA(h, sgemm(0, 0, m, n, m, -hp.lr, L.U, m, h->sMt, n, decay, W, n, s));
    count(h); h->stats.gemm_flops += 2.0 * m * n * m;
  } else {
    BR_CUDA(h, sgemm(0, 1, m, n, n, -hp.lr, h->sMt, n, L.V, n, decay, W, n, s));
    count(h); h->stats.gemm_flops += 2.0 * m * n * n;
  }
  return BR_OK;
}

br_status check_handle(br_handle* h) {
  if (!h) return BR_ERR_INVALID;
  cudaError_t e = cudaSetDevice(h->device);
  if (e != cudaSuccess) { h->err = format("cudaSetDevice: %s", cudaGetErrorString(e)); return BR_ERR_CUDA; }
  return BR_OK;
}

size_t buf_bytes(const Layer& L, int which, void** ptr) {
  const size_t m = L.d.m, n = L.d.n;
  switch (which) {
    case BR_BUF_W: *ptr = L.d.weight; return 4 * m * n;
    case BR_BUF_M: *ptr = L.M; return 4 * m * n;
    case BR_BUF_V2: *ptr = L.V2; return 4 * m * n;
    case BR_BUF_U: *ptr = L.U; return L.U ? 4 * m * m : 0;
    case BR_BUF_V: *ptr = L.V; return L.V ? 4 * n * n : 0;
    case BR_BUF_L: *ptr = L.L; return L.L ? 4 * m * m : 0;
    case BR_BUF_R: *ptr = L.R; return L.R ? 4 * n * n : 0;
    case BR_BUF_MROT: *ptr = L.use_tc ? L.M : nullptr; return L.use_tc ? 4 * m * n : 0;
    case BR_BUF_RING: *ptr = L.d.tau_max > 0 ? L.ring : nullptr; return L.d.tau_max > 0 ? (size_t)L.d.tau_max * m * n * dtype_size(L.d.grad_dtype) : 0;
    default: *ptr = nullptr; return 0;
  }
}

// Frees everything a handle owns; also the teardown of a br_create that failed half-way (every
// member is null or empty until it has been created).
void release(br_handle* h) {
  cudaSetDevice(h->device);
  cudaStreamSynchronize(h->stream);
  if (h->tc) tc_step_destroy(h->tc);
  for (int i = 1; i < br_handle::kMaxLanes; ++i) {
    if (h->lanes[i].stream) { cudaStreamSynchronize(h->lanes[i].stream); cudaStreamDestroy(h->lanes[i].stream); }
    if (h->lanes[i].done) cudaEventDestroy(h->lanes[i].done);
  }
  if (h->ev_begin) cudaEventDestroy(h->ev_begin);
  if (h->ev_cond) cudaEventDestroy(h->ev_cond);
  if (h->copy_stream) { cudaStreamSynchronize(h->copy_stream); cudaStreamDestroy(h->copy_stream); }
  if (h->ev_consumed) cudaEventDestroy(h->ev_consumed);
  if (h->ev_copied) cudaEventDestroy(h->ev_copied);
  if (h->h_cond) cudaFreeHost(h->h_cond);
  if (h->d_guard_offsets) cudaFree(h->d_guard_offsets);
  for (int i = 0; i < br_handle::kMaxLanes; ++i) {
    for (auto& kv : h->lanes[i].qr_graphs) if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
    for (QrTc* t : h->lanes[i].tcq) qr_tc_destroy(t);
  }
  for (auto& sp : h->stats.prof.spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
  for (auto e : h->stats.prof.free_events) cudaEventDestroy(e);
  if (h->slab) {
    if (h->alloc.alloc) h->alloc.free(h->slab, h->alloc.ctx); else cudaFree(h->slab);
  }
  (void)cudaGetLastError();
  delete h;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// C-ABI
// ---------------------------------------------------------------------------------------------
extern "C" {

br_status br_state_bytes(const br_layer_desc* layers, int n_layers, const br_hparams* hp,
                         size_t* total_bytes, size_t* overhead_bytes) {
  std::string err;
  br_status st = validate(layers, n_layers, hp, &err);
  if (st != BR_OK) { g_create_error = err; return st; }
  br_handle tmp;
  tmp.hp = *hp;
  init_layers(&tmp, layers, n_layers);
  Bump b;
  Sizes sz;
  layout(&tmp, b, &sz);
  sz.total += tc_step_scratch_bytes(tmp.layers, *hp);
  if (total_bytes) *total_bytes = sz.total;
  if (overhead_bytes) *overhead_bytes = sz.overhead;
  return BR_OK;
}

br_status br_create(br_handle** out, const br_layer_desc* layers, int n_layers, const br_hparams* hp,
                    int device, void* cuda_stream, const br_allocator* a) {
  if (!out) { g_create_error = "out is NULL"; return BR_ERR_INVALID; }
  *out = nullptr;
  std::string err;
  br_status st = validate(layers, n_layers, hp, &err);
  if (st != BR_OK) { g_create_error = err; return st; }
  for (int i = 0; i < n_layers; ++i) {
    if (!layers[i].weight || (reinterpret_cast<uintptr_t>(layers[i].weight) & 15)) {
      g_create_error = format("layer %d: weight pointer is NULL or not 16-byte aligned", i);
      return BR_ERR_INVALID;
    }
  }
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) { g_create_error = format("cudaSetDevice(%d): %s", device, cudaGetErrorString(e)); return BR_ERR_CUDA; }
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, device);
  if (e != cudaSuccess) { g_create_error = format("cudaGetDeviceProperties: %s", cudaGetErrorString(e)); return BR_ERR_CUDA; }
  if (prop.major != 10) {
    g_create_error = format("device %d is sm_%d%d; this library is built for sm_100a only", device, prop.major, prop.minor);
    return BR_ERR_CUDA;
  }
  br_handle* h = new br_handle();
  h->device = device;
  h->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  h->hp = *hp;
  if (a && a->alloc && a->free) h->alloc = *a;
  init_layers(h, layers, n_layers);

  Bump sizing;
  Sizes sz;
  layout(h, sizing, &sz);
  const size_t tc_bytes = align_up(tc_step_scratch_bytes(h->layers, h->hp));
  h->slab_bytes = sz.total + tc_bytes;
  void* p = nullptr;
  if (h->alloc.alloc) {
    p = h->alloc.alloc(h->slab_bytes, h->alloc.ctx);
  } else if (cudaMalloc(&p, h->slab_bytes) != cudaSuccess) {
    (void)cudaGetLastError();
    p = nullptr;
  }
  if (!p) {
    g_create_error = format("allocation of %zu bytes failed", h->slab_bytes);
    delete h;
    return BR_ERR_OOM;
  }
  h->slab = static_cast<char*>(p);
  Bump b;
  b.base = h->slab;
  Sizes sz2;
  layout(h, b, &sz2);

  // initial state: M = V~ = L = R = 0 (and everything else in the slab), U = V = I
  cudaStream_t s = h->stream;
  auto fail = [&](const char* what, cudaError_t ce) {
    g_create_error = format("%s: %s", what, cudaGetErrorString(ce));
    release(h);
    return BR_ERR_CUDA;
  };
  if ((e = cudaMemsetAsync(h->slab, 0, sz.total, s)) != cudaSuccess) return fail("cudaMemsetAsync", e);
  if (!h->guard_offsets.empty()) {
    const size_t gb = sizeof(unsigned long long) * h->guard_offsets.size();
    if ((e = cudaMalloc(reinterpret_cast<void**>(&h->d_guard_offsets), gb)) != cudaSuccess) return fail("cudaMalloc (canary table)", e);
    if ((e = cudaMemcpyAsync(h->d_guard_offsets, h->guard_offsets.data(), gb, cudaMemcpyHostToDevice, s)) != cudaSuccess) return fail("cudaMemcpyAsync", e);
    if ((e = guard_fill(h->slab, h->d_guard_offsets, (int)h->guard_offsets.size(), s)) != cudaSuccess) return fail("guard_fill", e);
  }
  for (Layer& L : h->layers) {
    if (L.U && (e = set_identity(L.U, L.d.m, s)) != cudaSuccess) return fail("set_identity", e);
    if (L.V && (e = set_identity(L.V, L.d.n, s)) != cudaSuccess) return fail("set_identity", e);
    if (L.use_tc) {
      if (L.U && (e = split_bf16(L.U, L.Uh, L.Ul, L.d.m * L.d.m, s)) != cudaSuccess) return fail("split_bf16", e);
      if (L.V && (e = split_bf16(L.V, L.Vh, L.Vl, L.d.n * L.d.n, s)) != cudaSuccess) return fail("split_bf16", e);
    }
  }
  h->lanes[0].stream = s;
  if (const char* env = std::getenv("BR_REFRESH_GRAPHS")) h->use_graphs = env[0] != '0';
  for (int i = 1; i < h->n_lanes; ++i) {
    if ((e = cudaStreamCreateWithFlags(&h->lanes[i].stream, cudaStreamNonBlocking)) != cudaSuccess) return fail("cudaStreamCreate", e);
    if ((e = cudaEventCreateWithFlags(&h->lanes[i].done, cudaEventDisableTiming)) != cudaSuccess) return fail("cudaEventCreate", e);
  }
  if ((e = cudaEventCreateWithFlags(&h->ev_begin, cudaEventDisableTiming)) != cudaSuccess) return fail("cudaEventCreate", e);
  if ((e = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking)) != cudaSuccess) return fail("cudaStreamCreate", e);
  if ((e = cudaEventCreateWithFlags(&h->ev_consumed, cudaEventDisableTiming)) != cudaSuccess) return fail("cudaEventCreate", e);
  if ((e = cudaEventCreateWithFlags(&h->ev_copied, cudaEventDisableTiming)) != cudaSuccess) return fail("cudaEventCreate", e);
  if ((e = cudaEventCreateWithFlags(&h->ev_cond, cudaEventDisableTiming)) != cudaSuccess) return fail("cudaEventCreate", e);
  h->cond_known.assign(2 * h->layers.size(), 0);
  if ((e = cudaMallocHost(reinterpret_cast<void**>(&h->h_cond), sizeof(int) * (h->cond_known.size() + 2))) != cudaSuccess)
    return fail("cudaMallocHost", e);
  if (h->tcq_bytes) {
    std::vector<int64_t> orders;
    for (const Layer& L : h->layers) {
      if (!L.use_tc) continue;
      for (int64_t k : {L.left ? L.d.m : (int64_t)0, L.right ? L.d.n : (int64_t)0})
        if (k && qr_tc_eligible(k) && std::find(orders.begin(), orders.end(), k) == orders.end()) orders.push_back(k);
    }
    for (int i = 0; i < h->n_lanes; ++i)
      for (int64_t k : orders) {
        if (!h->lanes[i].tcq_scratch || k > h->lanes[i].cap_k) continue;      // a small-order lane
        const char* qerr = nullptr;
        QrTc* t = qr_tc_create(k, h->lanes[i].tcq_scratch, device, s, &qerr);
        if (!t) {
          g_create_error = qerr ? qerr : "tensor-core projection plans could not be created";
          release(h);
          return BR_ERR_CUDA;
        }
        h->lanes[i].tcq.push_back(t);
      }
  }
  const char* tc_err = nullptr;
  h->tc = tc_step_create(h->layers, h->hp, h->slab + sz.total, tc_bytes, h->d_clip, h->clip_slots, device, s, &tc_err);
  if (!h->tc && tc_err) {
    g_create_error = tc_err;
    release(h);
    return BR_ERR_CUDA;
  }
  if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return fail("cudaStreamSynchronize", e);
  *out = h;
  return BR_OK;
}

br_status br_step(br_handle* h, const void* const* grads, int tau) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  if (!grads) { h->err = "grads is NULL"; return BR_ERR_INVALID; }
  const int nl = (int)h->layers.size();
  for (int i = 0; i < nl; ++i) {
    const Layer& L = h->layers[i];
    if (!grads[i] || (reinterpret_cast<uintptr_t>(grads[i]) & 15)) {
      h->err = format("layer %d: gradient pointer is NULL or not 16-byte aligned", i);
      return BR_ERR_INVALID;
    }
    if (tau < -1 || tau > L.d.tau_max) {
      h->err = format("layer %d: tau %d outside [0, %d]", i, tau, L.d.tau_max);
      return BR_ERR_TAU;
    }
  }
  // The integer state moves while the work is enqueued (the launches need the new values); when an
  // enqueue fails it is put back, so that calls, t, the refresh schedule and the ring slot read as
  // they did before the call.  Device buffers may already have been touched by the launches that
  // did go out: after BR_ERR_CUDA the handle is good for the accessors and br_destroy only.
  struct Snapshot { int64_t t, refresh_count, n_accum; };
  const int64_t calls_before = h->calls;
  std::vector<Snapshot> before(nl);
  for (int i = 0; i < nl; ++i) before[i] = {h->layers[i].t, h->layers[i].refresh_count, h->layers[i].n_accum};
  st = step_enqueue(h, grads, tau);
  if (st < 0) {
    h->calls = calls_before;
    for (int i = 0; i < nl; ++i) {
      h->layers[i].t = before[i].t; h->layers[i].refresh_count = before[i].refresh_count; h->layers[i].n_accum = before[i].n_accum;
    }
  }
  return st;
}

}  // extern "C"

namespace {

br_status step_enqueue(br_handle* h, const void* const* grads, int tau) {
  const int nl = (int)h->layers.size();
  br_status st = BR_OK;
  // ---- integer state (host) ---------------------------------------------------------------
  h->calls += 1;
  if (h->d_clip) {
    // clipping factor of this call's gradients (App. D.2), kept until they are applied
    std::vector<int64_t> numel(nl);
    std::vector<int> bf(nl);
    for (int i = 0; i < nl; ++i) { numel[i] = h->layers[i].d.m * h->layers[i].d.n; bf[i] = h->layers[i].d.grad_dtype == BR_BF16; }
    BR_CUDA(h, clip_factor(grads, numel.data(), bf.data(), nl, h->hp.clip_norm, h->d_clip_part,
                           h->d_clip + (h->calls - 1) % h->clip_slots, h->stream));
    count(h, (nl + 63) / 64 + 1);
  }
  std::vector<const void*> G(nl, nullptr);
  std::vector<const float*> GS(nl, nullptr);
  std::vector<char> stored(nl, 0);
  bool any = false;
  for (int i = 0; i < nl; ++i) {
    Layer& L = h->layers[i];
    const int tl = tau < 0 ? L.d.tau_max : tau;
    const int64_t src_call = h->calls - tl;     // Eq. (delayed_grad)
    if (src_call >= 1) {
      if (tl == 0 && L.use_tc) {
        // the tensor-core path reads through the ring: store g_c first (no older slot is needed)
        const size_t bytes = (size_t)L.d.m * L.d.n * dtype_size(L.d.grad_dtype);
        void* dst = const_cast<void*>(ring_slot_ptr(L, (h->calls - 1) % L.ring_slots));
        BR_CUDA(h, cudaMemcpyAsync(dst, grads[i], bytes, cudaMemcpyDeviceToDevice, h->stream));
        G[i] = dst;
        stored[i] = 1;
      } else {
        G[i] = (tl == 0) ? grads[i] : ring_slot_ptr(L, (src_call - 1) % L.ring_slots);
      }
      if (h->d_clip) GS[i] = h->d_clip + (src_call - 1) % h->clip_slots;
      L.t += 1;
      any = true;
    }
  }
  // ---- enqueue the updates ----------------------------------------------------------------
  const br_hparams& hp = h->hp;
  for (int i = 0; i < nl; ++i) {
    Layer& L = h->layers[i];
    if (!G[i]) continue;
    if (L.d.geom == BR_GEOM_NONE) {
      BR_CUDA(h, plain_adam(L.d.weight, L.M, L.V2, G[i], L.d.grad_dtype == BR_BF16, L.d.m * L.d.n,
                            hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay, GS[i], h->stream));
      count(h);
    } else if (!L.use_tc) {
      // a small matrix is bound by launch latency: its whole update is one launch, unless a refresh is due
      static const bool small_on = !(std::getenv("BR_SMALL_STEP") && std::getenv("BR_SMALL_STEP")[0] == '0');
      if (small_on && L.t % L.freq != 0 && small_step_eligible(L.d.m, L.d.n, L.left, L.right)) {
        const bool acc = L.d.src == BR_SRC_SECOND && hp.accum == BR_ACCUM_EVERY_STEP;
        const int64_t m = L.d.m, n = L.d.n;
        BR_CUDA(h, small_step(m, n, L.left, L.right, G[i], L.d.grad_dtype == BR_BF16, GS[i], L.M, L.V2, L.U, L.V, L.L, L.R,
                              L.d.weight, acc ? 1 : 0, hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay,
                              hp.beta_factor < 0.f ? hp.beta2 : hp.beta_factor, h->stream));
        count(h);
        h->stats.gemm_flops += (acc ? 2.0 : 0.0) * ((L.L ? m * m * n : 0) + (L.R ? n * n * m : 0)) +
                               6.0 * m * n * ((L.left ? m : 0) + (L.right ? n : 0));
        if (acc) L.n_accum += 1;
      } else if ((st = update_layer_simt(h, L, G[i], GS[i])) != BR_OK) {
        return st;
      }
    }
  }
  if (h->tc) {
    struct StepCtx { br_handle* h; const void* const* grads; std::vector<char>* stored; bool copied; };
    StepCtx sc{h, grads, &stored, false};
    TcStepCallbacks cb;
    cb.ctx = &sc;
    cb.refresh = [](void* ctx, const int* ids, int n) -> int {
      return (int)refresh_layers(static_cast<StepCtx*>(ctx)->h, ids, n);
    };
    static const bool side_copies = !(std::getenv("BR_RING_SIDE_STREAM") && std::getenv("BR_RING_SIDE_STREAM")[0] == '0');
    if (side_copies) cb.consumed = [](void* ctx, const int* ids, int n) -> int {
      StepCtx* c = static_cast<StepCtx*>(ctx);
      br_handle* h = c->h;
      BR_CUDA(h, cudaEventRecord(h->ev_consumed, h->stream));
      BR_CUDA(h, cudaStreamWaitEvent(h->copy_stream, h->ev_consumed, 0));
      for (int j = 0; j < n; ++j) {
        Layer& L = h->layers[ids[j]];
        if (L.ring_slots <= 0 || (*c->stored)[ids[j]]) continue;
        const size_t bytes = (size_t)L.d.m * L.d.n * dtype_size(L.d.grad_dtype);
        void* dst = const_cast<void*>(ring_slot_ptr(L, (h->calls - 1) % L.ring_slots));
        BR_CUDA(h, cudaMemcpyAsync(dst, c->grads[ids[j]], bytes, cudaMemcpyDeviceToDevice, h->copy_stream));
        (*c->stored)[ids[j]] = 1;
        c->copied = true;
      }
      return (int)BR_OK;
    };
    const char* terr = nullptr;
    int rc = tc_step_run(h->tc, h->layers, G, h->calls, tau, hp, h->d_status, h->stream, &h->stats, cb, &terr);
    if (sc.copied) {
      // (also on a failed step: the side stream must not outlive the caller's view of this call)
      cudaEventRecord(h->ev_copied, h->copy_stream);
      cudaStreamWaitEvent(h->stream, h->ev_copied, 0);
    }
    if (rc != 0) {
      if (terr) h->err = terr; else if (h->err.empty()) h->err = "tensor-core step failed";
      return rc < 0 ? (br_status)rc : BR_ERR_CUDA;
    }
  }
  // ---- store g_c in the ring (after every reader of the slot it may overwrite) --------------
  for (int i = 0; i < nl; ++i) {
    Layer& L = h->layers[i];
    if (L.ring_slots <= 0 || stored[i]) continue;
    const size_t bytes = (size_t)L.d.m * L.d.n * dtype_size(L.d.grad_dtype);
    void* dst = const_cast<void*>(ring_slot_ptr(L, (h->calls - 1) % L.ring_slots));
    BR_CUDA(h, cudaMemcpyAsync(dst, grads[i], bytes, cudaMemcpyDeviceToDevice, h->stream));
  }
  return any ? BR_OK : BR_WARMUP;
}

}  // namespace

extern "C" {

br_status br_debug_inject(br_handle* h, int kind, int64_t countdown) {
  if (!h) return BR_ERR_INVALID;
  if (kind == BR_INJECT_NONE) { h->stats.fail_countdown = -1; return BR_OK; }
  if (kind != BR_INJECT_LAUNCH_FAILURE || countdown < 0) { h->err = "unknown injection kind or negative countdown"; return BR_ERR_INVALID; }
  h->stats.fail_countdown = countdown;
  return BR_OK;
}

br_status br_debug_check_canaries(br_handle* h) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  if (h->guard_offsets.empty()) { h->err = "the handle was created without BR_FLAG_DEBUG_CANARY"; return BR_ERR_STATE; }
  int* first_bad = h->d_status + 8;                   // a spare word of the status area
  const int none = 0x7fffffff;
  BR_CUDA(h, cudaStreamSynchronize(h->stream));
  BR_CUDA(h, cudaMemcpy(first_bad, &none, sizeof(int), cudaMemcpyHostToDevice));
  BR_CUDA(h, guard_check(h->slab, h->d_guard_offsets, (int)h->guard_offsets.size(), first_bad, h->stream));
  BR_CUDA(h, cudaStreamSynchronize(h->stream));
  int bad = none;
  BR_CUDA(h, cudaMemcpy(&bad, first_bad, sizeof(int), cudaMemcpyDeviceToHost));
  if (bad != none) {
    h->err = format("canary %d of %zu (slab offset %llu) was overwritten: the piece in front of it was overrun", bad,
                    h->guard_offsets.size(), h->guard_offsets[(size_t)bad]);
    return BR_ERR_STATE;
  }
  return BR_OK;
}

br_status br_debug_wait_timeout(br_handle* h, uint64_t limit_ns) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  if (limit_ns < 1000 || limit_ns > 2000000000ull) { h->err = "limit outside [1 us, 2 s]"; return BR_ERR_INVALID; }
  BR_CUDA(h, tc_wait_probe(limit_ns, h->d_status, h->stream));
  count(h);
  return BR_OK;
}

br_status br_set_lr(br_handle* h, float lr) {
  if (!h) return BR_ERR_INVALID;
  if (!std::isfinite(lr)) { h->err = "lr is not finite"; return BR_ERR_INVALID; }
  h->hp.lr = lr;
  return BR_OK;
}

br_status br_refresh_basis(br_handle* h, int layer) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  const int nl = (int)h->layers.size();
  if (layer < -1 || layer >= nl) { h->err = "layer index out of range"; return BR_ERR_INVALID; }
  const int lo = layer < 0 ? 0 : layer, hi = layer < 0 ? nl : layer + 1;
  for (int i = lo; i < hi; ++i) {
    const Layer& L = h->layers[i];
    if (L.d.geom != BR_GEOM_NONE && L.t == 0) {
      h->err = format("layer %d: refresh before the first update (factor is all zero)", i);
      return BR_ERR_STATE;
    }
  }
  std::vector<int> ids, tc_ids;
  for (int i = lo; i < hi; ++i) {
    if (h->layers[i].d.geom == BR_GEOM_NONE) continue;
    ids.push_back(i);
    if (h->layers[i].use_tc) tc_ids.push_back(i);
  }
  // tensor-core layers keep the rotated momentum: back to the original space with the old basis,
  // forward again with the new one
  const char* terr = nullptr;
  std::vector<int64_t> count_before(nl);
  for (int i = 0; i < nl; ++i) count_before[i] = h->layers[i].refresh_count;
  auto undo = [&](br_status code) {            // a failed enqueue: the integer state reads as before the call
    for (int i = 0; i < nl; ++i) h->layers[i].refresh_count = count_before[i];
    return code;
  };
  if (!tc_ids.empty()) {
    int rc = tc_step_reexpress(h->tc, h->layers, tc_ids.data(), (int)tc_ids.size(), 0, h->d_status, h->stream, &h->stats, &terr);
    if (rc != 0) { h->err = terr ? terr : "re-expression failed"; return (br_status)rc; }
    for (int i : tc_ids) {
      Layer& L = h->layers[i];
      if (L.Morig) BR_CUDA(h, cudaMemcpyAsync(L.Morig, L.M, 4 * (size_t)L.d.m * L.d.n, cudaMemcpyDeviceToDevice, h->stream));
    }
  }
  if ((st = refresh_layers(h, ids.data(), (int)ids.size())) != BR_OK) return undo(st);
  if (!tc_ids.empty()) {
    int rc = tc_step_reexpress(h->tc, h->layers, tc_ids.data(), (int)tc_ids.size(), 1, h->d_status, h->stream, &h->stats, &terr);
    if (rc != 0) { h->err = terr ? terr : "re-expression failed"; return undo((br_status)rc); }
  }
  return BR_OK;
}

br_status br_sync_status(br_handle* h) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  BR_CUDA(h, cudaStreamSynchronize(h->stream));
  int word = 0;
  BR_CUDA(h, cudaMemcpy(&word, h->d_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (word > 0) BR_CUDA(h, cudaMemset(h->d_status, 0, sizeof(int)));
  if (word < 0) h->err = format("device status word %d (%s)", word, br_strerror(word));
  return (br_status)word;
}

br_status br_get_counters(br_handle* h, int layer, br_counters* out) {
  if (!h || !out) return BR_ERR_INVALID;
  if (layer < 0 || layer >= (int)h->layers.size()) { h->err = "layer index out of range"; return BR_ERR_INVALID; }
  const Layer& L = h->layers[layer];
  out->calls = h->calls;
  out->t = L.t;
  out->ring_slot = L.d.tau_max > 0 ? h->calls % L.d.tau_max : 0;
  out->refresh_count = L.refresh_count;
  out->next_refresh_t = (L.t / L.freq + 1) * L.freq;
  if (h->cond_pending) {
    if (cudaSetDevice(h->device) != cudaSuccess || cudaEventSynchronize(h->ev_cond) != cudaSuccess) {
      h->err = "could not read the conditioning notes of the last refresh"; return BR_ERR_CUDA;
    }
    for (size_t i = 0; i < h->cond_known.size(); ++i) h->cond_known[i] = h->h_cond[i];
    h->cond_pending = false;
  }
  out->basis_flags = (h->cond_known[2 * layer] & 1) | ((h->cond_known[2 * layer + 1] & 1) << 1) |
                     ((h->cond_known[2 * layer] & 2) << 1) | ((h->cond_known[2 * layer + 1] & 2) << 2);
  return BR_OK;
}

br_status br_set_counters(br_handle* h, int layer, const br_counters* in) {
  if (!h || !in) return BR_ERR_INVALID;
  if (layer < 0 || layer >= (int)h->layers.size()) { h->err = "layer index out of range"; return BR_ERR_INVALID; }
  if (in->calls < 0 || in->t < 0 || in->t > in->calls || in->refresh_count < 0) { h->err = "inconsistent counters"; return BR_ERR_INVALID; }
  Layer& L = h->layers[layer];
  h->calls = in->calls;
  L.t = in->t;
  L.refresh_count = in->refresh_count;
  L.n_accum = std::max(L.n_accum, h->hp.accum == BR_ACCUM_EVERY_STEP ? in->t : in->refresh_count);
  {
    br_status st = check_handle(h);
    if (st != BR_OK) return st;
    BR_CUDA(h, cudaStreamSynchronize(h->stream));
    if (h->cond_pending) {
      for (size_t i = 0; i < h->cond_known.size(); ++i) h->cond_known[i] = h->h_cond[i];
      h->cond_pending = false;
    }
    const int v[2] = {(int)((in->basis_flags & 1) | ((in->basis_flags >> 1) & 2)),
                      (int)(((in->basis_flags >> 1) & 1) | ((in->basis_flags >> 2) & 2))};
    h->cond_known[2 * layer] = v[0];
    h->cond_known[2 * layer + 1] = v[1];
    BR_CUDA(h, cudaMemcpy(h->d_cond + 2 * layer, v, sizeof v, cudaMemcpyHostToDevice));
  }
  return BR_OK;
}

br_status br_get_state(br_handle* h, int layer, int which, void* host_dst, size_t bytes) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  if (!host_dst || layer < 0 || layer >= (int)h->layers.size()) { h->err = "bad argument"; return BR_ERR_INVALID; }
  if (which == BR_BUF_CLIP) {
    if (!h->d_clip) { h->err = "clipping is off: no such buffer"; return BR_ERR_STATE; }
    if (bytes != sizeof(float) * (size_t)h->clip_slots) { h->err = "wrong size for the clipping factors"; return BR_ERR_SHAPE; }
    BR_CUDA(h, cudaStreamSynchronize(h->stream));
    BR_CUDA(h, cudaMemcpy(host_dst, h->d_clip, bytes, cudaMemcpyDeviceToHost));
    return BR_OK;
  }
  const Layer& L = h->layers[layer];
  void* p = nullptr;
  const size_t want = buf_bytes(L, which, &p);
  if (!p || want == 0) { h->err = "this layer has no such buffer"; return BR_ERR_STATE; }
  if (bytes != want) { h->err = format("buffer is %zu bytes, caller passed %zu", want, bytes); return BR_ERR_SHAPE; }
  BR_CUDA(h, cudaStreamSynchronize(h->stream));
  if (which == BR_BUF_M && L.use_tc) {
    // the state is M~: hand out M = U M~ V^T, computed with fp32 FFMA products into temporaries
    float* tmp = tmp_alloc(h, 2 * bytes);
    if (!tmp) { h->err = format("allocation of %zu bytes failed", 2 * bytes); return BR_ERR_OOM; }
    Layer& Lm = h->layers[layer];
    float* out = tmp + (size_t)L.d.m * L.d.n;
    st = rotate_back_simt(h, Lm, L.M, tmp, out);
    cudaError_t ce = cudaStreamSynchronize(h->stream);
    if (st == BR_OK && ce == cudaSuccess) ce = cudaMemcpy(host_dst, out, bytes, cudaMemcpyDeviceToHost);
    tmp_free(h, tmp);
    if (st != BR_OK) return st;
    if (ce != cudaSuccess) { h->err = format("get_state: %s", cudaGetErrorString(ce)); return BR_ERR_CUDA; }
  } else if (which == BR_BUF_RING) {
    const size_t row = (size_t)L.d.m * L.d.n * dtype_size(L.d.grad_dtype);
    BR_CUDA(h, cudaMemcpy2D(host_dst, row, p, L.slot_stride, row, L.d.tau_max, cudaMemcpyDeviceToHost));
  } else {
    BR_CUDA(h, cudaMemcpy(host_dst, p, bytes, cudaMemcpyDeviceToHost));
  }
  return BR_OK;
}

br_status br_set_state(br_handle* h, int layer, int which, const void* host_src, size_t bytes) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  if (!host_src || layer < 0 || layer >= (int)h->layers.size()) { h->err = "bad argument"; return BR_ERR_INVALID; }
  if (which == BR_BUF_CLIP) {
    if (!h->d_clip) { h->err = "clipping is off: no such buffer"; return BR_ERR_STATE; }
    if (bytes != sizeof(float) * (size_t)h->clip_slots) { h->err = "wrong size for the clipping factors"; return BR_ERR_SHAPE; }
    BR_CUDA(h, cudaStreamSynchronize(h->stream));
    BR_CUDA(h, cudaMemcpy(h->d_clip, host_src, bytes, cudaMemcpyHostToDevice));
    return BR_OK;
  }
  Layer& L = h->layers[layer];
  void* p = nullptr;
  const size_t want = buf_bytes(L, which, &p);
  if (!p || want == 0) { h->err = "this layer has no such buffer"; return BR_ERR_STATE; }
  if (bytes != want) { h->err = format("buffer is %zu bytes, caller passed %zu", want, bytes); return BR_ERR_SHAPE; }
  BR_CUDA(h, cudaStreamSynchronize(h->stream));
  const size_t mn_bytes = 4 * (size_t)L.d.m * L.d.n;
  if (L.use_tc && (which == BR_BUF_M || which == BR_BUF_U || which == BR_BUF_V)) {
    // The state of a tensor-core layer is M~ = U^T M V.  Setting M stores its rotation; setting a
    // basis keeps M (original space) as it is, so M~ is carried over: M~' = U'^T (U M~) or (M~ V^T) V'.
    float* tmp = tmp_alloc(h, 2 * mn_bytes);
    if (!tmp) { h->err = format("allocation of %zu bytes failed", 2 * mn_bytes); return BR_ERR_OOM; }
    float* tmp2 = tmp + (size_t)L.d.m * L.d.n;
    const int64_t m = L.d.m, n = L.d.n;
    cudaStream_t s = h->stream;
    cudaError_t ce = cudaSuccess;
    if (which == BR_BUF_M) {
      ce = cudaMemcpy(tmp, host_src, bytes, cudaMemcpyHostToDevice);
      if (ce == cudaSuccess) st = rotate_simt(h, L, tmp, tmp2, L.M);
    } else if (which == BR_BUF_U) {
      ce = sgemm(0, 0, m, n, m, 1.f, L.U, m, L.M, n, 0.f, tmp, n, s);                 // U_old M~
      if (ce == cudaSuccess) ce = cudaStreamSynchronize(s);
      if (ce == cudaSuccess) ce = cudaMemcpy(L.U, host_src, bytes, cudaMemcpyHostToDevice);
      if (ce == cudaSuccess) ce = sgemm(1, 0, m, n, m, 1.f, L.U, m, tmp, n, 0.f, L.M, n, s);   // U_new^T (.)
      count(h, 2);
    } else {
      ce = sgemm(0, 1, m, n, n, 1.f, L.M, n, L.V, n, 0.f, tmp, n, s);                 // M~ V_old^T
      if (ce == cudaSuccess) ce = cudaStreamSynchronize(s);
      if (ce == cudaSuccess) ce = cudaMemcpy(L.V, host_src, bytes, cudaMemcpyHostToDevice);
      if (ce == cudaSuccess) ce = sgemm(0, 0, m, n, n, 1.f, tmp, n, L.V, n, 0.f, L.M, n, s);   // (.) V_new
      count(h, 2);
    }
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(s);
    tmp_free(h, tmp);
    if (st != BR_OK) return st;
    if (ce != cudaSuccess) { h->err = format("set_state: %s", cudaGetErrorString(ce)); return BR_ERR_CUDA; }
  } else if (which == BR_BUF_RING) {
    const size_t row = (size_t)L.d.m * L.d.n * dtype_size(L.d.grad_dtype);
    BR_CUDA(h, cudaMemcpy2D(p, L.slot_stride, host_src, row, row, L.d.tau_max, cudaMemcpyHostToDevice));
  } else {
    BR_CUDA(h, cudaMemcpy(p, host_src, bytes, cudaMemcpyHostToDevice));
  }
  if (which == BR_BUF_L || which == BR_BUF_R) L.n_accum = (int64_t)1 << 40;   // a factor given by the caller: taken as full rank
  // a factor or a basis given by the caller: nothing is known about how well the basis tracks the factor
  if (which == BR_BUF_L || which == BR_BUF_U || which == BR_BUF_R || which == BR_BUF_V) {
    if (h->cond_pending) {
      BR_CUDA(h, cudaEventSynchronize(h->ev_cond));
      for (size_t i = 0; i < h->cond_known.size(); ++i) h->cond_known[i] = h->h_cond[i];
      h->cond_pending = false;
    }
    const int ci = 2 * layer + ((which == BR_BUF_R || which == BR_BUF_V) ? 1 : 0);
    const int zero = 0;
    h->cond_known[ci] = 0;
    BR_CUDA(h, cudaMemcpy(h->d_cond + ci, &zero, sizeof(int), cudaMemcpyHostToDevice));
  }
  if (L.use_tc && which == BR_BUF_U) { BR_CUDA(h, split_bf16(L.U, L.Uh, L.Ul, L.d.m * L.d.m, h->stream)); count(h); }
  if (L.use_tc && which == BR_BUF_V) { BR_CUDA(h, split_bf16(L.V, L.Vh, L.Vl, L.d.n * L.d.n, h->stream)); count(h); }
  BR_CUDA(h, cudaStreamSynchronize(h->stream));
  return BR_OK;
}

br_status br_get_launch_stats(br_handle* h, int64_t* kernel_launches, double* gemm_flops) {
  if (!h) return BR_ERR_INVALID;
  if (kernel_launches) *kernel_launches = h->stats.launches;
  if (gemm_flops) *gemm_flops = h->stats.gemm_flops;
  return BR_OK;
}

br_status br_profile(br_handle* h, int enable) {
  if (!h) return BR_ERR_INVALID;
  h->stats.prof.on = enable != 0;
  return BR_OK;
}

br_status br_get_profile(br_handle* h, br_profile_stats* out) {
  br_status st = check_handle(h);
  if (st != BR_OK) return st;
  if (!out) return BR_ERR_INVALID;
  BR_CUDA(h, cudaStreamSynchronize(h->stream));
  std::memset(out, 0, sizeof *out);
  Profiler& P = h->stats.prof;
  for (auto& sp : P.spans) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, sp.a, sp.b);
    if (sp.cls == PROF_TC) { out->tc_ms += ms; out->tc_launches += 1; }
    else if (sp.cls == PROF_EMA) { out->ema_ms += ms; out->ema_launches += 1; }
    else { out->refresh_ms += ms; out->refresh_spans += 1; }
    P.free_events.push_back(sp.a);
    P.free_events.push_back(sp.b);
  }
  P.spans.clear();
  out->tc_flops = P.units[PROF_TC];
  out->ema_bytes = P.units[PROF_EMA];
  out->refresh_flops = P.units[PROF_REFRESH];
  P.units[0] = P.units[1] = P.units[2] = 0.0;
  return BR_OK;
}

br_status br_destroy(br_handle* h) {
  if (!h) return BR_OK;
  release(h);
  return BR_OK;
}

br_status br_lr_warmup_cosine(int64_t step, int64_t total_steps, double warmup_fraction, double base_lr,
                              double min_lr, double* out_lr) {
  if (!out_lr || total_steps < 1 || step < 0 || step >= total_steps || !(warmup_fraction >= 0.0) ||
      !(warmup_fraction <= 1.0) || !std::isfinite(base_lr) || !std::isfinite(min_lr))
    return BR_ERR_INVALID;
  const int64_t W = (int64_t)std::ceil(warmup_fraction * (double)total_steps);
  if (step < W) { *out_lr = base_lr * (double)(step + 1) / (double)W; return BR_OK; }
  const int64_t rest = std::max<int64_t>(1, total_steps - W);
  const double pi = 3.14159265358979323846;
  *out_lr = min_lr + (base_lr - min_lr) * 0.5 * (1.0 + std::cos(pi * (double)(step - W) / (double)rest));
  return BR_OK;
}

br_status br_stage_aware_freq(int P, int tau, int f0, int* out_freq) {
  if (!out_freq || P < 1 || tau < 0 || f0 < 1) return BR_ERR_INVALID;
  const long long mid = P / 2 - 1;
  if (mid <= 0) return BR_ERR_INVALID;
  const long long n = tau > mid ? mid - tau : mid + 1 - tau;
  const long long den = mid - n;                 // (1 - n / mid) * mid
  if (den <= 0) return BR_ERR_INVALID;
  long long f = ((long long)f0 * mid) / den;     // both positive: truncation is the floor
  if (f < 1) f = 1;
  if (f > 0x7fffffffLL) f = 0x7fffffffLL;
  *out_freq = (int)f;
  return BR_OK;
}

br_status br_effective_delay(const double* C, const int* tau, int n, double* out) {
  if (!C || !tau || !out || n < 1) return BR_ERR_INVALID;
  double num = 0.0, den = 0.0;
  for (int i = 0; i < n; ++i) {
    if (tau[i] < 0 || !std::isfinite(C[i])) return BR_ERR_INVALID;
    const double c2 = C[i] * C[i];
    num += c2 * (double)tau[i] * (double)tau[i];
    den += c2;
  }
  if (!(den > 0.0)) return BR_ERR_INVALID;
  *out = std::sqrt(num / den);
  return BR_OK;
}

const char* br_strerror(int status) {
  switch (status) {
    case BR_OK: return "ok";
    case BR_WARMUP: return "warm-up call: no update applied";
    case BR_WARN_RANK_DEFICIENT: return "refresh met a rank-deficient factor";
    case BR_ERR_INVALID: return "invalid argument";
    case BR_ERR_SHAPE: return "bad shape or size";
    case BR_ERR_DTYPE: return "bad dtype";
    case BR_ERR_TAU: return "tau out of range";
    case BR_ERR_OOM: return "out of device memory";
    case BR_ERR_CUDA: return "CUDA error";
    case BR_ERR_STATE: return "operation not valid in this state";
    case BR_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

const char* br_last_error(const br_handle* h) { return h ? h->err.c_str() : g_create_error.c_str(); }

}  // extern "C"
