// Internal declarations shared by the translation units of libbr.  Nothing here is part of
// the public C-ABI (see include/br.h).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include <vector>

#include "br.h"

namespace br {

// ---------------------------------------------------------------------------------------------
// Launch accounting (reported through br_get_launch_stats)
// ---------------------------------------------------------------------------------------------
// Optional per-class device timing: CUDA events recorded around the library's own launches on
// the handle's stream (classes: tensor-core contraction, momentum EMA, refresh).
enum ProfClass { PROF_TC = 0, PROF_EMA = 1, PROF_REFRESH = 2, PROF_NCLASS = 3 };

struct Profiler {
  bool on = false;
  struct Span { cudaEvent_t a, b; int cls; };
  std::vector<Span> spans;
  std::vector<cudaEvent_t> free_events;
  double units[PROF_NCLASS] = {0, 0, 0};     // flops (TC, refresh) or bytes (EMA) issued while on
  cudaEvent_t get() {
    cudaEvent_t e;
    if (!free_events.empty()) { e = free_events.back(); free_events.pop_back(); return e; }
    cudaEventCreate(&e);
    return e;
  }
  int begin(int cls, cudaStream_t s) {
    if (!on) return -1;
    Span sp{get(), get(), cls};
    cudaEventRecord(sp.a, s);
    spans.push_back(sp);
    return (int)spans.size() - 1;
  }
  void end(int idx, cudaStream_t s, double u) {
    if (idx < 0) return;
    cudaEventRecord(spans[idx].b, s);
    units[spans[idx].cls] += u;
  }
};

struct LaunchStats {
  int64_t launches = 0;
  double gemm_flops = 0.0;
  Profiler prof;
  // Host-side fault injection (br_debug_inject): when >= 0, counts down once per CUDA call the
  // library is about to issue for this handle; the call that finds it at 0 is NOT issued and reports
  // cudaErrorLaunchFailure instead.  Nothing on the device is touched by the injected failure.
  int64_t fail_countdown = -1;
  bool inject() {
    if (fail_countdown < 0) return false;
    return fail_countdown-- == 0;
  }
};

// ---------------------------------------------------------------------------------------------
// Element-wise kernels (elem.cu).  All take a stream and return the launch error.
// ---------------------------------------------------------------------------------------------
cudaError_t set_identity(float* Q, int64_t k, cudaStream_t s);

// Alg. 1 (momentum update): M <- beta1 M + (1-beta1) G.  G is fp32 or bf16 (g_is_bf16).  Optional outputs:
// Gf32 (G widened to fp32), Mh/Ml (bf16 hi/lo split of the new M).
// gscale (optional, DEVICE): clipping factor the gradient is multiplied by
cudaError_t ema_momentum(float* M, const void* G, int g_is_bf16, int64_t numel, float beta1,
                         float* Gf32, __nv_bfloat16* Mh, __nv_bfloat16* Ml, const float* gscale, cudaStream_t s);
// Global-norm clipping factor of one call: *out = min(1, clip / ||all gradients||_2).  part: scratch of
// 296 * ceil(n / 64) doubles.  Fixed summation order.
cudaError_t clip_factor(const void* const* grads, const int64_t* numel, const int* is_bf16, int n, float clip,
                        double* part, float* out, cudaStream_t s);

// Eq. (adam): plain Adam, eps inside the sqrt, no bias correction, decoupled weight decay.
cudaError_t plain_adam(float* W, float* M, float* V, const void* G, int g_is_bf16, int64_t numel,
                       float lr, float beta1, float beta2, float eps, float wd, const float* gscale, cudaStream_t s);

// Alg. 1 (second-moment update and scaling) (element-wise part): V~ <- beta2 V~ + (1-beta2) G~^2 ; X = M~/sqrt(V~+eps).
// X overwrites Mt.
cudaError_t second_moment_scale(float* V2, const float* Gt, float* Mt, int64_t numel, float beta2,
                                float eps, cudaStream_t s);

// fp32 -> bf16 hi (+ optional lo = bf16(x - hi)).
cudaError_t split_bf16(const float* X, __nv_bfloat16* hi, __nv_bfloat16* lo, int64_t numel,
                       cudaStream_t s);
cudaError_t widen_bf16(const __nv_bfloat16* X, float* out, int64_t numel, cudaStream_t s);
// out(double) <- in(float) ; out(float) <- in(double)
cudaError_t f64_to_f32(const double* X, float* out, int64_t numel, cudaStream_t s);
cudaError_t f32_to_f64(const float* X, double* out, int64_t numel, cudaStream_t s);
// Three-term bf16 split (all 24 bits of the fp32 rounding of x) of a rows x cols block of a strided
// fp64 matrix, or of a contiguous fp32 array, into compact planes; A (fp64, strided) -= D (fp32, compact).
cudaError_t split3_f64(const double* X, int64_t ld, int64_t rows, int64_t cols, __nv_bfloat16* p1,
                       __nv_bfloat16* p2, __nv_bfloat16* p3, cudaStream_t s);
cudaError_t split3_f32(const float* X, int64_t numel, __nv_bfloat16* p1, __nv_bfloat16* p2, __nv_bfloat16* p3,
                       cudaStream_t s);
cudaError_t sub_f32_from_f64(double* A, int64_t ld, int64_t rows, int64_t cols, const float* D, cudaStream_t s);
// out <- beta1 M + (1-beta1) G (out-of-place form of Alg. 1 (momentum update))
cudaError_t ema_out(float* out, const float* M, const void* G, int g_is_bf16, int64_t numel, float beta1,
                    const float* gscale, cudaStream_t s);

// One whole update (Alg. 1 (momentum, rotation, second moment, weight update) and the factor EMAs of Alg. 2, no refresh) of a matrix with both
// dimensions <= 128 in a single one-CTA launch (small_step.cu).  accumulate: update L and R as well.
bool small_step_eligible(int64_t m, int64_t n, bool left, bool right);
cudaError_t small_step(int64_t m, int64_t n, bool left, bool right, const void* G, int g_is_bf16, const float* gscale,
                       float* M, float* V2, float* U, float* V, float* L, float* R, float* W, int accumulate, float lr,
                       float beta1, float beta2, float eps, float weight_decay, float beta_factor, cudaStream_t s);

// Debug canaries (BR_FLAG_DEBUG_CANARY): n guards of 256 bytes at byte offsets offs[] (DEVICE array) of the slab.
cudaError_t guard_fill(char* slab, const unsigned long long* offs, int n, cudaStream_t s);
cudaError_t guard_check(const char* slab, const unsigned long long* offs, int n, int* first_bad, cudaStream_t s);

// ---------------------------------------------------------------------------------------------
// SIMT contractions (gemm_simt.cu):  C = alpha * op(A) op(B) + beta * C, row-major.
// op(X) = X or X^T (ta / tb).  M, N, K are the dimensions of the product.
// ---------------------------------------------------------------------------------------------
cudaError_t sgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, float alpha, const float* A,
                  int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                  cudaStream_t s);
// fp32 inputs, fp64 accumulation and output (power step F Q of a refresh)
cudaError_t sdgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const float* A,
                   int64_t lda, const float* B, int64_t ldb, double beta, double* C, int64_t ldc,
                   cudaStream_t s);
cudaError_t dgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const double* A,
                  int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                  cudaStream_t s);
// As dgemm, with the contraction split into nsplit ranges of K whose partial products (nsplit * M * N
// doubles in `partial`) are added in a fixed order by a second kernel, and with an optional DEVICE
// flag that cancels the launches when it is non-zero at the time they run.
cudaError_t dgemm_ex(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const double* A,
                     int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                     int nsplit, double* partial, const int* skip, cudaStream_t s);

// ---------------------------------------------------------------------------------------------
// QR with positive diagonal in fp64 (qr.cu).  A (k x k, row-major, ld = k) is overwritten by
// its Q factor.  work: at least qr_work_doubles(k) doubles.  status: device int, set to
// BR_WARN_RANK_DEFICIENT when a pivot underflows.  Returns the number of launches in *launches.
// ---------------------------------------------------------------------------------------------
size_t qr_work_doubles(int64_t k);
// Optional tensor-core form of the block projections (see qr.cu): plans and scratch for one order
// k, created once.  qr_tc_scratch_bytes is 0 when the order is not eligible.
struct QrTc;
bool qr_tc_eligible(int64_t k);
size_t qr_tc_scratch_bytes(int64_t k);
QrTc* qr_tc_create(int64_t k, char* scratch, int device, cudaStream_t s, const char** err);
void qr_tc_destroy(QrTc* t);
int64_t qr_tc_order(const QrTc* t);
// Completion of a product that is short of rank: A[:, j] += 1e-6 * ||A[:, j]|| * Q[:, j] (Q fp32, the
// current basis; a zero column becomes Q[:, j]), and BR_WARN_RANK_DEFICIENT is raised in *status.
// work: the QR work area of this order (used for the column norms).
cudaError_t qr_complete_columns(double* A, const float* Q, int64_t k, double* work, int* status, cudaStream_t s);
// *out (fp32, k x k, owned by t) = Frest U on the tensor cores (three-term bf16 splits, six products)
cudaError_t qr_tc_power(QrTc* t, const double* Frest, const double* U, int* status, cudaStream_t s, const float** out);
cudaError_t qr_tc_project(QrTc* t, int node, double* A, int64_t k, int64_t jp, int64_t wp, int64_t jt,
                          int64_t wt, int* status, cudaStream_t s);
// tc: null, or the plans for this order: the first sweep then projects on the tensor cores (ask for it
// only when the previous refresh of this basis left *cond_out == 1).  cond_out: DEVICE int that
// receives 1 when no column shrank below 1e-3 of its length during this factorisation, else 0.
// Acopy / Qprev (both k x k fp64, or both null): a second copy of A and the basis the product was formed
// from.  With them, a product that turns out rank-deficient -- some |R_jj| <= 1e-12 max |R_kk| -- is
// factorised again in the same call with 1e-6 ||A_j|| Qprev_j added to every column (the completion rule
// for rank-deficient products), so that the result is orthonormal either way; BR_WARN_RANK_DEFICIENT is
// raised.  The launches of that second factorisation are always enqueued and return at once when the
// product has full rank.
cudaError_t qr_pos_inplace(double* A, int64_t k, double* work, int* status, cudaStream_t s,
                           int64_t* launches, double* flops, QrTc* tc = nullptr, int* cond_out = nullptr,
                           const double* Acopy = nullptr, const double* Qprev = nullptr);

// ---------------------------------------------------------------------------------------------
// tcgen05 grouped contraction (gemm_tc.cu)
// ---------------------------------------------------------------------------------------------
enum Epilogue : int32_t {
  EPI_AXPBY_F32 = 0,    // D <- alpha*acc + beta*D                 (factor EMA, weight write, plain)
  EPI_SPLIT_BF16 = 1,   // Dh <- bf16(acc), Dl <- bf16(acc - Dh)   (Dl optional)
  EPI_SECOND_MOMENT = 2,// D(V~) <- beta*D + alpha*acc^2
  EPI_SCALE_BF16 = 3,   // Dh(X) <- bf16(acc / sqrt(D(V~) + eps))
  // Alg. 1 (momentum and second-moment updates, scaling) in rotated coordinates, acc = G~:
  //   D2(M~) <- beta1 D2 + (1-beta1) acc ; D(V~) <- beta D + alpha acc^2 ; Dh(X) <- bf16(D2 / sqrt(D + eps))
  EPI_ROTATED_ADAM = 4
};

struct TcOperand {
  const void* ptr = nullptr;      // bf16, DEVICE (slot 0 when the operand lives in a ring)
  int64_t ld = 0;                 // elements
  int32_t mn_major = 0;           // 1: stored K x MN (MN contiguous); 0: stored MN x K (K contiguous)
  int32_t ring_slots = 0;         // > 0: the operand is the stale-gradient ring of this many slots
  int64_t slot_stride_bytes = 0;  // distance between ring slots
};

struct TcProblem {
  int64_t Md = 0, Nd = 0, K = 0;
  int32_t n_pairs = 0;            // 1..3; all pairs share majors
  TcOperand A[3], B[3];
  int32_t epilogue = EPI_AXPBY_F32;
  int32_t tau_max = 0;            // of the layer (delay bookkeeping on the device)
  int32_t dyn_scalars = 0;        // 1: alpha / beta come from the launch arguments
  // global-norm clipping: the accumulator of this problem is built from a gradient that carries the
  // factor clip[(calls - 1 - tau) mod clip_slots]; clip_mode 1 multiplies it by the factor (G~), 2 by
  // its square (G G^T), 0 leaves it alone
  const float* clip = nullptr; int32_t clip_slots = 0; int32_t clip_mode = 0;
  int32_t fold_kb = 0;            // > 0: accumulate in chunks of this many 64-deep k-blocks, summed outside the tensor
                                  // core (a plan whose problems all ask for it runs the folded form of the kernel)
  int32_t symmetric = 0;          // 1: A_p = B_p and D is square: only tiles touching the upper triangle are
                                  // computed, the rest of D is written as their mirror image (EPI_AXPBY_F32 only)
  float alpha = 1.f, beta = 0.f, eps = 0.f, beta1 = 0.f;
  float* D = nullptr; int64_t ldd = 0;                                   // fp32 in/out
  float* D2 = nullptr;                                                   // second fp32 in/out (same ld)
  __nv_bfloat16* Dh = nullptr; __nv_bfloat16* Dl = nullptr; int64_t ldh = 0;  // bf16 outputs
};

struct TcPlan;  // opaque: device problem table with its tensor maps, built on the host

// Build a plan for problems that may run concurrently in one launch.  Synchronises `s` once.
// Returns nullptr and sets *err on failure.
TcPlan* tc_plan_create(const TcProblem* problems, int n, int device, cudaStream_t s, const char** err);
void tc_plan_destroy(TcPlan* p);
// calls / tau: delay bookkeeping (a problem whose layer has calls - tau < 1 is skipped; ring
// operands read slot (calls - 1 - tau) mod slots; tau < 0 means the layer's tau_max).
cudaError_t tc_plan_launch(TcPlan* p, long long calls, int tau, float dyn_alpha, float dyn_beta,
                           int* status_word, cudaStream_t s);
double tc_plan_flops(const TcPlan* p);
// Launch only the problems [first, first + count) of a plan (e.g. one node of a recursion whose
// problems all live in one plan), and the flop count of that range.
cudaError_t tc_plan_launch_range(TcPlan* p, int first, int count, long long calls, int tau, float dyn_alpha,
                                 float dyn_beta, int* status_word, cudaStream_t s);
double tc_plan_flops_range(const TcPlan* p, int first, int count);
int tc_supported(int device);
// Exercises the bounded mbarrier wait of the contraction kernel: a wait that nothing satisfies, limit_ns long.
cudaError_t tc_wait_probe(uint64_t limit_ns, int* status_word, cudaStream_t s);

}  // namespace br
