/*
 * br.h -- C-ABI of the basis-rotation optimizer step for NVIDIA B200 (sm_100a).
 *
 * One handle owns the optimizer state of a set of independent weight matrices
 * ("layers").  Each call of br_step() submits one gradient per layer and applies
 * the update that is due under a delay of tau calls:
 *
 *   Algorithm 1 ("Adam with Basis Rotation") of the paper, per W in R^{m x n}:
 *     M  <- beta1 M + (1-beta1) G
 *     if t mod freq == 0:  U, V <- Eigenbasis-Estimation (Algorithm 2)
 *     G~ <- U^T G V ;  M~ <- U^T M V
 *     V~ <- beta2 V~ + (1-beta2) G~ .* G~
 *     W  <- W - eta U ( M~ / sqrt(V~ + eps) ) V^T
 *   Algorithm 2, source S in {1st, 2nd} x geometry in {unilateral, bilateral}:
 *     S=2nd: L <- beta L + (1-beta) G G^T, U <- Power(L, U); bilateral: same with R = G^T G, V
 *     S=1st: U <- Power(M M^T, U); bilateral: V <- Power(M^T M, V)
 *     unilateral: only the smaller dimension is rotated (Sec. 3.2)
 *   Power(A, Q) = Q-factor of the QR decomposition of A Q (Sec. 3.2), made unique
 *   by a positive diagonal of R.
 *   Geometry NONE is plain Adam as Eq. (adam) writes it: eps inside the square
 *   root, no bias correction.
 *   Delay (App. B, Eq. delayed_grad): the gradient applied at a call is the one
 *   submitted tau calls earlier; the first tau calls apply no update.
 *
 * All pointers named DEVICE are CUDA device pointers on the handle's device; all
 * others are host pointers.  Matrices are row-major and contiguous.  Every entry
 * point returns a br_status: 0 = ok, > 0 informational (state is valid), < 0
 * error.  An error detected on the host leaves the handle unchanged; BR_ERR_CUDA from br_step or
 * br_refresh_basis (a failed enqueue) leaves the integer state as it was before the call, but device
 * buffers may be partly updated: the handle is then good for the accessors and br_destroy only.  Work is
 * enqueued on the handle's stream; only the calls documented as synchronising
 * wait for it.  There is no CPU fallback: every step of the path runs in CUDA
 * kernels, and the calls fail with BR_ERR_CUDA when no device is usable.
 */
#ifndef BR_H_
#define BR_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BR_API __attribute__((visibility("default")))
#else
#define BR_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct br_handle br_handle; /* opaque; owned by the library */

typedef enum {
  BR_OK = 0,
  BR_WARMUP = 1,              /* no layer applied an update (call index <= tau)            */
  BR_WARN_RANK_DEFICIENT = 2, /* a refresh met a numerically rank-deficient factor         */
  BR_ERR_INVALID = -1,        /* NULL pointer, bad enum, bad hyper-parameter               */
  BR_ERR_SHAPE = -2,
  BR_ERR_DTYPE = -3,
  BR_ERR_TAU = -4,            /* tau outside [0, tau_max]                                  */
  BR_ERR_OOM = -5,            /* allocator returned NULL; br_last_error has the byte count */
  BR_ERR_CUDA = -6,
  BR_ERR_STATE = -7,          /* e.g. forced refresh before the first update               */
  BR_ERR_TIMEOUT = -8         /* a bounded device-side wait gave up (status word)          */
} br_status;

typedef enum { BR_GEOM_NONE = 0, BR_GEOM_UNILATERAL = 1, BR_GEOM_BILATERAL = 2 } br_geometry;
typedef enum { BR_SRC_FIRST = 1, BR_SRC_SECOND = 2 } br_source;
typedef enum { BR_F32 = 0, BR_BF16 = 1 } br_dtype;
/* Arithmetic of the rotation / factor contractions.
 *   BR_GEMM_FP32: fp32 FFMA kernels (relative error ~1e-7 per product).
 *   BR_GEMM_BF16: tcgen05 tensor-core tiles on bf16 operands with fp32 accumulation in
 *   tensor memory; fp32 operands of the forward rotations are carried as a bf16 hi/lo pair.
 *   Layers whose dimensions are not multiples of 8 always use the fp32 kernels. */
typedef enum { BR_GEMM_FP32 = 0, BR_GEMM_BF16 = 2 } br_gemm_prec;
/* When L and R are accumulated: at every update (default), or only inside the refresh as
 * Algorithm 2 literally places the line. */
typedef enum { BR_ACCUM_EVERY_STEP = 0, BR_ACCUM_ON_REFRESH = 1 } br_accum_mode;

typedef struct {
  int64_t m, n;        /* W is m x n, row-major, leading dimension n                        */
  int32_t geom;        /* br_geometry                                                      */
  int32_t src;         /* br_source (ignored for BR_GEOM_NONE)                             */
  int32_t grad_dtype;  /* br_dtype of the gradients passed to br_step                      */
  int32_t tau_max;     /* ring capacity in calls for this layer, >= 0                      */
  int32_t freq;        /* refresh period in updates; <= 0 -> br_hparams.freq               */
  int32_t reserved;
  float* weight;       /* DEVICE fp32 m*n, owned by the caller, updated in place           */
} br_layer_desc;

typedef struct {
  float lr, beta1, beta2, eps, weight_decay; /* weight decay is decoupled; paper default 0 here */
  float beta_factor;   /* EMA rate of L and R; < 0 -> beta2 (Algorithm 2 reuses beta2)       */
  int32_t freq;        /* default refresh period, >= 1 (the paper uses 10)                  */
  int32_t power_iters; /* Power() applications per refresh, >= 1 (the paper uses 1)         */
  int32_t accum;       /* br_accum_mode                                                    */
  int32_t gemm_prec;   /* br_gemm_prec                                                     */
  uint32_t flags;      /* BR_FLAG_* bits, 0 by default                                     */
  /* Global-norm gradient clipping (App. D.2 of the paper uses 1.0); 0 = off.  The gradients of one
   * call, over all layers of the handle, are scaled by min(1, clip_norm / their joint L2 norm); the
   * factor belongs to the call and goes with its gradients through the delay ring. */
  float clip_norm;
  uint64_t scratch_limit_bytes; /* cap on per-step transient scratch; 0 -> library default */
} br_hparams;

/* br_hparams.flags.  BR_FLAG_DEBUG_CANARY: a debugging layout of the handle's memory, with 256 bytes of
 * guard words behind every piece of state and scratch (a few hundred KB for a large layer set);
 * br_debug_check_canaries tells whether any kernel wrote past the piece in front of a guard. */
#define BR_FLAG_DEBUG_CANARY 1u

/* Device-memory allocator.  NULL (or NULL members) -> cudaMalloc / cudaFree.  alloc returns a
 * DEVICE pointer aligned to at least 256 bytes, or NULL. */
typedef struct {
  void* (*alloc)(size_t bytes, void* ctx);
  void (*free)(void* ptr, void* ctx);
  void* ctx;
} br_allocator;

typedef struct {
  int64_t calls;          /* br_step calls so far (handle-wide)                              */
  int64_t t;              /* updates applied to this layer (Algorithm 1's t)                 */
  int64_t ring_slot;      /* ring slot the next call writes: calls mod tau_max (0 if no ring) */
  int64_t refresh_count;  /* refreshes done for this layer, scheduled and forced             */
  int64_t next_refresh_t; /* next t with t mod freq == 0                                     */
  /* Not part of the method's integer state: what the library remembers about the conditioning of
   * the last refresh of this layer's bases.  Bit 0 (left) and bit 1 (right): no column of F Q shrank
   * below 1e-3 of its length under orthonormalisation; the next refresh of a tensor-core layer runs
   * its block projections on the tensor cores only for a basis whose bit is set.  Bit 2 (left) and
   * bit 3 (right): the last refresh met a numerically rank-deficient product (some |R_jj| <= 1e-12 of
   * the largest); the status word then holds BR_WARN_RANK_DEFICIENT and the basis was completed from the
   * previous one in that same refresh, so it is orthonormal.  Saved and restored with the other
   * counters so that a resumed run takes the same decisions. */
  int64_t basis_flags;
} br_counters;

typedef enum {
  BR_BUF_W = 0,   /* m*n fp32                                         */
  BR_BUF_M = 1,   /* m*n fp32, original space (tensor-core layers: U M~ V^T, see BR_BUF_MROT) */
  BR_BUF_V2 = 2,  /* m*n fp32, V~ in the rotated space                */
  BR_BUF_U = 3,   /* m*m fp32 (absent when the left side is unrotated) */
  BR_BUF_V = 4,   /* n*n fp32 (absent when the right side is unrotated) */
  BR_BUF_L = 5,   /* m*m fp32 (S=2nd, left side rotated)              */
  BR_BUF_R = 6,   /* n*n fp32 (S=2nd, right side rotated)             */
  BR_BUF_RING = 7, /* tau_max * m*n gradients in grad_dtype, slot-major */
  /* m*n fp32: the momentum in rotated coordinates, M~ = U^T M V.  Between two refreshes
   * M~_t = beta1 M~_{t-1} + (1-beta1) U^T G_t V holds exactly (Alg. 1 (momentum update) is linear), and this is
   * what layers on the tensor-core path store; BR_BUF_M converts on the way in and out with fp32
   * products.  A checkpoint that must resume bit-identically saves and restores this buffer (after
   * U and V) instead of BR_BUF_M.  Absent for layers on the fp32 path. */
  BR_BUF_MROT = 8,
  /* max(tau_max) + 1 floats: the clipping factors of the last calls (slot = (call - 1) mod length),
   * a handle-wide buffer read and written with layer = 0; absent when clip_norm == 0. */
  BR_BUF_CLIP = 9
} br_buf;

/* Bytes of device memory br_create would request for these layers (state, ring, operand
 * shadows and scratch).  Host only.  App. H's table is overhead_bytes: rotation matrices
 * plus factor buffers in fp32, summed over layers (either out pointer may be NULL). */
BR_API br_status br_state_bytes(const br_layer_desc* layers, int n_layers, const br_hparams* hp,
                         size_t* total_bytes, size_t* overhead_bytes);

/* Create a handle on `device`, enqueueing on `cuda_stream` (a cudaStream_t cast to void*;
 * NULL = the legacy default stream).  State starts as M = V~ = L = R = 0, U = V = I, t = 0.
 * Layer descriptors and hyper-parameters are copied.  Synchronises the stream once. */
BR_API br_status br_create(br_handle** out, const br_layer_desc* layers, int n_layers,
                    const br_hparams* hp, int device, void* cuda_stream,
                    const br_allocator* alloc);

/* One call of the delayed step.  grads: host array of n_layers DEVICE pointers, each m*n
 * elements of the layer's grad_dtype, owned by the caller and read only by the work this call
 * enqueues (the caller may overwrite them once the stream has passed that work).
 * tau in [0, tau_max] applies to every layer; tau = -1 uses each layer's own tau_max.
 * Returns BR_WARMUP when no layer applied an update.  Does not synchronise. */
BR_API br_status br_step(br_handle* h, const void* const* grads, int tau);

/* Learning rate eta_t used by the following steps. */
BR_API br_status br_set_lr(br_handle* h, float lr);

/* Run the Power() part of Algorithm 2 now, from the current L, R (S=2nd) or M (S=1st);
 * layer = -1 refreshes every rotated layer.  Does not change t.  BR_ERR_STATE if a target
 * layer has t == 0 (its factor is all zero).
 * Bases are refreshed several at a time on internal streams that fork from and join the
 * handle's stream inside the call (the same happens for the periodic refresh inside br_step, which
 * also stores the call's gradients through an internal stream that joins before it returns).  The
 * launch chain of a basis is captured into a CUDA graph the first time its (order, form) occurs and
 * replayed afterwards (plain launches if that capture fails).  Neither this call nor br_step may be
 * issued while the handle's stream is being captured by the caller: both read conditioning notes of
 * the previous refresh back from the device. */
BR_API br_status br_refresh_basis(br_handle* h, int layer);

/* Wait for the stream and return the device status word (BR_OK, BR_WARN_RANK_DEFICIENT,
 * BR_ERR_TIMEOUT ...); the word is cleared when it held a warning. */
BR_API br_status br_sync_status(br_handle* h);

BR_API br_status br_get_counters(br_handle* h, int layer, br_counters* out);
BR_API br_status br_set_counters(br_handle* h, int layer, const br_counters* in);

/* Copy a state buffer to / from HOST memory; `bytes` must equal the buffer's size.
 * Both synchronise the stream.  Setting U or V also refreshes the operand shadows and leaves the
 * momentum of the original space unchanged (a tensor-core layer re-expresses its M~ for the new
 * basis).  BR_BUF_M of a tensor-core layer needs 8*m*n bytes of temporary device memory from the
 * handle's allocator for the duration of the call. */
BR_API br_status br_get_state(br_handle* h, int layer, int which, void* host_dst, size_t bytes);
BR_API br_status br_set_state(br_handle* h, int layer, int which, const void* host_src, size_t bytes);

/* Counts of the library's own kernel launches and of floating-point operations issued by its
 * contraction kernels since creation (for benchmarks). */
BR_API br_status br_get_launch_stats(br_handle* h, int64_t* kernel_launches, double* gemm_flops);

/* Device-side timing of the library's own launches, by class, with CUDA events on the handle's
 * stream.  br_profile(h, 1) starts recording, br_profile(h, 0) stops; br_get_profile waits for the
 * stream, sums what was recorded since the last call and clears it. */
typedef struct {
  double tc_ms;          /* tensor-core contraction launches                                  */
  double tc_flops;       /* floating-point operations those launches issued                   */
  int64_t tc_launches;
  double ema_ms;         /* momentum EMA launches (Alg. 1 (momentum update), with the bf16 hi/lo of M)    */
  double ema_bytes;      /* bytes those launches must move (gradient, M in and out, hi/lo)    */
  int64_t ema_launches;
  double refresh_ms;     /* Power() spans: power product + QR + conversions                   */
  double refresh_flops;
  int64_t refresh_spans;
} br_profile_stats;
BR_API br_status br_profile(br_handle* h, int enable);
BR_API br_status br_get_profile(br_handle* h, br_profile_stats* out);

/* Free everything the handle allocated.  NULL is accepted.  Synchronises the stream. */
BR_API br_status br_destroy(br_handle* h);

/*
 * Stage-aware refresh period (App. I of the paper, "Stage-aware basis rotation implementation").
 * For a pipeline of P stages, a stage whose gradients are tau updates old and a base period f0:
 *   mid = floor(P / 2) - 1;  n = mid - tau if tau > mid, else mid + 1 - tau;
 *   f = floor(f0 / (1 - n / mid)),
 * evaluated in exact integer arithmetic as floor(f0 * mid / (mid - n)).  The printed rule is undefined
 * where mid - n <= 0 (for P = 32: tau <= 1) or mid <= 0 (P < 4): those arguments return BR_ERR_INVALID
 * and leave *out_freq alone, as do P < 1, tau < 0 or f0 < 1.  A result below 1 is raised to 1.
 * Host only.  The period is what br_layer_desc.freq takes, per layer.
 */
BR_API br_status br_stage_aware_freq(int P, int tau, int f0, int* out_freq);

/*
 * Effective delay of stage-dependent delays (Sec. 2.3, Eq. (effective-delay)):
 *   tau' = sqrt( sum_i C_i^2 tau_i^2 / sum_i C_i^2 )
 * for n groups of coordinates with smoothness constants C_i (HOST array, not all zero) and delays
 * tau_i >= 0 (HOST array).  Host only.
 */
BR_API br_status br_effective_delay(const double* C, const int* tau, int n, double* out);

/*
 * Learning-rate schedule of the paper's runs (App. D.2): linear warm-up over the first
 * warmup_fraction of total_steps (the paper uses 0.012), then cosine decay that would reach min_lr at step = total_steps:
 *   step <  W = ceil(warmup_fraction * total_steps):  base_lr * (step + 1) / W
 *   step >= W:  min_lr + (base_lr - min_lr) * (1 + cos(pi * (step - W) / max(1, total_steps - W))) / 2
 * step counts from 0.  Host only; the result is what br_set_lr takes.
 */
BR_API br_status br_lr_warmup_cosine(int64_t step, int64_t total_steps, double warmup_fraction, double base_lr,
                                     double min_lr, double* out_lr);

/*
 * Failure-path diagnostics (every device-side wait is bounded and reports through the status word;
 * host errors leave the integer state untouched).  Neither call faults,
 * traps or hangs the GPU.
 *
 * br_debug_inject: host-side fault injection.  With kind = BR_INJECT_LAUNCH_FAILURE the library counts
 * the CUDA calls (launches, copies, event operations) it is about to issue for this handle; the one
 * that finds `countdown` at 0 is not issued and reports a launch failure instead, so the entry point
 * that was running returns BR_ERR_CUDA.  BR_INJECT_NONE disarms it.  After an injected failure inside
 * br_step the integer state (calls, t, refresh_count, ring slot) reads as before the call; device
 * buffers may have been touched by the launches that went out before it.
 *
 * br_debug_wait_timeout: enqueues a one-warp kernel that waits, with the contraction kernel's own bounded
 * wait, on a barrier that nothing will ever arrive on, for limit_ns (1 us .. 2 s).  The wait gives up,
 * the kernel returns, and the status word holds BR_ERR_TIMEOUT from then on: br_sync_status returns it,
 * later contraction launches of the handle return at once without touching their outputs, and the
 * handle can still be read and destroyed.
 */
typedef enum { BR_INJECT_NONE = 0, BR_INJECT_LAUNCH_FAILURE = 1 } br_inject_kind;
BR_API br_status br_debug_inject(br_handle* h, int kind, int64_t countdown);
BR_API br_status br_debug_wait_timeout(br_handle* h, uint64_t limit_ns);
/* Waits for the stream and checks the guard words of a handle created with BR_FLAG_DEBUG_CANARY: BR_OK, or
 * BR_ERR_STATE with the first overwritten guard in br_last_error (also when the handle has no guards). */
BR_API br_status br_debug_check_canaries(br_handle* h);

BR_API const char* br_strerror(int status);
/* Message of the last error on this handle (or of the last failed br_create when h is NULL). */
BR_API const char* br_last_error(const br_handle* h);

/*
 * Stand-alone contraction entry point (used by tests and profiling of the tensor-core tile
 * kernel): D = sum_p A_p * B_p^T with bf16 operands and fp32 accumulation, where A_p is
 * Md x K and B_p is Nd x K.  a_mn / b_mn != 0 means the operand is stored with its M (or N)
 * index contiguous, i.e. as a K x Md (K x Nd) row-major array; otherwise K is contiguous.
 * lda / ldb are leading dimensions in elements.  D (fp32, ld = ldd) receives
 * alpha * acc + beta * D.  All pointers DEVICE; dims and leading dimensions multiples of 8.
 * Enqueues on `cuda_stream`, does not synchronise.  n_pairs in [1, 3].
 */
BR_API br_status br_gemm_bf16(void* cuda_stream, int64_t Md, int64_t Nd, int64_t K, int n_pairs,
                       const void* const* A, const void* const* B, int a_mn, int b_mn,
                       int64_t lda, int64_t ldb, float* D, int64_t ldd, float alpha, float beta);

/*
 * One Power(F, Q) application without any allocation.  (The paper has no counterpart: this is a
 * library convenience around the Power() step it describes.)
 *
 * For callers that cannot allocate device memory when they need a refresh: processes whose
 * framework already owns all of HBM, services that forbid allocation after start-up, loops that
 * cannot afford the device-wide synchronisation of cudaMalloc / cudaFree.  Q (k x k fp32, DEVICE,
 * row-major) is replaced by the Q factor, with a positive diagonal of R, of the fp64 product F*Q;
 * F is k x k fp32, DEVICE, read only.  The caller owns F and Q.  device_flag, if not NULL, is a
 * DEVICE int that receives 0 or BR_WARN_RANK_DEFICIENT.
 *
 * Scratch lives in a fixed array inside the library's device image (about 2.9 MB on every GPU
 * that loads the library, held until the process exits), so k is limited to 512: larger orders
 * return BR_ERR_SHAPE and must use br_create / br_refresh_basis.  The call itself, and everything
 * it calls, performs no cudaMalloc, cudaFree or other allocating routine.  The first call on a
 * device looks the array's address up (once per device); make that first call outside any stream
 * capture.  All calls on a GPU share the one array, which keeps the previous call's contents: the
 * call clears what must start at zero, and two calls whose work overlaps on the GPU (different
 * streams, or different threads) race on it -- serialise them.  Enqueues on cuda_stream (the
 * device of that stream must be current) and does not synchronise.
 */
BR_API br_status br_power_static(void* cuda_stream, const float* F, float* Q, int64_t k,
                                 int* device_flag);

#ifdef __cplusplus
}
#endif
#endif /* BR_H_ */
