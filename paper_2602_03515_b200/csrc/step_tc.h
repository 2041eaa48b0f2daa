// Per-layer state record and the interface of the tensor-core step planner (step_tc.cu).
#pragma once
#include <string>
#include <vector>

#include "br_internal.h"

namespace br {

struct Layer {
  br_layer_desc d{};
  bool left = false, right = false;   // which sides carry a rotation
  bool use_tc = false;                // contractions run on the tcgen05 tile kernel
  int freq = 1;
  // M holds the momentum of Alg. 1 (momentum update): in the original space on the fp32 path, in ROTATED
  // coordinates (M~ = U^T M V) on the tensor-core path (see step_tc.cu)
  float *M = nullptr, *V2 = nullptr, *U = nullptr, *V = nullptr, *L = nullptr, *R = nullptr;
  float* Morig = nullptr;             // tensor-core layers with S = 1st: M_t in the original space for a refresh
  __nv_bfloat16 *Uh = nullptr, *Ul = nullptr, *Vh = nullptr, *Vl = nullptr;  // bf16 hi/lo of U, V
  char* ring = nullptr;
  int ring_slots = 0;                 // physical slots: tau_max, or 1 for a tensor-core layer without delay
  size_t slot_stride = 0;             // bytes between ring slots
  int64_t t = 0, refresh_count = 0;
  int64_t n_accum = 0;                // gradients accumulated into L / R so far (bounds their rank)
};

std::string format(const char* fmt, ...);
size_t dtype_size(int dt);
void rotated_sides(int64_t m, int64_t n, int geom, bool* left, bool* right);

cudaError_t fdgemm(int ta, int tb, int64_t M, int64_t N, int64_t K, double alpha, const float* A,
                   int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                   cudaStream_t s);

struct TcStep;
struct TcStepCallbacks {
  void* ctx = nullptr;
  // runs Power() for the given layers (independent of one another), returns br_status
  int (*refresh)(void* ctx, const int* layers, int n) = nullptr;
  // optional: told, once the last launch that reads the gradients of these layers is enqueued (their
  // ring slots may then be overwritten behind an event on the step's stream); returns br_status
  int (*consumed)(void* ctx, const int* layers, int n) = nullptr;
};

// Transient scratch (bytes) the tensor-core step needs for these layers.
size_t tc_step_scratch_bytes(const std::vector<Layer>& layers, const br_hparams& hp);
// Returns nullptr with *err == nullptr when no layer uses the tensor-core path.
// clip / clip_slots: the handle's ring of clipping factors (null when clipping is off)
TcStep* tc_step_create(std::vector<Layer>& layers, const br_hparams& hp, char* scratch, size_t bytes,
                       const float* clip, int clip_slots, int device, cudaStream_t s, const char** err);
// Enqueue the updates of every tensor-core layer whose G[i] is non-null.  0 on success,
// a negative br_status otherwise (message in *err).
int tc_step_run(TcStep* t, std::vector<Layer>& layers, const std::vector<const void*>& G, long long calls,
                int tau, const br_hparams& hp, int* d_status, cudaStream_t s, LaunchStats* stats,
                const TcStepCallbacks& cb, const char** err);
// Re-express the momentum buffer of the given tensor-core layers in place: forward = 0 turns M~ into
// M = U M~ V^T, forward = 1 turns M into M~ = U^T M V, with the bases as they are at that point.
int tc_step_reexpress(TcStep* t, std::vector<Layer>& layers, const int* ids, int n, int forward, int* d_status,
                      cudaStream_t s, LaunchStats* stats, const char** err);
void tc_step_destroy(TcStep* t);

}  // namespace br
