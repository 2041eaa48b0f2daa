// br_power_static: one Power(F, Q) application (fp64 product F*Q, QR with positive diagonal,
// result rounded to fp32) that allocates nothing.
//
// Who needs this.  Some hosts may not allocate device memory at the moment they want a basis
// refresh: a training process that handed the whole HBM to its framework's pool at start-up (a
// raw cudaMalloc then fails or has to fight the pool for memory), a service that forbids
// allocation after initialisation so that a late out-of-memory cannot happen, or a latency-bound
// loop that cannot take the device-wide synchronisation that cudaMalloc / cudaFree imply.  The
// handle-based path asks its allocator for one slab in br_create; this entry point instead keeps
// its scratch in a fixed array that lives in the library's device image.
//
// The array is loaded on every GPU that loads the library and stays there until the process
// exits (2.9 MB per GPU), which is why the supported order is capped at kMaxOrder.
//
// `g_power_scratch` is a device symbol: in host code its name is only a stand-in, never a device
// address, so the host obtains the real address with cudaGetSymbolAddress -- once per device,
// with that device current -- and passes that pointer to the kernels.
#include <mutex>

#include "br_internal.h"

namespace {

constexpr int64_t kMaxOrder = 512;
// k*k doubles for the product F*Q (rounded up to a 256-byte boundary), the QR work area (91,200
// doubles at order kMaxOrder, the largest over all orders up to it), and 64 doubles holding the
// rank-deficiency flag.
constexpr size_t kWorkDoubles = 98304;
constexpr size_t kScratchDoubles = (size_t)kMaxOrder * kMaxOrder + kWorkDoubles + 64;

static __device__ __align__(256) double g_power_scratch[kScratchDoubles];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
double* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch on the current device (set up on first use on that device).
cudaError_t scratch_for_current_device(double** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[dev]) {
    double* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_power_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" br_status br_power_static(void* cuda_stream, const float* F, float* Q, int64_t k,
                                     int* device_flag) {
  using namespace br;
  if (!F || !Q || k < 1) return BR_ERR_INVALID;
  if (k > kMaxOrder) return BR_ERR_SHAPE;   // beyond the fixed scratch: use the handle-based path
  // the work area starts on a 256-byte boundary whatever the parity of k: its sub-buffers are
  // accessed with 16-byte vector loads and stores
  const size_t work_off = ((size_t)k * k + 31) / 32 * 32;
  if (work_off + qr_work_doubles(k) + 64 > kScratchDoubles) return BR_ERR_SHAPE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  double* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) { (void)cudaGetLastError(); return BR_ERR_CUDA; }
  double* A = scratch;                                   // k x k product, overwritten by its Q factor
  double* work = scratch + work_off;
  int* flag = device_flag ? device_flag : reinterpret_cast<int*>(scratch + (kScratchDoubles - 64));
  // The array keeps whatever the previous call left.  Only the flag has to start at zero; every
  // other word is written by this call before it is read.
  if (cudaMemsetAsync(flag, 0, sizeof(int), s) != cudaSuccess) return BR_ERR_CUDA;
  if (sdgemm(0, 0, k, k, k, 1.0, F, k, Q, k, 0.0, A, k, s) != cudaSuccess) return BR_ERR_CUDA;
  if (qr_pos_inplace(A, k, work, flag, s, nullptr, nullptr) != cudaSuccess) return BR_ERR_CUDA;
  if (f64_to_f32(A, Q, k * k, s) != cudaSuccess) return BR_ERR_CUDA;
  return BR_OK;
}
