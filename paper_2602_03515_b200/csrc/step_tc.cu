// placeholder until the tensor-core planner lands
#include "step_tc.h"
namespace br {
size_t tc_step_scratch_bytes(const std::vector<Layer>&, const br_hparams&) { return 0; }
TcStep* tc_step_create(std::vector<Layer>&, const br_hparams&, char*, size_t, int, cudaStream_t, const char** err) { if (err) *err = nullptr; return nullptr; }
int tc_step_run(TcStep*, std::vector<Layer>&, const std::vector<const void*>&, const br_hparams&, int*, cudaStream_t, LaunchStats*, const TcStepCallbacks&, const char**) { return 0; }
void tc_step_destroy(TcStep*) {}
}
extern "C" br_status br_gemm_bf16(void*, int64_t, int64_t, int64_t, int, const void* const*, const void* const*, int, int, int64_t, int64_t, float*, int64_t, float, float) { return BR_ERR_STATE; }
