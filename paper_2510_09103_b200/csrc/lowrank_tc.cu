// Tensor-core (tcgen05) kernels of the low-rank path.
#include "adapm_internal.h"

namespace adapm {

bool tensor_path_supports(const adapm_ctx*, const std::vector<int64_t>&) { return false; }
int build_tensor_program(adapm_ctx*, const std::vector<int64_t>&, int64_t&) { return ADAPM_EUNSUPPORTED; }
int run_tensor_launch(adapm_ctx*, const Launch&, const Bases&, const StepScalars&, cudaStream_t) {
  return ADAPM_EUNSUPPORTED;
}
void destroy_tensor_program(adapm_ctx*) {}

}  // namespace adapm
