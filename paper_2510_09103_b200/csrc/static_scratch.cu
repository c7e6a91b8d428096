// adapm_group_meansq_static: the block mean of g^2 for callers that cannot allocate device memory.
//
// The two-stage reduction behind adapm_group_meansq needs a few partial sums per group between its
// stages.  Here they live in a fixed array that is part of the library image, so the caller passes
// only the gradient and the output.
#include <mutex>

#include "adapm_internal.h"

namespace adapm {
void set_error_text(const char* text);   // ctx.cu
}

namespace {

// Partial sums of one call.  Every GPU that loads the library holds this 1 MiB until the process exits.
static __device__ __align__(256) float g_static_partials[ADAPM_STATIC_SCRATCH_FLOATS];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_partials_addr[kMaxDevices] = {};   // device address of g_static_partials, per device ordinal

// `g_static_partials` as written in host code is only a handle; the address a kernel can use has to
// be asked for, once per device, while that device is current.
int partials_for_current_device(float** out) {
  int dev = -1;
  ADAPM_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ADAPM_ERANGE;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_partials_addr[dev]) {
    float* p = nullptr;
    ADAPM_CUDA(cudaGetSymbolAddress((void**)&p, g_static_partials));
    if (!p) return ADAPM_ECUDA;
    g_partials_addr[dev] = p;
  }
  *out = g_partials_addr[dev];
  return ADAPM_OK;
}

}  // namespace

extern "C" int adapm_group_meansq_static(const void* g, int32_t grad_dtype, int64_t n_groups, int64_t group_elems,
                                         float* out, adapm_stream stream) {
  using namespace adapm;
  if (!g || !out || n_groups <= 0 || group_elems <= 0) return ADAPM_EINVAL;
  if (grad_dtype != ADAPM_GRAD_F32 && grad_dtype != ADAPM_GRAD_BF16) return ADAPM_EINVAL;
  if ((uintptr_t)g % 16) return ADAPM_EALIGN;
  const int64_t cpg = (group_elems + kWarpUnitMax - 1) / kWarpUnitMax;
  if (cpg > INT32_MAX || n_groups > (int64_t)ADAPM_STATIC_SCRATCH_FLOATS / cpg) {
    set_error_text("adapm_group_meansq_static: n_groups * ceil(group_elems / 2048) exceeds "
                   "ADAPM_STATIC_SCRATCH_FLOATS; use adapm_group_meansq with caller scratch");
    return ADAPM_ERANGE;
  }
  float* partials = nullptr;
  int rc = partials_for_current_device(&partials);
  if (rc != ADAPM_OK) return rc;
  // Stage 1 writes partial[0 .. n_groups*cpg) and stage 2 reads exactly those, so what an earlier
  // call left in the array never has to be cleared.
  cudaStream_t s = (cudaStream_t)stream;
  rc = launch_meansq_partial(g, grad_dtype, n_groups, group_elems, (int)cpg, partials, s);
  if (rc != ADAPM_OK) return rc;
  return launch_meansq_final(partials, n_groups, group_elems, (int)cpg, out, s);
}
