// tcgen05 / TMEM / TMA projection kernels: not wired yet; the fp32 path carries every configuration.
#include "gemm_tc.cuh"

namespace galore {

bool tensor_path_eligible(const galore_config_t&) { return false; }
int tensor_proj_splits(const galore_config_t&, bool) { return 1; }
galore_status_t tensor_plan_init(TensorPlan*, const galore_config_t&, bool, void*, void*, float*, int) {
  return GALORE_ERR_UNIMPLEMENTED;
}
bool tensor_operands_aligned(const galore_config_t&, const void*, int64_t, const void*, int64_t) { return false; }
galore_status_t step_tensor(TensorPlan*, const galore_config_t&, bool, void*, int64_t, const void*, int64_t, float,
                            const AdamParams&, float*, float*, uint8_t*, float*, uint8_t*, float*, int, int64_t,
                            int32_t*, cudaStream_t) {
  return GALORE_ERR_UNIMPLEMENTED;
}

}  // namespace galore
