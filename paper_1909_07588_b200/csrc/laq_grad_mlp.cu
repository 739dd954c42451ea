// Step 1 of the LAQ iteration for the one-hidden-layer ReLU network of the paper's supplement.
#include "laq_internal.cuh"

namespace laq {

const char* mlp_check_shape(int, int, int) { return "LAQ_MODEL_MLP2 is not available in this build"; }
size_t mlp_scratch_bytes(const laq_config&) { return 0; }
laq_status mlp_setup(MlpPlan&, const Params&, void*, cudaStream_t) { return LAQ_EINVAL; }
int mlp_convert_shard(MlpPlan&, const Params&, int, const float*, long long, cudaStream_t) { return 0; }
int mlp_launch_gradients(MlpPlan&, const Params&, cudaStream_t) { return 0; }
void mlp_teardown(MlpPlan&) {}

}  // namespace laq
