// placeholder until the tensor-core kernel lands
#include "common.cuh"
namespace falcon {
bool tree_attn_tc_supports(const falcon_ctx*, const falcon_attn_args&) { return false; }
int launch_tree_attn_tc(falcon_ctx*, const falcon_attn_args&, cudaStream_t) { return FALCON_ERR_UNSUPPORTED; }
void tree_attn_tc_release(falcon_ctx*) {}
}  // namespace falcon
