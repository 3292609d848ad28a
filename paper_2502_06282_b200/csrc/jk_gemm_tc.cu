// Tensor-core (tcgen05) path of the dense contractions.  Placeholder: not available yet, the
// CUDA-core kernels run instead.
#include "jk_common.cuh"

size_t jk_tc_partial_bytes(const jk_config&) { return 0; }
void jk_tc_destroy(jk_ctx* ctx) { if (ctx) ctx->tc_state = nullptr; }
int jk_tc_available(const jk_ctx*) { return 0; }
int jk_tc_expert_ffn(jk_ctx*, cudaStream_t, const jk_draft_weights*, int, const int32_t*, int,
                     float*, int, int, long long) {
  return JK_ERR_SHAPE;
}
