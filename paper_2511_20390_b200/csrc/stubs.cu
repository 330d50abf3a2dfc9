// Entry points declared in the public header whose kernels are not written yet.
#include "common.cuh"
extern "C" {
int free_create(const free_model_desc*, const free_drafter_desc*, free_ctx**) { return FREE_ERR_UNSUPPORTED; }
int free_destroy(free_ctx*) { return FREE_ERR_UNSUPPORTED; }
size_t free_workspace_bytes(const free_ctx*, int) { return 0; }
int dit_verify_pass(free_ctx*, int, const float*, const int32_t*, const int32_t*, float, const free_schedule*,
                    float*, float*, void*, void*, size_t, void*) { return FREE_ERR_UNSUPPORTED; }
int draft_step(free_ctx*, int, const float*, const void*, const int32_t*, const int32_t*, float,
               const free_schedule*, const float*, float*, float*, void*, void*, size_t, void*) { return FREE_ERR_UNSUPPORTED; }
int sample_trajectory(free_ctx*, int, const float*, const int32_t*, const free_schedule*, const free_spec_params*,
                      const float*, const float*, const float*, float*, free_traj_stats*, void*, size_t, void*) { return FREE_ERR_UNSUPPORTED; }
size_t free_op_linear_workspace_bytes(void) { return 0; }
int free_op_linear(int, int, int, int, int, int, const void*, const void*, const float*, void*, float*, const float*,
                   int64_t, int, void*, size_t, void*) { return FREE_ERR_UNSUPPORTED; }
int free_op_ln_modulate(int, int, int, int, const float*, const float*, const float*, int64_t, void*, void*) { return FREE_ERR_UNSUPPORTED; }
int free_op_attention(int, int, int, int, int, const void*, void*, void*, size_t, void*) { return FREE_ERR_UNSUPPORTED; }
size_t free_op_attention_workspace_bytes(int, int, int, int, int) { return 0; }
}
