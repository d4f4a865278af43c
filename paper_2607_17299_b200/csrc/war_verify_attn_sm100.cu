// Tensor-core verify attention (placeholder until the tcgen05 kernel lands): forwards to the plain kernel.
#include "war_common.cuh"
#include "war_attn_plan.cuh"

war_status_t war_attn_launch_sm100(const void* q, const void* k, const void* v, const int32_t* page_table,
                                   const int32_t* prefix_len, const war_attn_params_t* p, const AttnWorkspace& w,
                                   void* out, float* lse, int* status_word, cudaStream_t s) {
    return war_attn_launch_simple(q, k, v, page_table, prefix_len, p, w, out, lse, status_word, s);
}
