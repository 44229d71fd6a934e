// Fast-transform execution of the compression (power-of-two lengths): declarations.
#pragma once
#include "common.cuh"

namespace freqkv {

struct FdctPlan {
    float2* twiddle = nullptr;  // device tables owned by the plan
    int32_t n_in = 0, n_keep = 0;
};

bool fdct_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep);
cudaError_t fdct_make_plan(int32_t n_in, int32_t n_keep, cudaStream_t stream, FdctPlan* out);
void fdct_free_plan(FdctPlan* plan);
cudaError_t launch_fdct(const CacheView& view, int32_t dtype, int32_t n_mat, const FdctPlan& plan, int32_t sink,
                        cudaStream_t stream);

}  // namespace freqkv
