// Tensor-core (tcgen05) execution of the compression Y = P X: declarations.
#pragma once
#include "common.cuh"

namespace freqkv {

struct GemmState {
    const char* last_error = nullptr;
};

bool gemm_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep);
cudaError_t launch_gemm(GemmState* state, const CacheView& view, const freqkv_layout& layout, void* k, void* v,
                        int32_t batch0, int32_t batch_count, const Basis& basis, int32_t sink, int32_t* status_dev,
                        int sm_count, cudaStream_t stream);
void gemm_release(GemmState* state);

}  // namespace freqkv
