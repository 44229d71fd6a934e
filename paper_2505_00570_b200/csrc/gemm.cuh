// Tensor-core (tcgen05) execution of the compression Y = P X: declarations.
#pragma once
#include <vector>

#include "common.cuh"

namespace freqkv {

struct GemmState {
    const char* last_error = nullptr;
    int kernels_last_call = 0;
    bool attr_set = false;
    int max_clusters = 0;     // CTA pairs that can be resident at once
    void* scratch = nullptr;  // folded inputs U, V: [pairs][K|V][U|V][ceil(n_in/2)][128] bf16 per pass
    size_t scratch_bytes = 0;
    void* ragged_meta = nullptr;  // tensor maps, shapes and fold jobs of a ragged batch (device)
    size_t ragged_meta_bytes = 0;
    unsigned long long wait_limit_ns = 2000000000ull;  // bound of every mbarrier wait inside the kernel (2 s)
};

// Called on the launching stream right before and right after the tensor-core kernel itself
// (not the copy kernels around it), so that a caller can bracket it with events.
struct LaunchHooks {
    void (*before)(void* user, cudaStream_t stream) = nullptr;
    void (*after)(void* user, cudaStream_t stream) = nullptr;
    void* user = nullptr;
};

// Power-spectrum mode: device arrays [layers][kv_heads][n_in] (either may be null) that receive
// scale * (sum over the 128 channels of the squared DCT components), accumulated over the batch.
struct SpectrumOut {
    float* k = nullptr;
    float* v = nullptr;
    float scale = 1.f;
};

bool gemm_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep);
cudaError_t launch_gemm(GemmState* state, const CacheView& view, const Basis& basis, int32_t sink, int32_t* status_dev,
                        int sm_count, const LaunchHooks& hooks, cudaStream_t stream, const SpectrumOut* spectrum = nullptr);
cudaError_t gemm_prepare(GemmState* state, int32_t pairs, const Basis& basis, int sm_count);
// At most 256 kept rows: one tile per (batch, layer, kv_head), no fold pass, the dense basis (Basis::dense).
bool gemm_is_direct(int32_t n_keep);
// 0, 1 or 2 levels of the symmetry fold for a plain compression of these lengths (see gemm.cu).
int32_t gemm_fold_levels(int32_t n_in, int32_t n_keep, int32_t first);
cudaError_t launch_gemm_direct(GemmState* state, const CacheView& view, const Basis& basis, int32_t sink,
                               int32_t* status_dev, int sm_count, const LaunchHooks& hooks, cudaStream_t stream);
// One sequence of a ragged batch: its index in the cache and the (folded) basis of its lengths.
struct RaggedItem {
    int32_t batch_index;
    Basis basis;
};
// Every listed sequence in one fold launch and one tensor-core launch (each needs more than 256 kept
// rows: the folded form).  `view` covers the whole cache.  cudaErrorMemoryAllocation before anything is
// enqueued when the folded inputs do not fit: the caller then goes sequence by sequence.
cudaError_t launch_gemm_ragged(GemmState* state, const CacheView& view, const std::vector<RaggedItem>& items, int32_t sink,
                               int32_t* status_dev, int sm_count, const LaunchHooks& hooks, cudaStream_t stream);
void gemm_release(GemmState* state);
// A one-thread kernel that waits, with the tensor-core kernel's own bounded wait, on an mbarrier
// nothing arrives on: after `limit_ns` it sets a bit in *status_dev and returns.
cudaError_t launch_wait_probe(int32_t* status_dev, unsigned long long limit_ns, cudaStream_t stream);

}  // namespace freqkv
