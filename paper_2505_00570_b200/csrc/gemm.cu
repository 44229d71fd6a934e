#include "gemm.cuh"
namespace freqkv {
bool gemm_supported(int32_t, int32_t, int32_t, int32_t) { return false; }
cudaError_t launch_gemm(GemmState*, const CacheView&, const freqkv_layout&, void*, void*, int32_t, int32_t, const Basis&,
                        int32_t, int32_t*, int, cudaStream_t) { return cudaErrorNotSupported; }
void gemm_release(GemmState*) {}
}
