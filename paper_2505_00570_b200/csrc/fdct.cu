#include "fdct.cuh"
namespace freqkv {
bool fdct_supported(int32_t, int32_t, int32_t, int32_t) { return false; }
cudaError_t fdct_make_plan(int32_t, int32_t, cudaStream_t, FdctPlan*) { return cudaErrorNotSupported; }
void fdct_free_plan(FdctPlan*) {}
cudaError_t launch_fdct(const CacheView&, int32_t, int32_t, const FdctPlan&, int32_t, cudaStream_t) { return cudaErrorNotSupported; }
}
