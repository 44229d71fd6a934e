// Decode-time attention over the cache (Section 3.4): declarations.
#pragma once
#include "common.cuh"

namespace freqkv {

constexpr int ATTEND_MAX_BATCH = 128;  // sequences per launch (lengths travel as kernel arguments)

bool attend_supported(int32_t head_dim, int32_t q_heads_per_kv);
// Row splits per (sequence, kv head) so that the launch fills the device.
int32_t attend_splits(int32_t batch, int32_t kv_heads, int32_t max_len, int32_t q_heads_per_kv, int32_t dtype, int sm_count);
size_t attend_partial_bytes(int32_t splits, int32_t batch, int32_t q_heads);
// table[pos][c] = (cos, sin)(pos * base^(-2c/128)), pos < rows, c < 64.
cudaError_t launch_rope_table(float2* table, int32_t rows, double base, cudaStream_t stream);
// q, out: [batch, kv_heads * g, 128] in the cache dtype; table may be null (no RoPE).
cudaError_t launch_attend(const freqkv_layout& l, const void* k, const void* v, int32_t layer, const void* q, void* out,
                          int32_t g, const int32_t* lens_host, const float2* table, float scale, int32_t splits,
                          float* partial, cudaStream_t stream);

}  // namespace freqkv
