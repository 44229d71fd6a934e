// Attention of a chunk of incoming tokens over the cache (Section 3.3, chunk-wise prefilling): declarations.
#pragma once
#include "common.cuh"

namespace freqkv {

constexpr int PREFILL_MAX_BATCH = 128;            // sequences per launch (lengths travel as kernel arguments)
constexpr int32_t PREFILL_ERR_WAIT = 0x200;       // status-word bit: a barrier wait of the kernel ran out

bool prefill_supported(int32_t dtype, int32_t head_dim, int32_t q_heads_per_kv);
// Scratch for the rotated keys of one layer (fp16) and for the rotated, scaled queries of the chunk (fp16).
size_t prefill_key_scratch_bytes(const freqkv_layout& l);
size_t prefill_query_scratch_bytes(const freqkv_layout& l, int32_t q_heads_per_kv, int32_t n_new);
// q, out: [batch, kv_heads * g, n_new, 128] bf16; table: [capacity][64] (cos, sin) or null (no RoPE);
// status: device status word (bits are OR-ed in); wait_limit_ns: bound of every barrier wait in the kernel; *error receives a message when the launch cannot be set up.
cudaError_t launch_prefill(const freqkv_layout& l, const void* k, const void* v, int32_t layer, const void* q, void* out,
                           int32_t g, int32_t n_new, const int32_t* lens_host, const float2* table, float scale,
                           void* key_scratch, void* query_scratch, int32_t* status, unsigned long long wait_limit_ns,
                           const char** error, int32_t* kernels_launched, cudaStream_t stream);

}  // namespace freqkv
