// Shared declarations of the FreqKV CUDA library (internal; the public surface is
// include/freqkv.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "freqkv.h"

namespace freqkv {

// Device-side view of the K and V caches: matrix i of a call is tensor i / mats_per_tensor
// (0 = K, 1 = V), and inside the tensor (batch, layer, kv_head) in row-major order.
struct CacheView {
    void* base[2];
    int64_t stride_batch, stride_layer, stride_head, stride_token;  // elements
    int32_t layers, kv_heads, head_dim;
    int32_t mats_per_tensor;  // batch * layers * kv_heads
    int32_t batch0;           // first batch index covered (ragged calls address one sequence)
};

__host__ __device__ inline int64_t matrix_offset(const CacheView& v, int32_t idx_in_tensor)
{
    const int32_t h = idx_in_tensor % v.kv_heads;
    const int32_t l = (idx_in_tensor / v.kv_heads) % v.layers;
    const int32_t b = idx_in_tensor / (v.kv_heads * v.layers) + v.batch0;
    return (int64_t)b * v.stride_batch + (int64_t)l * v.stride_layer + (int64_t)h * v.stride_head;
}

__host__ __device__ inline void* tensor_base(const CacheView& v, int32_t tensor)
{
    return tensor ? v.base[1] : v.base[0];  // a select, not an indexed load of the parameter struct
}

// Projection basis of one (n_in, n_keep) pair: P[m][n], row-major with leading dimension ld,
// rows padded to rows_pad and columns to ld with zeros.
struct Basis {
    float* f32 = nullptr;  // SIMT path
    int32_t n_in = 0, n_keep = 0, ld = 0, rows_pad = 0;
    int32_t first = 0;     // first retained DCT component (0 = the lowest n_keep components)
    // Tensor-core path: the even-frequency and odd-frequency parts Pe, Po of P restricted to
    // m < ceil(n_keep/2), n < ceil(n_in/2), bf16, two planes of fold_rows_pad x fold_ld (see basis.cu).
    __nv_bfloat16* fold = nullptr;
    int32_t fold_ld = 0, fold_rows_pad = 0;
    // The same folded once more, where the lengths allow it (n_in a multiple of 4, n_keep even, first = 0):
    // Pe is itself the basis of a half-size compression, so it splits again into Pee | Peo; four planes of
    // fold2_rows_pad x fold_ld -- Pee, Peo, the first ceil(n_keep/4) rows of Po, and the mirrored rows
    // Po[n_keep/2 - 1 - m] -- stored behind the two planes above in the same allocation (see basis.cu).
    __nv_bfloat16* fold2 = nullptr;
    int32_t fold2_rows_pad = 0;
    int64_t fold_alloc_elems = 0;  // bf16 elements of the allocation `fold` points to
    // Tensor-core path for at most 256 kept rows: the whole P in bf16, dense_rows_pad (256) x ld.
    __nv_bfloat16* dense = nullptr;
    int32_t dense_rows_pad = 0;
};

// ---- kernel launchers (each returns the cudaError_t of its launch) ----

// P[m][n] for m < n_keep, n < n_in from the closed form; zero padding elsewhere.
// (`first` = index of the first retained DCT component; 0 for the method's low-pass compression)
cudaError_t launch_build_basis(float* p_f32, __nv_bfloat16* p_bf16, int32_t n_in, int32_t n_keep, int32_t first,
                               int32_t ld, int32_t rows_pad, cudaStream_t stream);

// Pee, Peo, Po (first rows) and Po (mirrored rows) of the twice-folded basis: four planes of rows_pad x ld.
cudaError_t launch_build_folded2_basis(__nv_bfloat16* out, int32_t n_in, int32_t n_keep, int32_t ld, int32_t rows_pad,
                                       cudaStream_t stream);

// Pe and Po of the folded basis (two planes of rows_pad x ld), zero padding elsewhere.
cudaError_t launch_build_folded_basis(__nv_bfloat16* out, int32_t n_in, int32_t n_keep, int32_t first, int32_t ld,
                                      int32_t rows_pad, cudaStream_t stream);

// Even rows | odd rows of the orthonormal N-point DCT-II, restricted to n < ceil(N/2) (two planes of rows_pad x ld).
cudaError_t launch_build_dct_folded(__nv_bfloat16* out, int32_t n_in, int32_t ld, int32_t rows_pad, cudaStream_t stream);

// scratch[i - first][m][c] = sum_n P[m][n] * X_i[sink + n][c] for matrices first .. first+count-1.
cudaError_t launch_project_simt(const CacheView& view, int32_t dtype, int32_t first, int32_t count, const Basis& basis,
                                int32_t sink, void* scratch, cudaStream_t stream);

// cache rows [sink, sink + n_keep) of matrices first .. first+count-1 <- scratch.
cudaError_t launch_copy_back(const CacheView& view, int32_t dtype, int32_t first, int32_t count, int32_t n_keep,
                             int32_t sink, const void* scratch, cudaStream_t stream);

// rows [lens[b], lens[b] + n_new) of every matrix <- new rows.
cudaError_t launch_append(const CacheView& view, int32_t dtype, int32_t batch, const int32_t* lens_host,
                          int32_t n_new, const void* new_k, const void* new_v, cudaStream_t stream);

// Decode step with device-resident lengths (pieces of the graph api.cu builds).
constexpr int32_t DECODE_ERR_MIXED_LENGTHS = 0x100;  // status-word bit: some but not all sequences were full
cudaError_t add_decode_trigger_node(cudaGraph_t graph, cudaGraphNode_t* node, const int32_t* lens, int32_t batch,
                                    int32_t capacity, cudaGraphConditionalHandle handle, int32_t* status);
cudaError_t launch_decode_set_lens(int32_t* lens, int32_t batch, int32_t value, cudaStream_t stream);
// rows at lens[b] <- the new rows ([batch, layers, kv_heads, 1, head_dim]), then lens[b] += 1 (full sequences skipped)
cudaError_t launch_decode_append(const CacheView& view, int32_t dtype, int32_t batch, int32_t* lens, int32_t capacity,
                                 const void* new_k, const void* new_v, cudaStream_t stream);

// Set-up that must run once per DEVICE (cudaFuncSetAttribute applies to the current device only):
// run(f) calls f() the first time it is reached with a given device current, under a mutex.
struct PerDeviceOnce {
    std::mutex mutex;
    bool done[64] = {};
    template <class F>
    cudaError_t run(F&& f)
    {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        std::lock_guard<std::mutex> lock(mutex);
        if (dev < 0 || dev >= 64) return f();
        if (done[dev]) return cudaSuccess;
        e = f();
        if (e == cudaSuccess) done[dev] = true;
        return e;
    }
};

inline size_t dtype_size(int32_t dtype) { return dtype == FREQKV_F32 ? 4 : 2; }

}  // namespace freqkv
