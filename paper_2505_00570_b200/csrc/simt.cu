// CUDA-core (fp32 FFMA) execution of the compression Y = P X (Section 3.3, Eq. 2-3): the
// generic path for every shape and the only one that meets the fp32 tolerance for caches whose
// lengths are not powers of two.  One CTA computes a 64-row x 64-channel tile of one matrix's
// output with a classic shared-memory tiled product; results go to a scratch buffer and a
// second kernel copies them over rows [sink, sink + L) of the cache, because every output row
// depends on every input row of the same matrix and the two ranges overlap.
#include <algorithm>

#include "common.cuh"

namespace freqkv {
namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <typename T>
__device__ inline void load4(const T* p, float (&out)[4]);

template <>
__device__ inline void load4<float>(const float* p, float (&out)[4])
{
    const float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}

template <>
__device__ inline void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&out)[4])
{
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xffff0000u);
    out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xffff0000u);
}

__device__ inline void store4(float* p, const float (&v)[4])
{
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}

__device__ inline void store4(__nv_bfloat16* p, const float (&v)[4])
{
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(v[2], v[3]);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}

// grid: x = matrix (first + blockIdx.x), y = 64-row tile of the output, z = 64-channel tile.
template <typename T>
__global__ void __launch_bounds__(256) project_simt_kernel(CacheView view, int32_t first, const float* __restrict__ P,
                                                           int32_t ld, int32_t n_in, int32_t n_keep, int32_t sink,
                                                           T* __restrict__ scratch)
{
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN];

    const int32_t mat = first + blockIdx.x;
    const int32_t tensor = mat / view.mats_per_tensor;
    const T* x = static_cast<const T*>(tensor_base(view, tensor)) + matrix_offset(view, mat % view.mats_per_tensor) +
                 (int64_t)sink * view.stride_token;
    const int32_t m0 = blockIdx.y * TM, c0 = blockIdx.z * TN;
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;

    // loader roles
    const int a_m = tid / 4, a_k = (tid % 4) * 4;    // 64 rows x 16 k of P, float4 along k
    const int b_k = tid / 16, b_c = (tid % 16) * 4;  // 16 tokens x 64 channels of X, 4 channels each
    const bool b_c_ok = c0 + b_c < view.head_dim;

    float acc[4][4] = {};
    for (int32_t k0 = 0; k0 < n_in; k0 += TK) {
        {
            // P is zero-padded to whole tiles in both directions: no bounds checks needed.
            const float4 a = *reinterpret_cast<const float4*>(P + (int64_t)(m0 + a_m) * ld + k0 + a_k);
            As[a_k + 0][a_m] = a.x; As[a_k + 1][a_m] = a.y; As[a_k + 2][a_m] = a.z; As[a_k + 3][a_m] = a.w;
            float b[4] = {0.f, 0.f, 0.f, 0.f};
            if (b_c_ok && k0 + b_k < n_in) load4<T>(x + (int64_t)(k0 + b_k) * view.stride_token + c0 + b_c, b);
            Bs[b_k][b_c + 0] = b[0]; Bs[b_k][b_c + 1] = b[1]; Bs[b_k][b_c + 2] = b[2]; Bs[b_k][b_c + 3] = b[3];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

    const int32_t c = c0 + tx * 4;
    if (c < view.head_dim) {
        T* out = scratch + ((int64_t)blockIdx.x * n_keep) * view.head_dim;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int32_t m = m0 + ty * 4 + i;
            if (m < n_keep) store4(out + (int64_t)m * view.head_dim + c, acc[i]);
        }
    }
}

// One thread moves 16 bytes of one output row from the scratch buffer into the cache.
__global__ void copy_back_kernel(CacheView view, int32_t first, int32_t count, int32_t n_keep, int32_t sink,
                                 int32_t elt_size, const uint4* __restrict__ scratch)
{
    const int32_t vec_per_row = view.head_dim * elt_size / 16;
    const int64_t total = (int64_t)count * n_keep * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t vcol = (int32_t)(i % vec_per_row);
        const int64_t row = i / vec_per_row;
        const int32_t m = (int32_t)(row % n_keep);
        const int32_t mat = first + (int32_t)(row / n_keep);
        const int32_t tensor = mat / view.mats_per_tensor;
        const int64_t off = matrix_offset(view, mat % view.mats_per_tensor) + (int64_t)(sink + m) * view.stride_token;
        char* dst = static_cast<char*>(tensor_base(view, tensor)) + off * elt_size;
        reinterpret_cast<uint4*>(dst)[vcol] = scratch[i];
    }
}

constexpr int APPEND_MAX_BATCH = 128;
struct AppendLens {
    int32_t len[APPEND_MAX_BATCH];
};

// One thread moves 16 bytes of one new row.  new rows: [batch, layers, kv_heads, n_new, head_dim].
__global__ void append_kernel(CacheView view, int32_t batch, AppendLens lens, int32_t n_new, int32_t elt_size,
                              const uint4* __restrict__ new_k, const uint4* __restrict__ new_v)
{
    const int32_t vec_per_row = view.head_dim * elt_size / 16;
    const int32_t mats = batch * view.layers * view.kv_heads;
    const int64_t per_tensor = (int64_t)mats * n_new * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < 2 * per_tensor;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t tensor = i >= per_tensor;
        const int64_t j = i - tensor * per_tensor;
        const int32_t vcol = (int32_t)(j % vec_per_row);
        const int64_t row = j / vec_per_row;
        const int32_t r = (int32_t)(row % n_new);
        const int32_t idx = (int32_t)(row / n_new);  // (b, l, h) relative to batch0
        const int32_t b = idx / (view.layers * view.kv_heads);
        const int64_t off = matrix_offset(view, idx) + (int64_t)(lens.len[b] + r) * view.stride_token;
        char* dst = static_cast<char*>(tensor_base(view, tensor)) + off * elt_size;
        reinterpret_cast<uint4*>(dst)[vcol] = (tensor ? new_v : new_k)[j];
    }
}

// One new row per matrix (a decode step): one thread per 16 bytes, 32-bit index arithmetic, no grid-stride loop.
__global__ void __launch_bounds__(256) append_one_kernel(CacheView view, int32_t batch, AppendLens lens, int32_t elt_size,
                                                         const uint4* __restrict__ new_k, const uint4* __restrict__ new_v)
{
    const uint32_t vec_per_row = (uint32_t)(view.head_dim * elt_size / 16);
    const uint32_t per_tensor = (uint32_t)(batch * view.layers * view.kv_heads) * vec_per_row;
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 2 * per_tensor) return;
    const uint32_t tensor = i >= per_tensor, j = i - tensor * per_tensor;
    const uint32_t vcol = j % vec_per_row, idx = j / vec_per_row;
    const uint32_t b = idx / (uint32_t)(view.layers * view.kv_heads);
    const uint4 val = __ldg((tensor ? new_v : new_k) + j);
    const int64_t off = matrix_offset(view, (int32_t)idx) + (int64_t)lens.len[b] * view.stride_token;
    char* dst = static_cast<char*>(tensor_base(view, (int32_t)tensor)) + off * elt_size;
    reinterpret_cast<uint4*>(dst)[vcol] = val;
}

// Many new rows per matrix (prefill chunks): one block column per matrix, so that the matrix
// arithmetic is done once per thread and each thread then moves four 16-byte vectors per round,
// loads first.  Block (x, y): matrix x (K matrices first, then V), y-th share of its vectors.
__global__ void __launch_bounds__(256) append_rows_kernel(CacheView view, int32_t batch, AppendLens lens, int32_t n_new,
                                                          int32_t elt_size, const uint4* __restrict__ new_k,
                                                          const uint4* __restrict__ new_v)
{
    const uint32_t vec_per_row = (uint32_t)(view.head_dim * elt_size / 16);
    const uint32_t row_stride = (uint32_t)(view.stride_token * elt_size / 16);  // vectors between cache rows
    const int32_t mats = batch * view.layers * view.kv_heads;
    const int32_t tensor = (int32_t)blockIdx.x >= mats;
    const int32_t idx = (int32_t)blockIdx.x - tensor * mats;
    const int32_t b = idx / (view.layers * view.kv_heads);
    const uint32_t total = (uint32_t)n_new * vec_per_row;
    const uint4* src = (tensor ? new_v : new_k) + (int64_t)idx * total;
    uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(tensor_base(view, tensor)) +
                                          (matrix_offset(view, idx) + (int64_t)lens.len[b] * view.stride_token) * elt_size);
    const uint32_t stride = gridDim.y * blockDim.x;
    for (uint32_t i0 = blockIdx.y * blockDim.x + threadIdx.x; i0 < total; i0 += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t i = i0 + j * stride;
            if (i < total) v[j] = __ldg(src + i);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t i = i0 + j * stride;
            if (i < total) {
                const uint32_t r = i / vec_per_row, vcol = i - r * vec_per_row;
                dst[(size_t)r * row_stride + vcol] = v[j];
            }
        }
    }
}

// ---- decode step with the lengths on the device (replayed as a CUDA graph, see api.cu) ----

// One thread: decide whether this step must compress first.  Every sequence full -> the
// conditional body (the compression) runs; none full -> it is skipped; some but not all full ->
// the batch is not uniform, which this path does not take: an error bit is set, nothing is
// compressed and the full sequences are not appended to.
__global__ void decode_trigger_kernel(const int32_t* __restrict__ lens, int32_t batch, int32_t capacity,
                                      cudaGraphConditionalHandle handle, int32_t* status)
{
    int32_t full = 0;
    for (int32_t b = 0; b < batch; ++b) full += lens[b] >= capacity;
    if (full != 0 && full != batch) atomicOr(status, DECODE_ERR_MIXED_LENGTHS);
    cudaGraphSetConditional(handle, full == batch ? 1u : 0u);
}

__global__ void decode_set_lens_kernel(int32_t* lens, int32_t batch, int32_t value)
{
    const int32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) lens[b] = value;
}

// One new row per matrix, written at the sequence's device-resident length (full sequences are skipped).
// One thread per 16 bytes; 32-bit index arithmetic when the count allows it.
template <typename I>
__global__ void __launch_bounds__(256) decode_append_kernel(CacheView view, int32_t batch, const int32_t* __restrict__ lens,
                                                            int32_t capacity, int32_t elt_size, const uint4* __restrict__ new_k,
                                                            const uint4* __restrict__ new_v)
{
    const I vec_per_row = (I)(view.head_dim * elt_size / 16);
    const I per_tensor = (I)batch * (I)(view.layers * view.kv_heads) * vec_per_row;
    const I i = (I)blockIdx.x * (I)blockDim.x + (I)threadIdx.x;
    if (i >= 2 * per_tensor) return;
    const I tensor = i >= per_tensor ? 1 : 0, j = i - tensor * per_tensor;
    const I vcol = j % vec_per_row, idx = j / vec_per_row;
    const int32_t b = (int32_t)(idx / (I)(view.layers * view.kv_heads));
    const int32_t len = lens[b];
    if (len >= capacity) return;
    const uint4 val = __ldg((tensor ? new_v : new_k) + j);
    const int64_t off = matrix_offset(view, (int32_t)idx) + (int64_t)len * view.stride_token;
    char* dst = static_cast<char*>(tensor_base(view, (int32_t)tensor)) + off * elt_size;
    reinterpret_cast<uint4*>(dst)[vcol] = val;
}

__global__ void decode_advance_kernel(int32_t* lens, int32_t batch, int32_t capacity)
{
    const int32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch && lens[b] < capacity) lens[b] += 1;
}

unsigned grid_for(int64_t work_items, int threads)
{
    int64_t blocks = (work_items + threads - 1) / threads;
    const int64_t cap = 148 * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (unsigned)blocks;
}

}  // namespace

cudaError_t launch_project_simt(const CacheView& view, int32_t dtype, int32_t first, int32_t count, const Basis& basis,
                                int32_t sink, void* scratch, cudaStream_t stream)
{
    if (count <= 0) return cudaSuccess;
    const dim3 grid((unsigned)count, (unsigned)((basis.n_keep + TM - 1) / TM), (unsigned)((view.head_dim + TN - 1) / TN));
    if (dtype == FREQKV_F32)
        project_simt_kernel<float><<<grid, 256, 0, stream>>>(view, first, basis.f32, basis.ld, basis.n_in, basis.n_keep,
                                                             sink, static_cast<float*>(scratch));
    else
        project_simt_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(view, first, basis.f32, basis.ld, basis.n_in,
                                                                     basis.n_keep, sink,
                                                                     static_cast<__nv_bfloat16*>(scratch));
    return cudaGetLastError();
}

cudaError_t launch_copy_back(const CacheView& view, int32_t dtype, int32_t first, int32_t count, int32_t n_keep,
                             int32_t sink, const void* scratch, cudaStream_t stream)
{
    if (count <= 0 || n_keep <= 0) return cudaSuccess;
    const int32_t elt = (int32_t)dtype_size(dtype);
    const int64_t total = (int64_t)count * n_keep * (view.head_dim * elt / 16);
    copy_back_kernel<<<grid_for(total, 256), 256, 0, stream>>>(view, first, count, n_keep, sink, elt,
                                                               static_cast<const uint4*>(scratch));
    return cudaGetLastError();
}

cudaError_t add_decode_trigger_node(cudaGraph_t graph, cudaGraphNode_t* node, const int32_t* lens, int32_t batch,
                                    int32_t capacity, cudaGraphConditionalHandle handle, int32_t* status)
{
    void* args[] = {(void*)&lens, (void*)&batch, (void*)&capacity, (void*)&handle, (void*)&status};
    cudaKernelNodeParams kp = {};
    kp.func = (void*)decode_trigger_kernel;
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(1);
    kp.kernelParams = args;
    return cudaGraphAddKernelNode(node, graph, nullptr, 0, &kp);
}

cudaError_t launch_decode_set_lens(int32_t* lens, int32_t batch, int32_t value, cudaStream_t stream)
{
    decode_set_lens_kernel<<<(batch + 255) / 256, 256, 0, stream>>>(lens, batch, value);
    return cudaGetLastError();
}

cudaError_t launch_decode_append(const CacheView& view, int32_t dtype, int32_t batch, int32_t* lens, int32_t capacity,
                                 const void* new_k, const void* new_v, cudaStream_t stream)
{
    const int32_t elt = (int32_t)dtype_size(dtype);
    const int64_t vecs = (int64_t)2 * batch * view.layers * view.kv_heads * (view.head_dim * elt / 16);
    const unsigned blocks = (unsigned)((vecs + 255) / 256);
    if (vecs < ((int64_t)1 << 31))
        decode_append_kernel<uint32_t><<<blocks, 256, 0, stream>>>(view, batch, lens, capacity, elt, static_cast<const uint4*>(new_k),
                                                                  static_cast<const uint4*>(new_v));
    else
        decode_append_kernel<uint64_t><<<blocks, 256, 0, stream>>>(view, batch, lens, capacity, elt, static_cast<const uint4*>(new_k),
                                                                  static_cast<const uint4*>(new_v));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    decode_advance_kernel<<<(batch + 255) / 256, 256, 0, stream>>>(lens, batch, capacity);
    return cudaGetLastError();
}

cudaError_t launch_append(const CacheView& view, int32_t dtype, int32_t batch, const int32_t* lens_host, int32_t n_new,
                          const void* new_k, const void* new_v, cudaStream_t stream)
{
    const int32_t elt = (int32_t)dtype_size(dtype);
    const int64_t row_vecs = (int64_t)view.head_dim * elt / 16;
    const int64_t seq_vecs = (int64_t)view.layers * view.kv_heads * n_new * row_vecs;  // per sequence, per tensor
    for (int32_t b0 = 0; b0 < batch; b0 += APPEND_MAX_BATCH) {
        const int32_t nb = batch - b0 < APPEND_MAX_BATCH ? batch - b0 : APPEND_MAX_BATCH;
        AppendLens lens;
        for (int32_t i = 0; i < nb; ++i) lens.len[i] = lens_host[b0 + i];
        CacheView sub = view;
        sub.batch0 = view.batch0 + b0;
        const uint4* nk = static_cast<const uint4*>(new_k) + (int64_t)b0 * seq_vecs;
        const uint4* nv = static_cast<const uint4*>(new_v) + (int64_t)b0 * seq_vecs;
        const int64_t mat_vecs = (int64_t)n_new * row_vecs;  // per matrix
        const int64_t mats2 = (int64_t)2 * nb * view.layers * view.kv_heads;
        if (mat_vecs >= 4096 && mat_vecs < ((int64_t)1 << 31) && mats2 < ((int64_t)1 << 31)) {
            const unsigned gy = (unsigned)std::min<int64_t>((mat_vecs + 1023) / 1024, 64);
            append_rows_kernel<<<dim3((unsigned)mats2, gy), 256, 0, stream>>>(sub, nb, lens, n_new, elt, nk, nv);
        } else if (n_new == 1 && 2 * nb * seq_vecs < ((int64_t)1 << 31)) {
            append_one_kernel<<<(unsigned)((2 * nb * seq_vecs + 255) / 256), 256, 0, stream>>>(sub, nb, lens, elt, nk, nv);
        } else {
            append_kernel<<<grid_for(2 * nb * seq_vecs, 256), 256, 0, stream>>>(sub, nb, lens, n_new, elt, nk, nv);
        }
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace freqkv
