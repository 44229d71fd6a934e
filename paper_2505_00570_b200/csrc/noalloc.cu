// freqkv_compress_noalloc: the CUDA-core compression for callers that must not allocate.
//
// Some callers cannot call cudaMalloc at all: code holding a lock that the allocator's implicit
// device synchronisation would deadlock against, real-time serving loops with a frozen memory
// budget, and plug-ins whose host framework owns every byte of device memory.
// freqkv_compress needs a context (freqkv_create allocates) plus a plan and an output staging
// buffer obtained from cudaMalloc on first use.  This entry point needs none of that: the
// projection basis and the output staging live in two file-scope __device__ arrays of fixed
// size, which every GPU that loads the library holds until the process exits.
//
// In host code the names g_basis / g_staging are host-side stand-ins for the device symbols, not
// device addresses: handing them to a kernel would make it fault or touch the wrong memory.  The
// device addresses are looked up once per device with cudaGetSymbolAddress, with that device
// current, and those addresses are what the kernels receive.
#include <algorithm>
#include <mutex>

#include "common.cuh"

namespace freqkv {
namespace {

constexpr size_t kBasisElems = FREQKV_NOALLOC_MAX_BASIS_ELEMS;   // fp32 entries of the padded basis
constexpr size_t kStagingBytes = FREQKV_NOALLOC_STAGING_BYTES;   // compressed rows awaiting copy-back

static __device__ __align__(256) float g_basis[kBasisElems];
static __device__ __align__(256) unsigned char g_staging[kStagingBytes];

constexpr int kMaxDevices = 64;
struct DeviceArrays {
    bool ready = false;
    float* basis = nullptr;
    void* staging = nullptr;
};
DeviceArrays g_devices[kMaxDevices];
std::mutex g_mutex;

// Device addresses of the two arrays on `device`, which must be the current device.
cudaError_t arrays_for(int device, DeviceArrays* out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceArrays& d = g_devices[device];
    if (!d.ready) {
        float* b = nullptr;
        void* s = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&b), g_basis);
        if (e != cudaSuccess) return e;
        e = cudaGetSymbolAddress(&s, g_staging);
        if (e != cudaSuccess) return e;
        d.basis = b;
        d.staging = s;
        d.ready = true;
    }
    *out = d;
    return cudaSuccess;
}

}  // namespace
}  // namespace freqkv

using namespace freqkv;

extern "C" freqkv_status freqkv_compress_noalloc(const freqkv_layout* layout, void* k, void* v, int32_t cache_len,
                                                 int32_t kept_len, int32_t sink, void* cuda_stream)
{
    freqkv_status st = freqkv_check_compress(layout, k, v, cache_len, kept_len, sink);
    if (st != FREQKV_OK) return st;
    const int32_t n_in = cache_len - sink;
    if (n_in == 0 || kept_len == 0 || kept_len == n_in) return FREQKV_OK;  // nothing to rewrite

    // Size limits of the fixed arrays, checked before anything is enqueued.
    Basis basis;
    basis.n_in = n_in;
    basis.n_keep = kept_len;
    basis.ld = (n_in + 63) / 64 * 64;
    basis.rows_pad = (kept_len + 63) / 64 * 64;
    if ((size_t)basis.ld * basis.rows_pad > kBasisElems) return FREQKV_ERR_UNSUPPORTED;
    const size_t per_matrix = (size_t)kept_len * layout->head_dim * dtype_size(layout->dtype);
    if (per_matrix > kStagingBytes) return FREQKV_ERR_UNSUPPORTED;

    // The arrays used are those of the device that owns the cache: K and V must be plain device
    // memory of one and the same device.
    cudaPointerAttributes attr, attr_v;
    if (cudaPointerGetAttributes(&attr, k) != cudaSuccess || attr.type != cudaMemoryTypeDevice ||
        cudaPointerGetAttributes(&attr_v, v) != cudaSuccess || attr_v.type != cudaMemoryTypeDevice ||
        attr_v.device != attr.device) {
        cudaGetLastError();
        return FREQKV_ERR_INVALID_ARG;
    }
    const int device = attr.device;
    if (device < 0 || device >= kMaxDevices) return FREQKV_ERR_UNSUPPORTED;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return FREQKV_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return FREQKV_ERR_CUDA;

    freqkv_status result = FREQKV_OK;
    DeviceArrays arrays;
    if (arrays_for(device, &arrays) != cudaSuccess) {
        result = FREQKV_ERR_CUDA;
    } else {
        cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
        basis.f32 = arrays.basis;
        CacheView view;
        view.base[0] = k;
        view.base[1] = v;
        view.stride_batch = layout->stride_batch;
        view.stride_layer = layout->stride_layer;
        view.stride_head = layout->stride_head;
        view.stride_token = layout->stride_token;
        view.layers = layout->layers;
        view.kv_heads = layout->kv_heads;
        view.head_dim = layout->head_dim;
        view.mats_per_tensor = layout->batch * layout->layers * layout->kv_heads;
        view.batch0 = 0;
        const int32_t n_mat = 2 * view.mats_per_tensor;
        const int32_t chunk = (int32_t)std::min<size_t>(kStagingBytes / per_matrix, (size_t)n_mat);
        // The basis array keeps whatever the previous call left: the builder rewrites the whole
        // padded rectangle this call reads, zeros included.
        cudaError_t e = launch_build_basis(arrays.basis, nullptr, n_in, kept_len, 0, basis.ld, basis.rows_pad, stream);
        for (int32_t first = 0; e == cudaSuccess && first < n_mat; first += chunk) {
            const int32_t count = std::min(chunk, n_mat - first);
            e = launch_project_simt(view, layout->dtype, first, count, basis, sink, arrays.staging, stream);
            if (e == cudaSuccess)
                e = launch_copy_back(view, layout->dtype, first, count, kept_len, sink, arrays.staging, stream);
        }
        if (e != cudaSuccess) {
            cudaGetLastError();
            result = FREQKV_ERR_CUDA;
        }
    }
    if (prev != device) cudaSetDevice(prev);
    return result;
}
