// C ABI of the FreqKV library: argument validation, plan cache, variant choice and dispatch.
// All arithmetic of the hot path runs in the kernels this file launches; nothing here touches
// cache contents on the host.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <tuple>
#include <utility>
#include <vector>

#include "common.cuh"
#include "gemm.cuh"
#include "fdct.cuh"
#include "dctmm.cuh"
#include "attend.cuh"
#include "prefill.cuh"

using namespace freqkv;

struct freqkv_ctx {
    int device = 0;
    int sm_count = 0;
    freqkv_variant forced = FREQKV_AUTO;
    std::map<std::tuple<int32_t, int32_t, int32_t>, Basis> bases;  // (n_in, n_keep, first retained component)
    std::map<std::pair<int32_t, int32_t>, FdctPlan> fdct_plans;
    // keys: (n_in, n_keep, family of factorisation asked for: 0 = the kernel's own choice)
    std::map<std::tuple<int32_t, int32_t, int32_t>, DctmmPlan> dctmm_plans;
    std::map<std::tuple<int32_t, int32_t, int32_t>, bool> dctmm_fits;  // does a factorisation meet the kernel's limits
    int32_t fast_family = 0;
    size_t basis_bytes = 0;
    void* scratch = nullptr;
    size_t scratch_bytes = 0;
    int32_t* status_dev = nullptr;
    GemmState gemm;
    std::string last_error;
    // Work areas (fold scratch, staging, attention partials) are shared by all calls on this
    // context: a call on another stream than the previous one first waits for that one's work.
    cudaEvent_t work_done = nullptr;
    cudaStream_t work_stream = nullptr;
    bool work_recorded = false;
    // instrumentation
    bool timing = false;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> pending, spare;
    int64_t kernels_launched = 0;
    // host-buffer entry point: device staging caches
    void* stage[2] = {nullptr, nullptr};
    size_t stage_bytes = 0;
    // decode attention: RoPE table of one base, partial results of the row splits
    float2* rope_table = nullptr;
    int32_t rope_rows = 0;
    double rope_base = 0.0;
    float* attend_partial = nullptr;
    size_t attend_partial_bytes = 0;
    void* prefill_keys = nullptr;     // rotated keys of one layer, fp16
    size_t prefill_keys_bytes = 0;
    void* prefill_queries = nullptr;  // rotated, scaled queries of one chunk, fp16
    size_t prefill_queries_bytes = 0;
    cudaStream_t pipe[3] = {nullptr, nullptr, nullptr};  // copy in, compress, copy out
    cudaEvent_t pipe_begin = nullptr, pipe_end = nullptr;
    std::vector<cudaEvent_t> pipe_events;                // per group: copied in, compressed
};

namespace {

constexpr size_t kScratchChunkBytes = size_t(1) << 30;  // per-chunk output staging of the scratch paths
constexpr int32_t kDctRows = -1;  // plan key of the plain DCT matrix (power spectrum) among the retained-band offsets
constexpr size_t kBasisBudgetBytes = size_t(12) << 30;  // plan cache is flushed beyond this

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// Orders the calls that use the context's work areas: on entry the caller's stream waits for the
// previous such call if that one ran on a different stream; on exit the end of this call's work
// is recorded.  (Calls on one stream are ordered anyway and pay nothing.)
struct WorkOrder {
    freqkv_ctx* ctx;
    cudaStream_t stream;
    WorkOrder(freqkv_ctx* c, cudaStream_t s);
    ~WorkOrder();
};

freqkv_status cuda_fail(freqkv_ctx* ctx, cudaError_t e, const char* where)
{
    if (ctx) ctx->last_error = std::string(where) + ": " + cudaGetErrorString(e);
    cudaGetLastError();  // clear the sticky-free error state
    return e == cudaErrorMemoryAllocation ? FREQKV_ERR_ALLOC : FREQKV_ERR_CUDA;
}

#define FREQKV_CUDA(ctx, call)                                             \
    do {                                                                   \
        const cudaError_t e__ = (call);                                    \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__, #call);       \
    } while (0)

WorkOrder::WorkOrder(freqkv_ctx* c, cudaStream_t s) : ctx(c), stream(s)
{
    if (ctx->work_recorded && ctx->work_stream != stream) cudaStreamWaitEvent(stream, ctx->work_done, 0);
}

WorkOrder::~WorkOrder()
{
    if (!ctx->work_done && cudaEventCreateWithFlags(&ctx->work_done, cudaEventDisableTiming) != cudaSuccess) {
        ctx->work_done = nullptr;
        cudaGetLastError();
        return;
    }
    if (cudaEventRecord(ctx->work_done, stream) == cudaSuccess) {
        ctx->work_stream = stream;
        ctx->work_recorded = true;
    } else {
        cudaGetLastError();
    }
}

int64_t span_elements(const freqkv_layout& l)
{
    return (int64_t)(l.batch - 1) * l.stride_batch + (int64_t)(l.layers - 1) * l.stride_layer +
           (int64_t)(l.kv_heads - 1) * l.stride_head + (int64_t)(l.capacity - 1) * l.stride_token + l.head_dim;
}

freqkv_status check_layout(const freqkv_layout* l)
{
    if (!l) return FREQKV_ERR_INVALID_ARG;
    if (l->dtype != FREQKV_BF16 && l->dtype != FREQKV_F32) return FREQKV_ERR_UNSUPPORTED;
    if (l->batch < 1 || l->layers < 1 || l->kv_heads < 1 || l->capacity < 1 || l->head_dim < 1)
        return FREQKV_ERR_INVALID_ARG;
    if (l->head_dim % 8 != 0 || l->head_dim > 256) return FREQKV_ERR_UNSUPPORTED;
    if ((int64_t)l->batch * l->layers * l->kv_heads > (int64_t)1 << 29) return FREQKV_ERR_UNSUPPORTED;
    const int64_t strides[4] = {l->stride_token, l->stride_head, l->stride_layer, l->stride_batch};
    const int64_t extents[4] = {l->capacity, l->kv_heads, l->layers, l->batch};
    for (int i = 0; i < 4; ++i) {
        if (strides[i] < 0) return FREQKV_ERR_INVALID_ARG;
        if (strides[i] % 8 != 0) return FREQKV_ERR_UNSUPPORTED;
    }
    // No two matrices may overlap: ordered by stride, each axis must step over the whole extent
    // of the axes below it (axes of extent 1 never step).
    std::vector<std::pair<int64_t, int64_t>> axes;  // (stride, extent)
    for (int i = 0; i < 4; ++i)
        if (extents[i] > 1) axes.emplace_back(strides[i], extents[i]);
    std::sort(axes.begin(), axes.end());
    int64_t below = l->head_dim;
    for (const auto& a : axes) {
        if (a.first < below) return FREQKV_ERR_UNSUPPORTED;
        below = a.first * a.second;
    }
    if (l->stride_token < l->head_dim && l->capacity > 1) return FREQKV_ERR_UNSUPPORTED;
    return FREQKV_OK;
}

freqkv_status check_tensors(const freqkv_layout& l, const void* k, const void* v)
{
    if (!k || !v) return FREQKV_ERR_INVALID_ARG;
    if (((uintptr_t)k | (uintptr_t)v) & 15) return FREQKV_ERR_UNSUPPORTED;
    const int64_t bytes = span_elements(l) * (int64_t)dtype_size(l.dtype);
    const char* a = static_cast<const char*>(k);
    const char* b = static_cast<const char*>(v);
    if (a < b + bytes && b < a + bytes) return FREQKV_ERR_INVALID_ARG;  // K and V overlap
    return FREQKV_OK;
}

CacheView make_view(const freqkv_layout& l, void* k, void* v, int32_t batch0, int32_t batch_count)
{
    CacheView w;
    w.base[0] = k;
    w.base[1] = v;
    w.stride_batch = l.stride_batch;
    w.stride_layer = l.stride_layer;
    w.stride_head = l.stride_head;
    w.stride_token = l.stride_token;
    w.layers = l.layers;
    w.kv_heads = l.kv_heads;
    w.head_dim = l.head_dim;
    w.mats_per_tensor = batch_count * l.layers * l.kv_heads;
    w.batch0 = batch0;
    return w;
}

bool is_pow2(int32_t x) { return x > 0 && (x & (x - 1)) == 0; }

bool gemm_applicable(const freqkv_layout& l, int32_t n_in, int32_t n_keep)
{
    return gemm_supported(l.dtype, l.head_dim, n_in, n_keep);
}

bool fdct_applicable(const freqkv_layout& l, int32_t n_in, int32_t n_keep)
{
    return fdct_supported(l.dtype, l.head_dim, n_in, n_keep) && is_pow2(n_in) && is_pow2(n_keep);
}

// The fast transform as tensor-core stages: bf16 caches whose lengths factor within the kernel's limits.
bool dctmm_applicable(freqkv_ctx* ctx, const freqkv_layout& l, int32_t n_in, int32_t n_keep)
{
    if (l.dtype != FREQKV_BF16 || l.head_dim % 8 != 0) return false;
    const auto key = std::make_tuple(n_in, n_keep, ctx->fast_family);
    auto it = ctx->dctmm_fits.find(key);
    if (it != ctx->dctmm_fits.end()) return it->second;
    const bool ok = dctmm_supported(l.dtype, l.head_dim, n_in, n_keep, ctx->fast_family);
    if (ctx->dctmm_fits.size() > 4096) ctx->dctmm_fits.clear();
    ctx->dctmm_fits[key] = ok;
    return ok;
}

// Variant table, from measurements on B200 (7B shape, 2048 matrices of head_dim 128, bf16): the
// tensor-core projection takes 2.04 ms at 4092 -> 2046 (fold pass included; 2.02 ms at 4096 -> 2048)
// and the fast transform 2.49 ms (2.77 ms); at 4092 -> 1023, 3000 -> 1500 and 2046 -> 1023 the
// projection is 1.5 to 2.3 times faster (its work shrinks with both lengths, the fast transform's
// per-slab chain of steps does not), at 4092 -> 3069 they are level.  So bf16 caches with head_dim
// 128 go to the projection whenever a tile can be filled; the fast transform serves what the
// projection does not take (bf16 with other head sizes: 40 times faster there than the CUDA cores;
// fp32 caches of power-of-two length); everything else runs as a projection on the CUDA cores.
int32_t resolve(freqkv_ctx* ctx, const freqkv_layout& l, int32_t n_in, int32_t n_keep)
{
    const bool g = gemm_applicable(l, n_in, n_keep);
    const bool f = fdct_applicable(l, n_in, n_keep) || dctmm_applicable(ctx, l, n_in, n_keep);
    switch (ctx->forced) {
        case FREQKV_GEMM: return g ? FREQKV_GEMM : -1;
        case FREQKV_FDCT: return f ? FREQKV_FDCT : -1;
        case FREQKV_SIMT: return FREQKV_SIMT;
        default: break;
    }
    if (g && n_in >= 128) return FREQKV_GEMM;
    if (f) return FREQKV_FDCT;
    return FREQKV_SIMT;
}

void free_bases(freqkv_ctx* ctx)
{
    for (auto& kv : ctx->bases) {
        if (kv.second.f32) cudaFree(kv.second.f32);
        if (kv.second.fold) cudaFree(kv.second.fold);
        if (kv.second.dense) cudaFree(kv.second.dense);
    }
    ctx->bases.clear();
    ctx->basis_bytes = 0;
}

// Projection basis for (n_in, n_keep) holding at least the requested forms: the full fp32 matrix
// (CUDA-core path) and/or the folded bf16 pair Pe, Po (tensor-core path).
freqkv_status get_basis(freqkv_ctx* ctx, int32_t n_in, int32_t n_keep, int32_t first, bool need_f32, bool need_fold,
                        cudaStream_t stream, Basis* out)
{
    const auto key = std::make_tuple(n_in, n_keep, first);
    Basis b;
    auto it = ctx->bases.find(key);
    if (it != ctx->bases.end()) b = it->second;
    // the tensor-core path wants the folded pair, or, for few kept rows, the dense bf16 matrix
    const bool direct = need_fold && first != kDctRows && gemm_is_direct(n_keep);
    const bool make_f32 = need_f32 && !b.f32, make_fold = need_fold && !direct && !b.fold, make_dense = direct && !b.dense;
    if (make_f32 || make_fold || make_dense) {
        auto shape = [&](Basis& x) {
            x.n_in = n_in;
            x.n_keep = n_keep;
            x.first = first;
            x.ld = (n_in + 63) / 64 * 64;
            x.rows_pad = (n_keep + 63) / 64 * 64;
            x.fold_ld = ((n_in + 1) / 2 + 63) / 64 * 64;
            x.fold_rows_pad = ((n_keep + 1) / 2 + 255) / 256 * 256;
            x.dense_rows_pad = 256;
            // the second fold needs n_in / 2 and n_keep / 2 to be whole and n_in / 2 even
            x.fold2_rows_pad = (first == 0 && n_in % 4 == 0 && n_keep % 2 == 0) ? ((n_keep / 2 + 1) / 2 + 255) / 256 * 256 : 0;
        };
        shape(b);
        const size_t elems = (size_t)b.ld * b.rows_pad;
        const size_t fold1_elems = (size_t)2 * b.fold_ld * b.fold_rows_pad;
        const size_t fold_elems = fold1_elems + (size_t)4 * b.fold_ld * b.fold2_rows_pad;
        const size_t dense_elems = (size_t)256 * b.ld;
        const size_t want = (make_f32 ? elems * 4 : 0) + (make_fold ? fold_elems * 2 : 0) + (make_dense ? dense_elems * 2 : 0);
        if (ctx->basis_bytes + want > kBasisBudgetBytes) {
            FREQKV_CUDA(ctx, cudaDeviceSynchronize());  // bases may be in use by enqueued kernels
            free_bases(ctx);
            b = Basis();
            shape(b);
        }
        float* pf = nullptr;
        __nv_bfloat16* pb = nullptr;
        __nv_bfloat16* pd = nullptr;
        if (need_f32 && !b.f32) FREQKV_CUDA(ctx, cudaMalloc(&pf, elems * 4));
        if (direct && !b.dense) {
            const cudaError_t e = cudaMalloc(&pd, dense_elems * 2);
            if (e != cudaSuccess) {
                if (pf) cudaFree(pf);
                return cuda_fail(ctx, e, "cudaMalloc(basis)");
            }
        }
        if (need_fold && !direct && !b.fold) {
            const cudaError_t e = cudaMalloc(&pb, fold_elems * 2);
            if (e != cudaSuccess) {
                if (pf) cudaFree(pf);
                return cuda_fail(ctx, e, "cudaMalloc(basis)");
            }
        }
        cudaError_t e = cudaSuccess;
        if (pf) {
            e = launch_build_basis(pf, nullptr, n_in, n_keep, first, b.ld, b.rows_pad, stream);
            ctx->kernels_launched += 1;
        }
        if (e == cudaSuccess && pb) {
            e = first == kDctRows ? launch_build_dct_folded(pb, n_in, b.fold_ld, b.fold_rows_pad, stream)
                                  : launch_build_folded_basis(pb, n_in, n_keep, first, b.fold_ld, b.fold_rows_pad, stream);
            ctx->kernels_launched += 1;
            if (e == cudaSuccess && b.fold2_rows_pad) {
                e = launch_build_folded2_basis(pb + fold1_elems, n_in, n_keep, b.fold_ld, b.fold2_rows_pad, stream);
                ctx->kernels_launched += 1;
            }
        }
        if (e == cudaSuccess && pd) {
            e = launch_build_basis(nullptr, pd, n_in, n_keep, first, b.ld, 256, stream);
            ctx->kernels_launched += 1;
        }
        if (e != cudaSuccess) {
            if (pf) cudaFree(pf);
            if (pb) cudaFree(pb);
            if (pd) cudaFree(pd);
            return cuda_fail(ctx, e, "build_basis");
        }
        if (pd) { b.dense = pd; ctx->basis_bytes += dense_elems * 2; }
        if (pf) { b.f32 = pf; ctx->basis_bytes += elems * 4; }
        if (pb) {
            b.fold = pb;
            b.fold2 = b.fold2_rows_pad ? pb + fold1_elems : nullptr;
            b.fold_alloc_elems = (int64_t)fold_elems;
            ctx->basis_bytes += fold_elems * 2;
        }
        ctx->bases[key] = b;
    }
    *out = b;
    return FREQKV_OK;
}

size_t basis_device_bytes(const Basis& b)
{
    return (b.f32 ? (size_t)b.ld * b.rows_pad * 4 : 0) + (b.fold ? (size_t)b.fold_alloc_elems * 2 : 0) +
           (b.dense ? (size_t)256 * b.ld * 2 : 0);
}

// Remove the plan of (n_in, n_keep, first) from the cache without freeing it: the caller owns its
// device memory from now on (later calls on the context build a fresh one).
void disown_basis(freqkv_ctx* ctx, int32_t n_in, int32_t n_keep, int32_t first)
{
    auto it = ctx->bases.find(std::make_tuple(n_in, n_keep, first));
    if (it == ctx->bases.end()) return;
    const size_t bytes = basis_device_bytes(it->second);
    ctx->basis_bytes = ctx->basis_bytes > bytes ? ctx->basis_bytes - bytes : 0;
    ctx->bases.erase(it);
}

void free_basis(Basis* b)
{
    if (b->f32) cudaFree(b->f32);
    if (b->fold) cudaFree(b->fold);
    if (b->dense) cudaFree(b->dense);
    *b = Basis();
}

freqkv_status get_scratch(freqkv_ctx* ctx, size_t bytes, void** out)
{
    if (bytes > ctx->scratch_bytes) {
        if (ctx->scratch) {
            FREQKV_CUDA(ctx, cudaDeviceSynchronize());  // earlier launches may still read it
            cudaFree(ctx->scratch);
            ctx->scratch = nullptr;
            ctx->scratch_bytes = 0;
        }
        FREQKV_CUDA(ctx, cudaMalloc(&ctx->scratch, bytes));
        ctx->scratch_bytes = bytes;
    }
    *out = ctx->scratch;
    return FREQKV_OK;
}

struct TransformTimer {
    freqkv_ctx* ctx;
    cudaStream_t stream;
    std::pair<cudaEvent_t, cudaEvent_t> ev{nullptr, nullptr};
    TransformTimer(freqkv_ctx* c, cudaStream_t s) : ctx(c), stream(s) { begin(); }
    TransformTimer(freqkv_ctx* c, cudaStream_t s, bool start_now) : ctx(c), stream(s)
    {
        if (start_now) begin();
    }
    void begin()
    {
        if (!ctx->timing) return;
        if (!ctx->spare.empty()) {
            ev = ctx->spare.back();
            ctx->spare.pop_back();
        } else if (cudaEventCreate(&ev.first) != cudaSuccess || cudaEventCreate(&ev.second) != cudaSuccess) {
            ev = {nullptr, nullptr};
            cudaGetLastError();
            return;
        }
        cudaEventRecord(ev.first, stream);
    }
    void end()
    {
        if (!ev.first) return;
        cudaEventRecord(ev.second, stream);
        ctx->pending.push_back(ev);
        ev = {nullptr, nullptr};
    }
    ~TransformTimer() { end(); }
};

// Compress `count` sequences starting at batch0, all with the same (n_in, n_keep).
freqkv_status compress_group(freqkv_ctx* ctx, const freqkv_layout& l, void* k, void* v, int32_t batch0,
                             int32_t batch_count, int32_t n_in, int32_t n_keep, int32_t sink, int32_t variant,
                             cudaStream_t stream, int32_t first = 0, GemmState* own_gemm = nullptr,
                             const Basis* own_basis = nullptr)
{
    const CacheView view = make_view(l, k, v, batch0, batch_count);
    const int32_t n_mat = 2 * view.mats_per_tensor;

    if (variant == FREQKV_FDCT && first == 0 && dctmm_applicable(ctx, l, n_in, n_keep)) {
        DctmmPlan plan;
        const auto key = std::make_tuple(n_in, n_keep, ctx->fast_family);
        auto it = ctx->dctmm_plans.find(key);
        if (it == ctx->dctmm_plans.end()) {
            const cudaError_t e = dctmm_make_plan(n_in, n_keep, ctx->fast_family, stream, &plan);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "dctmm_make_plan");
            ctx->dctmm_plans[key] = plan;
        } else {
            plan = it->second;
        }
        cudaError_t e;
        {
            TransformTimer timer(ctx, stream);
            e = launch_dctmm(view, n_mat, plan, sink, ctx->status_dev, ctx->gemm.wait_limit_ns, ctx->sm_count, stream);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e, "launch_dctmm");
        ctx->kernels_launched += 1;
        return FREQKV_OK;
    }
    if (variant == FREQKV_FDCT) {
        FdctPlan plan;
        const auto key = std::make_pair(n_in, n_keep);
        auto it = ctx->fdct_plans.find(key);
        if (it == ctx->fdct_plans.end()) {
            const cudaError_t e = fdct_make_plan(n_in, n_keep, stream, &plan);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "fdct_make_plan");
            ctx->fdct_plans[key] = plan;
        } else {
            plan = it->second;
        }
        cudaError_t e;
        {
            TransformTimer timer(ctx, stream);
            e = launch_fdct(view, l.dtype, n_mat, plan, sink, stream);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e, "launch_fdct");
        ctx->kernels_launched += 1;
        return FREQKV_OK;
    }

    Basis basis;
    const bool gemm = variant == FREQKV_GEMM;
    freqkv_status st = FREQKV_OK;
    if (own_basis)
        basis = *own_basis;
    else
        st = get_basis(ctx, n_in, n_keep, first, !gemm, gemm, stream, &basis);
    if (st != FREQKV_OK) return st;

    if (gemm) {
        GemmState* gs = own_gemm ? own_gemm : &ctx->gemm;
        gs->wait_limit_ns = ctx->gemm.wait_limit_ns;
        TransformTimer timer(ctx, stream, false);
        LaunchHooks hooks;
        hooks.user = &timer;
        hooks.before = [](void* u, cudaStream_t) { static_cast<TransformTimer*>(u)->begin(); };
        hooks.after = [](void* u, cudaStream_t) { static_cast<TransformTimer*>(u)->end(); };
        const cudaError_t e =
            gemm_is_direct(n_keep)
                ? launch_gemm_direct(gs, view, basis, sink, ctx->status_dev, ctx->sm_count, hooks, stream)
                : launch_gemm(gs, view, basis, sink, ctx->status_dev, ctx->sm_count, hooks, stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, gs->last_error ? gs->last_error : "launch_gemm");
        ctx->kernels_launched += gs->kernels_last_call;
        return FREQKV_OK;
    }

    const size_t per_mat = (size_t)n_keep * l.head_dim * dtype_size(l.dtype);
    int64_t chunk = (int64_t)std::max<size_t>(1, kScratchChunkBytes / per_mat);
    chunk = std::min<int64_t>(chunk, n_mat);
    chunk = std::min<int64_t>(chunk, 1 << 30);
    void* scratch = nullptr;
    st = get_scratch(ctx, (size_t)chunk * per_mat, &scratch);
    if (st != FREQKV_OK) return st;
    for (int32_t first = 0; first < n_mat; first += (int32_t)chunk) {
        const int32_t count = (int32_t)std::min<int64_t>(chunk, n_mat - first);
        cudaError_t e;
        {
            TransformTimer timer(ctx, stream);
            e = launch_project_simt(view, l.dtype, first, count, basis, sink, scratch, stream);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e, "project_simt");
        e = launch_copy_back(view, l.dtype, first, count, n_keep, sink, scratch, stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "copy_back");
        ctx->kernels_launched += 2;
    }
    return FREQKV_OK;
}

freqkv_status check_lengths(const freqkv_layout& l, int64_t cache_len, int64_t kept_len, int64_t sink)
{
    if (sink < 0 || cache_len < 0 || kept_len < 0) return FREQKV_ERR_INVALID_ARG;
    if (sink > cache_len || cache_len > l.capacity) return FREQKV_ERR_INVALID_ARG;
    if (kept_len > cache_len - sink) return FREQKV_ERR_INVALID_ARG;
    return FREQKV_OK;
}

}  // namespace

extern "C" {

freqkv_status freqkv_layout_contiguous(freqkv_layout* out, freqkv_dtype dtype, int32_t batch, int32_t layers,
                                       int32_t kv_heads, int32_t capacity, int32_t head_dim)
{
    if (!out) return FREQKV_ERR_INVALID_ARG;
    out->dtype = dtype;
    out->batch = batch;
    out->layers = layers;
    out->kv_heads = kv_heads;
    out->capacity = capacity;
    out->head_dim = head_dim;
    out->stride_token = head_dim;
    out->stride_head = (int64_t)capacity * head_dim;
    out->stride_layer = out->stride_head * kv_heads;
    out->stride_batch = out->stride_layer * layers;
    return check_layout(out);
}

freqkv_status freqkv_create(freqkv_ctx** out, int device)
{
    if (!out) return FREQKV_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return FREQKV_ERR_CUDA;  // no CPU fallback
    }
    if (device < 0 || device >= n) return FREQKV_ERR_INVALID_ARG;
    freqkv_ctx* ctx = new (std::nothrow) freqkv_ctx();
    if (!ctx) return FREQKV_ERR_ALLOC;
    ctx->device = device;
    DeviceGuard g(device);
    cudaDeviceProp prop;
    if (!g.ok || cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
        delete ctx;
        return FREQKV_ERR_CUDA;
    }
    if (prop.major != 10) {  // kernels are built for sm_100a only
        delete ctx;
        return FREQKV_ERR_UNSUPPORTED;
    }
    ctx->sm_count = prop.multiProcessorCount;
    if (cudaMalloc(&ctx->status_dev, sizeof(int32_t)) != cudaSuccess ||
        cudaMemset(ctx->status_dev, 0, sizeof(int32_t)) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return FREQKV_ERR_ALLOC;
    }
    *out = ctx;
    return FREQKV_OK;
}

freqkv_status freqkv_destroy(freqkv_ctx* ctx)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaDeviceSynchronize();
    free_bases(ctx);
    for (auto& kv : ctx->fdct_plans) fdct_free_plan(&kv.second);
    for (auto& kv : ctx->dctmm_plans) dctmm_free_plan(&kv.second);
    gemm_release(&ctx->gemm);
    if (ctx->scratch) cudaFree(ctx->scratch);
    if (ctx->status_dev) cudaFree(ctx->status_dev);
    for (int i = 0; i < 2; ++i)
        if (ctx->stage[i]) cudaFree(ctx->stage[i]);
    if (ctx->work_done) cudaEventDestroy(ctx->work_done);
    if (ctx->rope_table) cudaFree(ctx->rope_table);
    if (ctx->attend_partial) cudaFree(ctx->attend_partial);
    if (ctx->prefill_keys) cudaFree(ctx->prefill_keys);
    if (ctx->prefill_queries) cudaFree(ctx->prefill_queries);
    for (int i = 0; i < 3; ++i)
        if (ctx->pipe[i]) cudaStreamDestroy(ctx->pipe[i]);
    if (ctx->pipe_begin) cudaEventDestroy(ctx->pipe_begin);
    if (ctx->pipe_end) cudaEventDestroy(ctx->pipe_end);
    for (auto ev : ctx->pipe_events) cudaEventDestroy(ev);
    for (auto* list : {&ctx->pending, &ctx->spare})
        for (auto& ev : *list) {
            cudaEventDestroy(ev.first);
            cudaEventDestroy(ev.second);
        }
    cudaGetLastError();
    delete ctx;
    return FREQKV_OK;
}

freqkv_status freqkv_set_variant(freqkv_ctx* ctx, freqkv_variant variant)
{
    if (!ctx || variant < FREQKV_AUTO || variant > FREQKV_SIMT) return FREQKV_ERR_INVALID_ARG;
    ctx->forced = variant;
    return FREQKV_OK;
}

freqkv_status freqkv_set_fast_family(freqkv_ctx* ctx, int32_t family)
{
    if (!ctx || (family != 0 && family != DCTMM_COOLEY_TUKEY && family != DCTMM_PRIME_FACTOR)) return FREQKV_ERR_INVALID_ARG;
    ctx->fast_family = family;
    return FREQKV_OK;
}

freqkv_status freqkv_resolve_variant(freqkv_ctx* ctx, const freqkv_layout* layout, int32_t n_in, int32_t n_keep,
                                     int32_t* out_variant)
{
    if (!ctx || !out_variant) return FREQKV_ERR_INVALID_ARG;
    const freqkv_status st = check_layout(layout);
    if (st != FREQKV_OK) return st;
    if (n_in < 1 || n_keep < 1 || n_keep > n_in) return FREQKV_ERR_INVALID_ARG;
    *out_variant = resolve(ctx, *layout, n_in, n_keep);
    return *out_variant < 0 ? FREQKV_ERR_UNSUPPORTED : FREQKV_OK;
}

freqkv_status freqkv_plan(freqkv_ctx* ctx, int32_t n_in, int32_t n_keep, freqkv_dtype dtype, freqkv_variant variant,
                          void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    if (n_in < 1 || n_keep < 1 || n_keep > n_in) return FREQKV_ERR_INVALID_ARG;
    if (dtype != FREQKV_BF16 && dtype != FREQKV_F32) return FREQKV_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (variant == FREQKV_FDCT && dtype == FREQKV_BF16 && n_keep < n_in && dctmm_supported(dtype, 128, n_in, n_keep, ctx->fast_family)) {
        const auto key = std::make_tuple(n_in, n_keep, ctx->fast_family);
        if (ctx->dctmm_plans.find(key) == ctx->dctmm_plans.end()) {
            DctmmPlan plan;
            const cudaError_t e = dctmm_make_plan(n_in, n_keep, ctx->fast_family, stream, &plan);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "dctmm_make_plan");
            ctx->dctmm_plans[key] = plan;
        }
        return FREQKV_OK;
    }
    if (variant == FREQKV_FDCT) {
        if (!is_pow2(n_in) || !is_pow2(n_keep) || !fdct_supported(dtype, 128, n_in, n_keep)) return FREQKV_ERR_UNSUPPORTED;
        const auto key = std::make_pair(n_in, n_keep);
        if (ctx->fdct_plans.find(key) == ctx->fdct_plans.end()) {
            FdctPlan plan;
            const cudaError_t e = fdct_make_plan(n_in, n_keep, stream, &plan);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "fdct_make_plan");
            ctx->fdct_plans[key] = plan;
        }
        return FREQKV_OK;
    }
    if (variant == FREQKV_GEMM && dtype != FREQKV_BF16) return FREQKV_ERR_UNSUPPORTED;
    Basis b;
    const bool gemm = variant == FREQKV_GEMM;
    const bool both = variant == FREQKV_AUTO;
    return get_basis(ctx, n_in, n_keep, 0, !gemm || both, (gemm || both) && dtype == FREQKV_BF16, stream, &b);
}

freqkv_status freqkv_check_compress(const freqkv_layout* layout, const void* k, const void* v, int32_t cache_len,
                                    int32_t kept_len, int32_t sink)
{
    freqkv_status st = check_layout(layout);
    if (st != FREQKV_OK) return st;
    st = check_tensors(*layout, k, v);
    if (st != FREQKV_OK) return st;
    return check_lengths(*layout, cache_len, kept_len, sink);
}

freqkv_status freqkv_check_append(const freqkv_layout* layout, const void* k, const void* v, const void* new_k,
                                  const void* new_v, int32_t n_new, const int32_t* lens)
{
    if (!lens) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = check_layout(layout);
    if (st != FREQKV_OK) return st;
    st = check_tensors(*layout, k, v);
    if (st != FREQKV_OK) return st;
    if (n_new < 0) return FREQKV_ERR_INVALID_ARG;
    if (n_new > 0 && (!new_k || !new_v)) return FREQKV_ERR_INVALID_ARG;
    if (n_new > 0 && (((uintptr_t)new_k | (uintptr_t)new_v) & 15)) return FREQKV_ERR_UNSUPPORTED;
    for (int32_t b = 0; b < layout->batch; ++b) {
        if (lens[b] < 0 || lens[b] > layout->capacity) return FREQKV_ERR_INVALID_ARG;
        if ((int64_t)lens[b] + n_new > layout->capacity) return FREQKV_ERR_CAPACITY;
    }
    return FREQKV_OK;
}

freqkv_status freqkv_compress(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, int32_t cache_len,
                              int32_t kept_len, int32_t sink, void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = freqkv_check_compress(layout, k, v, cache_len, kept_len, sink);
    if (st != FREQKV_OK) return st;
    const int32_t n_in = cache_len - sink;
    if (n_in == 0 || kept_len == 0 || kept_len == n_in) return FREQKV_OK;  // nothing to rewrite
    const int32_t variant = resolve(ctx, *layout, n_in, kept_len);
    if (variant < 0) return FREQKV_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    WorkOrder order(ctx, static_cast<cudaStream_t>(cuda_stream));
    return compress_group(ctx, *layout, k, v, 0, layout->batch, n_in, kept_len, sink, variant,
                          static_cast<cudaStream_t>(cuda_stream));
}

freqkv_status freqkv_compress_band(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, int32_t cache_len,
                                   int32_t kept_len, int32_t sink, int32_t first_component, void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = freqkv_check_compress(layout, k, v, cache_len, kept_len, sink);
    if (st != FREQKV_OK) return st;
    const int32_t n_in = cache_len - sink;
    if (first_component < 0 || (int64_t)first_component + kept_len > n_in) return FREQKV_ERR_INVALID_ARG;
    if (n_in == 0 || kept_len == 0 || kept_len == n_in) return FREQKV_OK;  // nothing to rewrite (a full band is the identity)
    int32_t variant = resolve(ctx, *layout, n_in, kept_len);
    if (variant == FREQKV_FDCT && first_component != 0) {  // the fast transform keeps the lowest components only
        if (ctx->forced == FREQKV_FDCT) return FREQKV_ERR_UNSUPPORTED;
        variant = FREQKV_SIMT;
    }
    if (variant < 0) return FREQKV_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    WorkOrder order(ctx, static_cast<cudaStream_t>(cuda_stream));
    return compress_group(ctx, *layout, k, v, 0, layout->batch, n_in, kept_len, sink, variant,
                          static_cast<cudaStream_t>(cuda_stream), first_component);
}

freqkv_status freqkv_power_spectrum(freqkv_ctx* ctx, const freqkv_layout* layout, const void* k, const void* v,
                                    int32_t cache_len, int32_t sink, float* spectrum_k, float* spectrum_v, void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = freqkv_check_compress(layout, k, v, cache_len, 0, sink);
    if (st != FREQKV_OK) return st;
    if (!spectrum_k && !spectrum_v) return FREQKV_ERR_INVALID_ARG;
    const freqkv_layout& l = *layout;
    const int32_t n_in = cache_len - sink;
    if (n_in < 1) return FREQKV_ERR_INVALID_ARG;
    if (!gemm_supported(l.dtype, l.head_dim, n_in, n_in)) return FREQKV_ERR_UNSUPPORTED;  // bf16, head_dim 128
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    WorkOrder order(ctx, stream);
    Basis basis;
    st = get_basis(ctx, n_in, n_in, kDctRows, false, true, stream, &basis);
    if (st != FREQKV_OK) return st;
    const size_t bytes = (size_t)l.layers * l.kv_heads * n_in * sizeof(float);
    if (spectrum_k) FREQKV_CUDA(ctx, cudaMemsetAsync(spectrum_k, 0, bytes, stream));
    if (spectrum_v) FREQKV_CUDA(ctx, cudaMemsetAsync(spectrum_v, 0, bytes, stream));
    SpectrumOut out;
    out.k = spectrum_k;
    out.v = spectrum_v;
    out.scale = 1.0f / ((float)l.batch * (float)l.head_dim);
    const CacheView view = make_view(l, const_cast<void*>(k), const_cast<void*>(v), 0, l.batch);
    TransformTimer timer(ctx, stream, false);
    LaunchHooks hooks;
    hooks.user = &timer;
    hooks.before = [](void* u, cudaStream_t) { static_cast<TransformTimer*>(u)->begin(); };
    hooks.after = [](void* u, cudaStream_t) { static_cast<TransformTimer*>(u)->end(); };
    const cudaError_t e = launch_gemm(&ctx->gemm, view, basis, sink, ctx->status_dev, ctx->sm_count, hooks, stream, &out);
    if (e != cudaSuccess) return cuda_fail(ctx, e, ctx->gemm.last_error ? ctx->gemm.last_error : "launch_gemm");
    ctx->kernels_launched += ctx->gemm.kernels_last_call;
    return FREQKV_OK;
}

freqkv_status freqkv_compress_ragged(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, int32_t* lens,
                                     const int32_t* kept_len, int32_t sink, void* cuda_stream)
{
    if (!ctx || !lens || !kept_len) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = check_layout(layout);
    if (st != FREQKV_OK) return st;
    st = check_tensors(*layout, k, v);
    if (st != FREQKV_OK) return st;
    std::vector<int32_t> variant(layout->batch, 0);
    for (int32_t b = 0; b < layout->batch; ++b) {
        st = check_lengths(*layout, lens[b], kept_len[b], sink);
        if (st != FREQKV_OK) return st;
        const int32_t n_in = lens[b] - sink;
        if (n_in == 0 || kept_len[b] == 0 || kept_len[b] == n_in) continue;
        variant[b] = resolve(ctx, *layout, n_in, kept_len[b]);
        if (variant[b] < 0) return FREQKV_ERR_UNSUPPORTED;
    }
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    WorkOrder order(ctx, stream);
    // When every sequence that needs work takes the folded tensor-core form, the whole batch runs
    // as one fold launch and one tensor-core launch; every plan is built and all memory is
    // allocated before the first of them.
    {
        bool all_folded = true;
        int32_t active = 0;
        for (int32_t b = 0; b < layout->batch; ++b) {
            if (variant[b] == 0) continue;
            ++active;
            if (variant[b] != FREQKV_GEMM || gemm_is_direct(kept_len[b])) all_folded = false;
        }
        if (all_folded && active > 1) {
            std::vector<RaggedItem> items;
            bool ok = true;
            for (int pass = 0; pass < 2 && ok; ++pass) {  // second pass: a flush of the plan cache may have dropped earlier plans
                items.clear();
                for (int32_t b = 0; b < layout->batch && ok; ++b) {
                    if (variant[b] == 0) continue;
                    Basis basis;
                    st = get_basis(ctx, lens[b] - sink, kept_len[b], 0, false, true, stream, &basis);
                    if (st != FREQKV_OK) return st;  // nothing enqueued but plan builders
                    items.push_back({b, basis});
                }
                bool intact = true;
                for (const RaggedItem& it : items) {
                    auto found = ctx->bases.find(std::make_tuple(it.basis.n_in, it.basis.n_keep, (int32_t)0));
                    if (found == ctx->bases.end() || found->second.fold != it.basis.fold) intact = false;
                }
                if (intact) break;
                if (pass == 1) ok = false;
            }
            if (ok) {
                const CacheView view = make_view(*layout, k, v, 0, layout->batch);
                TransformTimer timer(ctx, stream, false);
                LaunchHooks hooks;
                hooks.user = &timer;
                hooks.before = [](void* u, cudaStream_t) { static_cast<TransformTimer*>(u)->begin(); };
                hooks.after = [](void* u, cudaStream_t) { static_cast<TransformTimer*>(u)->end(); };
                ctx->gemm.last_error = nullptr;
                const cudaError_t e = launch_gemm_ragged(&ctx->gemm, view, items, sink, ctx->status_dev, ctx->sm_count, hooks, stream);
                if (e == cudaSuccess) {
                    ctx->kernels_launched += ctx->gemm.kernels_last_call;
                    for (int32_t b = 0; b < layout->batch; ++b) lens[b] = sink + kept_len[b];
                    return FREQKV_OK;
                }
                if (e != cudaErrorMemoryAllocation || ctx->gemm.kernels_last_call != 0)
                    return cuda_fail(ctx, e, ctx->gemm.last_error ? ctx->gemm.last_error : "launch_gemm_ragged");
                cudaGetLastError();  // the folded batch does not fit: go sequence by sequence
            }
        }
    }
    // Sequences are grouped by runs of equal (length, kept length); each run is one group.
    for (int32_t b = 0; b < layout->batch;) {
        int32_t e = b + 1;
        while (e < layout->batch && lens[e] == lens[b] && kept_len[e] == kept_len[b]) ++e;
        if (variant[b] > 0) {
            st = compress_group(ctx, *layout, k, v, b, e - b, lens[b] - sink, kept_len[b], sink, variant[b], stream);
            if (st != FREQKV_OK) return st;
        }
        b = e;
    }
    for (int32_t b = 0; b < layout->batch; ++b) lens[b] = sink + kept_len[b];
    return FREQKV_OK;
}

freqkv_status freqkv_append(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, const void* new_k,
                            const void* new_v, int32_t n_new, int32_t* lens, void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    const freqkv_status st = freqkv_check_append(layout, k, v, new_k, new_v, n_new, lens);
    if (st != FREQKV_OK) return st;
    if (n_new == 0) return FREQKV_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    const CacheView view = make_view(*layout, k, v, 0, layout->batch);
    const cudaError_t e =
        launch_append(view, layout->dtype, layout->batch, lens, n_new, new_k, new_v, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "append");
    ctx->kernels_launched += (layout->batch + 127) / 128;
    for (int32_t b = 0; b < layout->batch; ++b) lens[b] += n_new;
    return FREQKV_OK;
}

freqkv_status freqkv_compress_host(freqkv_ctx* ctx, const freqkv_layout* layout, void* k_host, void* v_host,
                                   int32_t cache_len, int32_t kept_len, int32_t sink, void* cuda_stream,
                                   int64_t* h2d_bytes, int64_t* d2h_bytes)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = freqkv_check_compress(layout, k_host, v_host, cache_len, kept_len, sink);
    if (st != FREQKV_OK) return st;
    if (h2d_bytes) *h2d_bytes = 0;
    if (d2h_bytes) *d2h_bytes = 0;
    const int32_t n_in = cache_len - sink;
    if (n_in == 0 || kept_len == 0 || kept_len == n_in) return FREQKV_OK;
    const freqkv_layout& l = *layout;
    const int32_t variant = resolve(ctx, l, n_in, kept_len);
    if (variant < 0) return FREQKV_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    WorkOrder order(ctx, stream);  // its end is recorded after the caller's stream has joined the pipeline's tail
    const size_t elt = dtype_size(l.dtype);
    const size_t bytes = (size_t)span_elements(l) * elt;
    // head stride below one matrix's rows (heads interleaved inside the token axis) is not
    // something a 2-D copy can express
    const size_t row_bytes = (size_t)l.stride_token * elt;
    if (l.kv_heads > 1 && (size_t)l.stride_head * elt < (size_t)(n_in - 1) * row_bytes + (size_t)l.head_dim * elt)
        return FREQKV_ERR_UNSUPPORTED;
    if (bytes > ctx->stage_bytes) {
        FREQKV_CUDA(ctx, cudaDeviceSynchronize());
        for (int i = 0; i < 2; ++i) {
            if (ctx->stage[i]) cudaFree(ctx->stage[i]);
            ctx->stage[i] = nullptr;
        }
        ctx->stage_bytes = 0;
        FREQKV_CUDA(ctx, cudaMalloc(&ctx->stage[0], bytes));
        FREQKV_CUDA(ctx, cudaMalloc(&ctx->stage[1], bytes));
        ctx->stage_bytes = bytes;
    }
    // Three-deep pipeline over groups of layers: the host->device copy of group g+1, the
    // compression of group g and the device->host copy of group g-1 run at the same time on three
    // streams of the context (PCIe carries both directions at once), ordered by events; the
    // caller's stream is the entry and the exit of the whole pipeline.
    if (!ctx->pipe[0]) {
        for (int i = 0; i < 3; ++i) FREQKV_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->pipe[i], cudaStreamNonBlocking));
        FREQKV_CUDA(ctx, cudaEventCreateWithFlags(&ctx->pipe_begin, cudaEventDisableTiming));
        FREQKV_CUDA(ctx, cudaEventCreateWithFlags(&ctx->pipe_end, cudaEventDisableTiming));
    }
    const int32_t per_group = std::max(1, (l.layers + 7) / 8);  // layers per group: about 8 groups per sequence
    const int32_t groups_per_seq = (l.layers + per_group - 1) / per_group;
    const size_t n_groups = (size_t)l.batch * groups_per_seq;
    while (ctx->pipe_events.size() < 2 * n_groups) {
        cudaEvent_t ev;
        FREQKV_CUDA(ctx, cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
        ctx->pipe_events.push_back(ev);
    }
    // One 2-D copy per (tensor, layer): `kv_heads` runs of rows, one run per head.  Rows of a
    // matrix are contiguous when stride_token == head_dim; padded rows are copied with their
    // padding (same layout on both sides).
    auto copy_rows = [&](bool to_device, int32_t b, int32_t y0, int32_t ny, int32_t row0, int32_t rows, cudaStream_t s,
                         int64_t* counter) -> cudaError_t {
        const size_t width = rows == 0 ? 0 : (size_t)(rows - 1) * row_bytes + (size_t)l.head_dim * elt;
        const size_t pitch = l.kv_heads == 1 ? width : (size_t)l.stride_head * elt;
        for (int t = 0; t < 2; ++t) {
            char* host = static_cast<char*>(t ? v_host : k_host);
            char* dev = static_cast<char*>(ctx->stage[t]);
            for (int32_t y = y0; y < y0 + ny; ++y) {
                const size_t off = ((size_t)b * l.stride_batch + (size_t)y * l.stride_layer + (size_t)row0 * l.stride_token) * elt;
                const cudaError_t e = cudaMemcpy2DAsync(to_device ? dev + off : host + off, pitch,
                                                        to_device ? host + off : dev + off, pitch, width, l.kv_heads,
                                                        to_device ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost, s);
                if (e != cudaSuccess) return e;
                if (counter) *counter += (int64_t)width * l.kv_heads;
            }
        }
        return cudaSuccess;
    };
    FREQKV_CUDA(ctx, cudaEventRecord(ctx->pipe_begin, stream));
    for (int i = 0; i < 3; ++i) FREQKV_CUDA(ctx, cudaStreamWaitEvent(ctx->pipe[i], ctx->pipe_begin, 0));
    // From here on work may be in flight on the three streams: whatever happens, the caller's
    // stream joins all of them before this call returns (on an error the host rows are undefined).
    auto pipeline = [&]() -> freqkv_status {
        size_t group = 0;
        for (int32_t b = 0; b < l.batch; ++b)
            for (int32_t y0 = 0; y0 < l.layers; y0 += per_group, ++group) {
                const int32_t ny = std::min(per_group, l.layers - y0);
                cudaEvent_t copied = ctx->pipe_events[2 * group], compressed = ctx->pipe_events[2 * group + 1];
                cudaError_t e = copy_rows(true, b, y0, ny, sink, n_in, ctx->pipe[0], h2d_bytes);
                if (e != cudaSuccess) return cuda_fail(ctx, e, "host->device copy");
                FREQKV_CUDA(ctx, cudaEventRecord(copied, ctx->pipe[0]));
                FREQKV_CUDA(ctx, cudaStreamWaitEvent(ctx->pipe[1], copied, 0));
                freqkv_layout sub = l;  // this group's layers of sequence b as a cache of its own
                sub.batch = 1;
                sub.layers = ny;
                const size_t off = ((size_t)b * l.stride_batch + (size_t)y0 * l.stride_layer) * elt;
                const freqkv_status gs = compress_group(ctx, sub, static_cast<char*>(ctx->stage[0]) + off,
                                                        static_cast<char*>(ctx->stage[1]) + off, 0, 1, n_in, kept_len, sink,
                                                        variant, ctx->pipe[1]);
                if (gs != FREQKV_OK) return gs;
                FREQKV_CUDA(ctx, cudaEventRecord(compressed, ctx->pipe[1]));
                FREQKV_CUDA(ctx, cudaStreamWaitEvent(ctx->pipe[2], compressed, 0));
                e = copy_rows(false, b, y0, ny, sink, kept_len, ctx->pipe[2], d2h_bytes);
                if (e != cudaSuccess) return cuda_fail(ctx, e, "device->host copy");
            }
        return FREQKV_OK;
    };
    const freqkv_status run = pipeline();
    // every copy back is on pipe[2], after the work it depends on; after an error the other two
    // streams may hold work that nothing on pipe[2] waits for, so all three are joined
    for (int i = run == FREQKV_OK ? 2 : 0; i < 3; ++i) {
        FREQKV_CUDA(ctx, cudaEventRecord(ctx->pipe_end, ctx->pipe[i]));
        FREQKV_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->pipe_end, 0));
    }
    return run;
}

// The context's cos/sin table for `rope_base`, built on `stream` when the base or the capacity has
// changed; *table stays null when RoPE is off.
static freqkv_status rope_table_for(freqkv_ctx* ctx, int32_t capacity, float rope_base, cudaStream_t stream, const float2** table)
{
    *table = nullptr;
    if (!(rope_base > 0.f)) return FREQKV_OK;
    if (!ctx->rope_table || ctx->rope_rows < capacity || ctx->rope_base != (double)rope_base) {
        if (ctx->rope_table) {
            FREQKV_CUDA(ctx, cudaDeviceSynchronize());  // an enqueued launch may still read the old table
            cudaFree(ctx->rope_table);
            ctx->rope_table = nullptr;
        }
        const int32_t rows = std::max(capacity, 2);
        FREQKV_CUDA(ctx, cudaMalloc(&ctx->rope_table, (size_t)rows * 64 * sizeof(float2)));
        const cudaError_t e = launch_rope_table(ctx->rope_table, rows, (double)rope_base, stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "rope_table");
        ctx->rope_rows = rows;
        ctx->rope_base = (double)rope_base;
        ctx->kernels_launched += 1;
    }
    *table = ctx->rope_table;
    return FREQKV_OK;
}

freqkv_status freqkv_check_attend(const freqkv_layout* layout, const void* k, const void* v, int32_t layer, const void* q,
                                  const void* out, int32_t q_heads_per_kv, const int32_t* lens)
{
    if (!lens) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = check_layout(layout);
    if (st != FREQKV_OK) return st;
    st = check_tensors(*layout, k, v);
    if (st != FREQKV_OK) return st;
    if (!q || !out || q == out) return FREQKV_ERR_INVALID_ARG;
    if (((uintptr_t)q | (uintptr_t)out) & 15) return FREQKV_ERR_UNSUPPORTED;
    if (layer < 0 || layer >= layout->layers || q_heads_per_kv < 1) return FREQKV_ERR_INVALID_ARG;
    if (!attend_supported(layout->head_dim, q_heads_per_kv)) return FREQKV_ERR_UNSUPPORTED;
    for (int32_t b = 0; b < layout->batch; ++b)
        if (lens[b] < 1 || lens[b] > layout->capacity) return FREQKV_ERR_INVALID_ARG;
    return FREQKV_OK;
}

freqkv_status freqkv_attend_decode(freqkv_ctx* ctx, const freqkv_layout* layout, const void* k, const void* v, int32_t layer,
                                   const void* q, void* out, int32_t q_heads_per_kv, const int32_t* lens, float rope_base,
                                   float scale, void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    const freqkv_status st = freqkv_check_attend(layout, k, v, layer, q, out, q_heads_per_kv, lens);
    if (st != FREQKV_OK) return st;
    if (!(scale == scale) || !(rope_base == rope_base)) return FREQKV_ERR_INVALID_ARG;  // NaN
    const freqkv_layout& l = *layout;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    WorkOrder order(ctx, stream);
    if (scale <= 0.f) scale = 1.0f / sqrtf((float)l.head_dim);
    int32_t max_len = 0;
    for (int32_t b = 0; b < l.batch; ++b) max_len = std::max(max_len, lens[b]);
    const float2* table = nullptr;
    const freqkv_status ts = rope_table_for(ctx, l.capacity, rope_base, stream, &table);
    if (ts != FREQKV_OK) return ts;
    const int32_t splits = attend_splits(l.batch, l.kv_heads, max_len, q_heads_per_kv, l.dtype, ctx->sm_count);
    const size_t need = attend_partial_bytes(splits, l.batch, l.kv_heads * q_heads_per_kv);
    if (need > ctx->attend_partial_bytes) {
        if (ctx->attend_partial) {
            FREQKV_CUDA(ctx, cudaDeviceSynchronize());
            cudaFree(ctx->attend_partial);
            ctx->attend_partial = nullptr;
            ctx->attend_partial_bytes = 0;
        }
        FREQKV_CUDA(ctx, cudaMalloc(&ctx->attend_partial, need));
        ctx->attend_partial_bytes = need;
    }
    cudaError_t e;
    {
        TransformTimer timer(ctx, stream);
        e = launch_attend(l, k, v, layer, q, out, q_heads_per_kv, lens, table, scale, splits, ctx->attend_partial, stream);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "attend");
    ctx->kernels_launched += 1 + (l.batch + ATTEND_MAX_BATCH - 1) / ATTEND_MAX_BATCH;
    return FREQKV_OK;
}

freqkv_status freqkv_check_attend_prefill(const freqkv_layout* layout, const void* k, const void* v, int32_t layer,
                                          const void* q, const void* out, int32_t q_heads_per_kv, int32_t n_new,
                                          const int32_t* lens)
{
    if (!lens) return FREQKV_ERR_INVALID_ARG;
    freqkv_status st = check_layout(layout);
    if (st != FREQKV_OK) return st;
    st = check_tensors(*layout, k, v);
    if (st != FREQKV_OK) return st;
    if (!q || !out || q == out) return FREQKV_ERR_INVALID_ARG;
    if (((uintptr_t)q | (uintptr_t)out) & 15) return FREQKV_ERR_UNSUPPORTED;
    if (layer < 0 || layer >= layout->layers || q_heads_per_kv < 1 || n_new < 1) return FREQKV_ERR_INVALID_ARG;
    if (!prefill_supported(layout->dtype, layout->head_dim, q_heads_per_kv)) return FREQKV_ERR_UNSUPPORTED;
    for (int32_t b = 0; b < layout->batch; ++b)
        if (lens[b] < n_new || lens[b] > layout->capacity) return FREQKV_ERR_INVALID_ARG;
    return FREQKV_OK;
}

freqkv_status freqkv_attend_prefill(freqkv_ctx* ctx, const freqkv_layout* layout, const void* k, const void* v, int32_t layer,
                                    const void* q, void* out, int32_t q_heads_per_kv, int32_t n_new, const int32_t* lens,
                                    float rope_base, float scale, void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    const freqkv_status st = freqkv_check_attend_prefill(layout, k, v, layer, q, out, q_heads_per_kv, n_new, lens);
    if (st != FREQKV_OK) return st;
    if (!(scale == scale) || !(rope_base == rope_base)) return FREQKV_ERR_INVALID_ARG;  // NaN
    const freqkv_layout& l = *layout;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    WorkOrder order(ctx, stream);
    if (scale <= 0.f) scale = 1.0f / sqrtf((float)l.head_dim);
    const float2* table = nullptr;
    const freqkv_status ts = rope_table_for(ctx, l.capacity, rope_base, stream, &table);
    if (ts != FREQKV_OK) return ts;
    struct Grow { void** p; size_t* have; size_t need; };
    const Grow scratch[2] = {{&ctx->prefill_keys, &ctx->prefill_keys_bytes, prefill_key_scratch_bytes(l)},
                             {&ctx->prefill_queries, &ctx->prefill_queries_bytes, prefill_query_scratch_bytes(l, q_heads_per_kv, n_new)}};
    for (const Grow& s : scratch) {
        if (s.need <= *s.have) continue;
        if (*s.p) {
            FREQKV_CUDA(ctx, cudaDeviceSynchronize());  // an enqueued launch may still use the old buffer
            cudaFree(*s.p);
            *s.p = nullptr;
            *s.have = 0;
        }
        if (cudaMalloc(s.p, s.need) != cudaSuccess) {
            cudaGetLastError();
            *s.p = nullptr;
            ctx->last_error = "out of device memory for the prefill attention scratch";
            return FREQKV_ERR_ALLOC;
        }
        *s.have = s.need;
    }
    const char* why = nullptr;
    int32_t launched = 0;
    cudaError_t e;
    {
        TransformTimer timer(ctx, stream);
        e = launch_prefill(l, k, v, layer, q, out, q_heads_per_kv, n_new, lens, table, scale, ctx->prefill_keys,
                           ctx->prefill_queries, ctx->status_dev, ctx->gemm.wait_limit_ns, &why, &launched, stream);
    }
    ctx->kernels_launched += launched;
    if (e != cudaSuccess) {
        if (why) {
            cudaGetLastError();
            ctx->last_error = why;
            return e == cudaErrorNotSupported ? FREQKV_ERR_UNSUPPORTED : FREQKV_ERR_CUDA;
        }
        return cuda_fail(ctx, e, "attend_prefill");
    }
    return FREQKV_OK;
}

// The graph's kernels have the addresses of the fold scratch and of the basis baked in, so the
// graph owns both: no later call on the context can free or move them under a replay.
struct freqkv_decode_graph {
    freqkv_ctx* ctx = nullptr;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    GemmState gemm;
    Basis basis;
};

freqkv_status freqkv_decode_graph_create(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, const void* new_k,
                                         const void* new_v, int32_t* lens_device, int32_t kept_len, int32_t sink,
                                         freqkv_decode_graph** out)
{
    if (!ctx || !out || !lens_device) return FREQKV_ERR_INVALID_ARG;
    *out = nullptr;
    freqkv_status st = check_layout(layout);
    if (st != FREQKV_OK) return st;
    const freqkv_layout& l = *layout;
    st = check_tensors(l, k, v);
    if (st != FREQKV_OK) return st;
    if (!new_k || !new_v) return FREQKV_ERR_INVALID_ARG;
    if (((uintptr_t)new_k | (uintptr_t)new_v | (uintptr_t)lens_device) & 15) return FREQKV_ERR_UNSUPPORTED;
    st = check_lengths(l, l.capacity, kept_len, sink);
    if (st != FREQKV_OK) return st;
    const int32_t n_in = l.capacity - sink;
    if (kept_len < 1 || kept_len >= n_in) return FREQKV_ERR_INVALID_ARG;  // a compression must make room
    if (!gemm_applicable(l, n_in, kept_len)) return FREQKV_ERR_UNSUPPORTED;  // the graph holds the tensor-core variant
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;

    // everything that allocates or builds tables happens here, outside the graph
    cudaStream_t cs = nullptr;
    FREQKV_CUDA(ctx, cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking));
    freqkv_decode_graph* dg = new (std::nothrow) freqkv_decode_graph();
    Basis basis;
    // a plan of this shape already in the cache may be in use by enqueued kernels and stays there;
    // the graph gets one of its own, built into the cache and then taken out of it
    Basis cached;
    const auto key = std::make_tuple(n_in, kept_len, (int32_t)0);
    const bool had = ctx->bases.count(key) != 0;
    if (had) {
        cached = ctx->bases[key];
        disown_basis(ctx, n_in, kept_len, 0);
    }
    st = dg ? get_basis(ctx, n_in, kept_len, 0, false, true, cs, &basis) : FREQKV_ERR_ALLOC;
    if (st == FREQKV_OK) {
        disown_basis(ctx, n_in, kept_len, 0);
        dg->basis = basis;
    }
    if (had) {  // put the context's own plan back
        ctx->bases[key] = cached;
        ctx->basis_bytes += basis_device_bytes(cached);
    }
    cudaError_t e = st == FREQKV_OK ? cudaStreamSynchronize(cs) : cudaSuccess;
    if (st == FREQKV_OK && e == cudaSuccess)
        e = gemm_prepare(&dg->gemm, gemm_is_direct(kept_len) ? 0 : l.batch * l.layers * l.kv_heads, basis, ctx->sm_count);
    auto fail = [&](freqkv_status code, cudaError_t ce, const char* where) {
        if (ce != cudaSuccess) code = cuda_fail(ctx, ce, where);
        if (dg) {
            if (dg->exec) cudaGraphExecDestroy(dg->exec);
            if (dg->graph) cudaGraphDestroy(dg->graph);
            gemm_release(&dg->gemm);
            free_basis(&dg->basis);
            delete dg;
        }
        cudaStreamDestroy(cs);
        cudaGetLastError();
        return code;
    };
    if (st != FREQKV_OK) return fail(st, cudaSuccess, "");
    if (e != cudaSuccess) return fail(FREQKV_ERR_CUDA, e, "decode graph set-up");
    if (!dg) return fail(FREQKV_ERR_ALLOC, cudaSuccess, "");
    dg->ctx = ctx;

    // graph: trigger -> IF (all sequences full) { fold, GEMM, lengths := sink + kept_len } -> append + advance
    if ((e = cudaGraphCreate(&dg->graph, 0)) != cudaSuccess) return fail(FREQKV_ERR_CUDA, e, "cudaGraphCreate");
    cudaGraphConditionalHandle handle;
    if ((e = cudaGraphConditionalHandleCreate(&handle, dg->graph, 0, cudaGraphCondAssignDefault)) != cudaSuccess)
        return fail(FREQKV_ERR_CUDA, e, "cudaGraphConditionalHandleCreate");
    cudaGraphNode_t trigger = nullptr, branch = nullptr;
    if ((e = add_decode_trigger_node(dg->graph, &trigger, lens_device, l.batch, l.capacity, handle, ctx->status_dev)) != cudaSuccess)
        return fail(FREQKV_ERR_CUDA, e, "trigger node");
    cudaGraphNodeParams cond = {};
    cond.type = cudaGraphNodeTypeConditional;
    cond.conditional.handle = handle;
    cond.conditional.type = cudaGraphCondTypeIf;
    cond.conditional.size = 1;
    if ((e = cudaGraphAddNode(&branch, dg->graph, &trigger, 1, &cond)) != cudaSuccess)
        return fail(FREQKV_ERR_CUDA, e, "conditional node");
    cudaGraph_t body = cond.conditional.phGraph_out[0];
    const bool was_timing = ctx->timing;
    ctx->timing = false;  // event records do not belong in the graph
    if ((e = cudaStreamBeginCaptureToGraph(cs, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed)) != cudaSuccess) {
        ctx->timing = was_timing;
        return fail(FREQKV_ERR_CUDA, e, "capture of the compression");
    }
    st = compress_group(ctx, l, k, v, 0, l.batch, n_in, kept_len, sink, FREQKV_GEMM, cs, 0, &dg->gemm, &dg->basis);
    e = st == FREQKV_OK ? launch_decode_set_lens(lens_device, l.batch, sink + kept_len, cs) : cudaSuccess;
    cudaGraph_t captured = nullptr;
    const cudaError_t e_end = cudaStreamEndCapture(cs, &captured);
    ctx->timing = was_timing;
    if (st != FREQKV_OK) return fail(st, cudaSuccess, "");
    if (e != cudaSuccess || e_end != cudaSuccess) return fail(FREQKV_ERR_CUDA, e != cudaSuccess ? e : e_end, "capture of the compression");
    // the append, after the branch
    if ((e = cudaStreamBeginCaptureToGraph(cs, dg->graph, &branch, nullptr, 1, cudaStreamCaptureModeRelaxed)) != cudaSuccess)
        return fail(FREQKV_ERR_CUDA, e, "capture of the append");
    e = launch_decode_append(make_view(l, k, v, 0, l.batch), l.dtype, l.batch, lens_device, l.capacity, new_k, new_v, cs);
    const cudaError_t e_end2 = cudaStreamEndCapture(cs, &captured);
    if (e != cudaSuccess || e_end2 != cudaSuccess) return fail(FREQKV_ERR_CUDA, e != cudaSuccess ? e : e_end2, "capture of the append");
    if ((e = cudaGraphInstantiate(&dg->exec, dg->graph, 0)) != cudaSuccess) return fail(FREQKV_ERR_CUDA, e, "cudaGraphInstantiate");
    cudaStreamDestroy(cs);
    *out = dg;
    return FREQKV_OK;
}

freqkv_status freqkv_decode_graph_launch(freqkv_decode_graph* graph, void* cuda_stream)
{
    if (!graph || !graph->exec) return FREQKV_ERR_INVALID_ARG;
    DeviceGuard g(graph->ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    WorkOrder order(graph->ctx, static_cast<cudaStream_t>(cuda_stream));  // the graph's kernels use the context's status word
    FREQKV_CUDA(graph->ctx, cudaGraphLaunch(graph->exec, static_cast<cudaStream_t>(cuda_stream)));
    graph->ctx->kernels_launched += 3;  // trigger, append, advance (the compression adds 3 when it runs)
    return FREQKV_OK;
}

freqkv_status freqkv_decode_graph_destroy(freqkv_decode_graph* graph)
{
    if (!graph) return FREQKV_ERR_INVALID_ARG;
    DeviceGuard g(graph->ctx->device);
    cudaDeviceSynchronize();
    if (graph->exec) cudaGraphExecDestroy(graph->exec);
    if (graph->graph) cudaGraphDestroy(graph->graph);
    gemm_release(&graph->gemm);
    free_basis(&graph->basis);
    cudaGetLastError();
    delete graph;
    return FREQKV_OK;
}

freqkv_status freqkv_set_timing(freqkv_ctx* ctx, int32_t enabled)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    ctx->timing = enabled != 0;
    return FREQKV_OK;
}

freqkv_status freqkv_get_timing(freqkv_ctx* ctx, int64_t* transform_launches, double* transform_ms,
                                int64_t* kernels_launched)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    double ms = 0.0;
    int64_t n = 0;
    for (auto& ev : ctx->pending) {
        FREQKV_CUDA(ctx, cudaEventSynchronize(ev.second));
        float t = 0.f;
        FREQKV_CUDA(ctx, cudaEventElapsedTime(&t, ev.first, ev.second));
        ms += t;
        ++n;
        ctx->spare.push_back(ev);
    }
    ctx->pending.clear();
    if (transform_launches) *transform_launches = n;
    if (transform_ms) *transform_ms = ms;
    if (kernels_launched) *kernels_launched = ctx->kernels_launched;
    return FREQKV_OK;
}

freqkv_status freqkv_last_device_status(freqkv_ctx* ctx, void* cuda_stream)
{
    if (!ctx) return FREQKV_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t word = 0;
    FREQKV_CUDA(ctx, cudaMemcpyAsync(&word, ctx->status_dev, sizeof(word), cudaMemcpyDeviceToHost, stream));
    FREQKV_CUDA(ctx, cudaMemsetAsync(ctx->status_dev, 0, sizeof(word), stream));
    FREQKV_CUDA(ctx, cudaStreamSynchronize(stream));
    if (word != 0) {
        char buf[128];
        if (word == DECODE_ERR_MIXED_LENGTHS) {
            snprintf(buf, sizeof(buf), "decode graph: some but not all sequences were full; the full ones were not appended to");
            ctx->last_error = buf;
            return FREQKV_ERR_CAPACITY;
        }
        snprintf(buf, sizeof(buf), "device status word 0x%08x (a bounded wait gave up)", (unsigned)word);
        ctx->last_error = buf;
        return FREQKV_ERR_TIMEOUT;
    }
    return FREQKV_OK;
}

freqkv_status freqkv_set_wait_limit(freqkv_ctx* ctx, int64_t nanoseconds)
{
    if (!ctx || nanoseconds < 1000) return FREQKV_ERR_INVALID_ARG;
    ctx->gemm.wait_limit_ns = (unsigned long long)nanoseconds;
    return FREQKV_OK;
}

freqkv_status freqkv_selftest_bounded_wait(freqkv_ctx* ctx, int64_t nanoseconds, void* cuda_stream)
{
    if (!ctx || nanoseconds < 1000 || nanoseconds > 1000000000ll) return FREQKV_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return FREQKV_ERR_CUDA;
    const cudaError_t e = launch_wait_probe(ctx->status_dev, (unsigned long long)nanoseconds, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "bounded wait probe");
    ctx->kernels_launched += 1;
    return FREQKV_OK;
}

freqkv_status freqkv_fast_plan_apply_host(int32_t n_in, int32_t n_keep, int32_t family, const double* x, int32_t channels,
                                          double* y, int32_t* factors)
{
    if (!x || !y || channels < 1 || n_in < 1 || n_keep < 1 || n_keep >= n_in) return FREQKV_ERR_INVALID_ARG;
    if (family != 0 && family != DCTMM_COOLEY_TUKEY && family != DCTMM_PRIME_FACTOR) return FREQKV_ERR_INVALID_ARG;
    DctmmHostPlan hp;
    if (!dctmm_host_plan(n_in, n_keep, family, &hp)) return FREQKV_ERR_UNSUPPORTED;
    if (factors) {
        factors[0] = hp.plan.n1;
        factors[1] = hp.plan.n2;
        factors[2] = hp.plan.l1;
        factors[3] = hp.plan.l2;
        factors[4] = hp.plan.family;
    }
    dctmm_host_apply(hp, x, channels, y);
    return FREQKV_OK;
}

int32_t freqkv_gemm_fold_levels(int32_t n_in, int32_t kept_len, int32_t first_component)
{
    if (n_in < 1 || kept_len < 1 || kept_len > n_in || first_component < 0) return -1;
    return gemm_fold_levels(n_in, kept_len, first_component);
}

const char* freqkv_last_error(freqkv_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

const char* freqkv_status_string(freqkv_status status)
{
    switch (status) {
        case FREQKV_OK: return "FREQKV_OK";
        case FREQKV_ERR_INVALID_ARG: return "FREQKV_ERR_INVALID_ARG";
        case FREQKV_ERR_UNSUPPORTED: return "FREQKV_ERR_UNSUPPORTED";
        case FREQKV_ERR_CAPACITY: return "FREQKV_ERR_CAPACITY";
        case FREQKV_ERR_ALLOC: return "FREQKV_ERR_ALLOC";
        case FREQKV_ERR_CUDA: return "FREQKV_ERR_CUDA";
        case FREQKV_ERR_TIMEOUT: return "FREQKV_ERR_TIMEOUT";
    }
    return "FREQKV_ERR_UNKNOWN";
}

int32_t freqkv_version(void) { return 100; }

}  // extern "C"
