// Tensor-core execution of the compression Y = P X (Section 3.3, Eq. 2-3 with the transforms
// of Appendix A folded into the basis P, see basis.cu) on the 5th-generation tensor cores of
// sm_100a: tcgen05.mma with accumulators in tensor memory, operands staged by TMA.
//
// Shape of the problem.  P is L x N (bf16, row-major: the contraction axis is contiguous, a
// "K-major" A operand) and is shared by every matrix.  X_i is N x 128 per (batch, layer,
// kv_head) and tensor (K or V), with the 128 channels contiguous: an "MN-major" B operand.  The
// K matrix and the V matrix of the same (batch, layer, kv_head) sit side by side in one
// 256-column B tile, so K and V are compressed by the same launch and the same instructions.
//
// One CTA per SM, persistent over output tiles of 256 rows x 256 columns:
//   warp 0      TMA producer: per 64-token slice of the contraction, 2 boxes of P (128 rows x 64)
//               and 4 boxes of X (64 tokens x 64 channels; K low/high, V low/high), 128-byte
//               swizzled, into a 3-stage ring of 64 KB stages;
//   warp 1      MMA issuer: per stage 4 (k = 16) x 2 (row halves) tcgen05.mma of 128 x 256 x 16
//               into 2 x 256 fp32 columns of tensor memory (all 512 columns of the SM);
//   warps 2-9   epilogue: tcgen05.ld, round to bf16 (nearest even), 16-byte global stores.
//
// Every output row of a matrix depends on every input row of the same matrix and the output
// rows overwrite input rows, so tiles write to a scratch buffer; a copy kernel moves the rows
// into the cache when the launch is over.
//
// Every wait on an mbarrier is bounded in time: a wait that runs out sets a bit in the status
// word, raises a CTA-wide abort flag that ends every other role's loop, the producer drains
// its copies in flight, tensor memory is freed and the kernel returns.
#include <cuda.h>

#include <algorithm>
#include <cstdio>

#include "gemm.cuh"

namespace freqkv {
namespace {

constexpr int BM = 256;        // output rows per tile (two UMMA row halves of 128)
constexpr int BN = 256;        // output columns per tile: K channels 0..127 | V channels 0..127
constexpr int BK = 64;         // contraction slice per stage (tokens)
constexpr int STAGES = 3;
constexpr int A_HALF_BYTES = 128 * BK * 2;         // 16 KB: 128 rows x 64 bf16, 128 B per row
constexpr int A_BYTES = 2 * A_HALF_BYTES;          // 32 KB
constexpr int B_CHUNK_BYTES = BK * 128;            // 8 KB: 64 tokens x 64 channels
constexpr int B_BYTES = 4 * B_CHUNK_BYTES;         // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;     // 64 KB
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int NUM_THREADS = 320;                   // 10 warps
constexpr int EPI_WARPS = 8;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // 2 s

constexpr uint32_t ERR_FULL_WAIT = 1u, ERR_EMPTY_WAIT = 2u, ERR_ACC_FULL_WAIT = 4u, ERR_ACC_EMPTY_WAIT = 8u,
                   ERR_DRAIN_WAIT = 16u;

struct GemmParams {
    int32_t n_in, n_keep;       // N, L
    int32_t pair0, pair_count;  // (batch, layer, kv_head) triples covered by this launch
    int32_t layers, kv_heads;
    int32_t m_tiles, k_steps;
    __nv_bfloat16* scratch;     // [2][pair_count][n_keep][128]
    int32_t* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Wait for the phase with the given parity to complete.  Gives up when another role has raised
// the abort flag or after WAIT_LIMIT_NS; in the second case it records `err_bit` and raises the
// flag itself.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          uint32_t err_bit)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > WAIT_LIMIT_NS) {
            atomicOr(status, (int32_t)err_bit);
            *abort_flag = 1;
            __threadfence_block();
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c0, int32_t c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c0, int32_t c1,
                                            int32_t c2, int32_t c3, int32_t c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}

// Shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte offsets
// (all in 16-byte units), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;  // version
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}

// Instruction descriptor, kind::f16: D fp32, A and B bf16, A K-major, B MN-major, M = 128, N = 256.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((256u >> 3) << 17) |
                           ((128u >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(IDESC), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(uint32_t lo_bits, uint32_t hi_bits)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(lo_bits), __uint_as_float(hi_bits));
    return *reinterpret_cast<const uint32_t*>(&v);
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
freqkv_gemm_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const GemmParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte swizzle atoms need 1024-byte alignment
    uint8_t* aligned = smem_raw + (base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(aligned + STAGES * STAGE_BYTES);
    const uint32_t bar0 = base + STAGES * STAGE_BYTES;
    // barrier slots: full[0..S), empty[S..2S), acc_full (2S), acc_empty (2S+1)
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    const uint32_t acc_full_bar = bar0 + 8u * (2 * STAGES), acc_empty_bar = bar0 + 8u * (2 * STAGES + 1);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int32_t total_tiles = prm.pair_count * prm.m_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(acc_full_bar, 1);
        mbar_init(acc_empty_bar, EPI_WARPS);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {  // tensor memory: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t it = 0;  // global slice counter: stage = it % STAGES, phase = it / STAGES
            bool alive = true;
            for (int32_t tile = blockIdx.x; tile < total_tiles && alive; tile += gridDim.x) {
                const int32_t pair = prm.pair0 + tile / prm.m_tiles, mt = tile % prm.m_tiles;
                const int32_t h = pair % prm.kv_heads, l = (pair / prm.kv_heads) % prm.layers,
                              b = pair / (prm.kv_heads * prm.layers);
                for (int32_t ks = 0; ks < prm.k_steps; ++ks, ++it) {
                    const int s = it % STAGES;
                    if (it >= STAGES &&
                        !mbar_wait(empty_bar(s), ((it / STAGES) - 1) & 1, abort_flag, prm.status, ERR_EMPTY_WAIT)) {
                        alive = false;
                        break;
                    }
                    const uint32_t stage = base + s * STAGE_BYTES;
                    mbar_expect_tx(full_bar(s), STAGE_BYTES);
                    const int32_t k0 = ks * BK;
                    tma_load_2d(stage, &map_p, full_bar(s), k0, mt * BM);
                    tma_load_2d(stage + A_HALF_BYTES, &map_p, full_bar(s), k0, mt * BM + 128);
                    const uint32_t bs = stage + A_BYTES;
                    tma_load_5d(bs + 0 * B_CHUNK_BYTES, &map_k, full_bar(s), 0, k0, h, l, b);
                    tma_load_5d(bs + 1 * B_CHUNK_BYTES, &map_k, full_bar(s), 64, k0, h, l, b);
                    tma_load_5d(bs + 2 * B_CHUNK_BYTES, &map_v, full_bar(s), 0, k0, h, l, b);
                    tma_load_5d(bs + 3 * B_CHUNK_BYTES, &map_v, full_bar(s), 64, k0, h, l, b);
                }
            }
            if (*abort_flag) {
                // drain: every slice issued but possibly not yet landed completes its full barrier
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    int dummy = 0;
                    mbar_wait(full_bar(j % STAGES), (j / STAGES) & 1, &dummy, prm.status, ERR_DRAIN_WAIT);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            uint32_t it = 0, tile_no = 0;
            bool alive = true;
            for (int32_t tile = blockIdx.x; tile < total_tiles && alive; tile += gridDim.x, ++tile_no) {
                if (tile_no > 0) {  // accumulators must have been drained by the epilogue
                    if (!mbar_wait(acc_empty_bar, (tile_no - 1) & 1, abort_flag, prm.status, ERR_ACC_EMPTY_WAIT)) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                }
                for (int32_t ks = 0; ks < prm.k_steps; ++ks, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(full_bar(s), (it / STAGES) & 1, abort_flag, prm.status, ERR_FULL_WAIT)) {
                        alive = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a0 = base + s * STAGE_BYTES, b0 = a0 + A_BYTES;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk) {
                        // B: 4 chunks of 64 channels 8 KB apart (leading offset), 8-token groups 1 KB apart
                        const uint64_t bd = smem_desc(b0 + kk * 2048, B_CHUNK_BYTES, 1024);
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            // A: 128 rows, 8-row groups 1 KB apart; 16 k-elements = 32 bytes inside the swizzled row
                            const uint64_t ad = smem_desc(a0 + half * A_HALF_BYTES + kk * 32, 16, 1024);
                            umma_bf16(tmem_base + half * 256, ad, bd, (ks | kk) != 0);
                        }
                    }
                    umma_commit(empty_bar(s));  // frees the stage when these MMAs have read it
                }
                if (alive) umma_commit(acc_full_bar);
            }
        }
    } else {
        // ---------------- epilogue ----------------
        const int ew = warp - 2, quarter = warp % 4, half = ew / 4;
        uint32_t tile_no = 0;
        for (int32_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tile_no) {
            if (!mbar_wait(acc_full_bar, tile_no & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int32_t pair_local = tile / prm.m_tiles, mt = tile % prm.m_tiles;
            const int32_t m = mt * BM + half * 128 + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + half * 256;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t r[32];
                tmem_ld32(taddr + c * 32, r);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (m < prm.n_keep) {
                    const int tensor = c / 4;
                    __nv_bfloat16* out = prm.scratch +
                                         (((int64_t)tensor * prm.pair_count + pair_local) * prm.n_keep + m) * 128 +
                                         (c % 4) * 32;
                    uint4* o4 = reinterpret_cast<uint4*>(out);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint4 v;
                        v.x = pack_bf16(r[8 * q + 0], r[8 * q + 1]);
                        v.y = pack_bf16(r[8 * q + 2], r[8 * q + 3]);
                        v.z = pack_bf16(r[8 * q + 4], r[8 * q + 5]);
                        v.w = pack_bf16(r[8 * q + 6], r[8 * q + 7]);
                        o4[q] = v;
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar);
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
    }
}

// ---- host side ----

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

bool encode_basis_map(CUtensorMap* map, const Basis& basis)
{
    const cuuint64_t dims[2] = {(cuuint64_t)basis.ld, (cuuint64_t)basis.rows_pad};
    const cuuint64_t strides[1] = {(cuuint64_t)basis.ld * 2};
    const cuuint32_t box[2] = {BK, 128};
    const cuuint32_t elem[2] = {1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, basis.bf16, dims, strides, box, elem,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The non-sink rows of one cache tensor as a 5-D tensor (channel, token, kv_head, layer, batch).
bool encode_cache_map(CUtensorMap* map, const freqkv_layout& l, void* base, int32_t batch0, int32_t batch_count,
                      int32_t n_in, int32_t sink)
{
    char* p = static_cast<char*>(base) + ((int64_t)batch0 * l.stride_batch + (int64_t)sink * l.stride_token) * 2;
    const cuuint64_t dims[5] = {(cuuint64_t)l.head_dim, (cuuint64_t)n_in, (cuuint64_t)l.kv_heads, (cuuint64_t)l.layers,
                                (cuuint64_t)batch_count};
    // an axis of extent 1 is never stepped; give it a harmless stride
    const cuuint64_t row = (cuuint64_t)l.stride_token * 2;
    const cuuint64_t strides[4] = {row, l.kv_heads > 1 ? (cuuint64_t)l.stride_head * 2 : row,
                                   l.layers > 1 ? (cuuint64_t)l.stride_layer * 2 : row,
                                   batch_count > 1 ? (cuuint64_t)l.stride_batch * 2 : row};
    const cuuint32_t box[5] = {64, BK, 1, 1, 1};
    const cuuint32_t elem[5] = {1, 1, 1, 1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, p, dims, strides, box, elem,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t kGemmScratchBytes = size_t(1) << 30;

}  // namespace

bool gemm_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep)
{
    return dtype == FREQKV_BF16 && head_dim == 128 && n_in >= 1 && n_keep >= 1 && n_keep <= n_in;
}

cudaError_t launch_gemm(GemmState* state, const CacheView& view, const freqkv_layout& layout, void* k, void* v,
                        int32_t batch0, int32_t batch_count, const Basis& basis, int32_t sink, int32_t* status_dev,
                        int sm_count, const LaunchHooks& hooks, cudaStream_t stream)
{
    state->kernels_last_call = 0;
    state->last_error = nullptr;
    if (!encode_fn()) {
        state->last_error = "cuTensorMapEncodeTiled is not available from this driver";
        return cudaErrorNotSupported;
    }
    if (!state->attr_set) {
        const cudaError_t e = cudaFuncSetAttribute(freqkv_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) {
            state->last_error = "cudaFuncSetAttribute(max dynamic shared memory)";
            return e;
        }
        state->attr_set = true;
    }
    CUtensorMap map_p, map_k, map_v;
    if (!encode_basis_map(&map_p, basis) ||
        !encode_cache_map(&map_k, layout, k, batch0, batch_count, basis.n_in, sink) ||
        !encode_cache_map(&map_v, layout, v, batch0, batch_count, basis.n_in, sink)) {
        state->last_error = "tensor map encoding rejected this layout";
        return cudaErrorInvalidValue;
    }

    const int32_t pairs = view.mats_per_tensor;
    const size_t per_pair = (size_t)2 * basis.n_keep * 128 * 2;
    int32_t chunk = (int32_t)std::max<size_t>(1, std::min<size_t>(kGemmScratchBytes / per_pair, (size_t)pairs));
    if ((size_t)chunk * per_pair > state->scratch_bytes) {
        if (state->scratch) {
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) return e;
            cudaFree(state->scratch);
            state->scratch = nullptr;
            state->scratch_bytes = 0;
        }
        const cudaError_t e = cudaMalloc(&state->scratch, (size_t)chunk * per_pair);
        if (e != cudaSuccess) {
            state->last_error = "cudaMalloc(gemm scratch)";
            return e;
        }
        state->scratch_bytes = (size_t)chunk * per_pair;
    }

    for (int32_t p0 = 0; p0 < pairs; p0 += chunk) {
        const int32_t count = std::min(chunk, pairs - p0);
        GemmParams prm;
        prm.n_in = basis.n_in;
        prm.n_keep = basis.n_keep;
        prm.pair0 = p0;
        prm.pair_count = count;
        prm.layers = view.layers;
        prm.kv_heads = view.kv_heads;
        prm.m_tiles = (basis.n_keep + BM - 1) / BM;
        prm.k_steps = (basis.n_in + BK - 1) / BK;
        prm.scratch = static_cast<__nv_bfloat16*>(state->scratch);
        prm.status = status_dev;
        const int32_t tiles = count * prm.m_tiles;
        const int grid = std::min<int32_t>(tiles, sm_count);
        if (hooks.before) hooks.before(hooks.user, stream);
        freqkv_gemm_kernel<<<grid, NUM_THREADS, SMEM_BYTES, stream>>>(map_p, map_k, map_v, prm);
        cudaError_t e = cudaGetLastError();
        if (hooks.after) hooks.after(hooks.user, stream);
        if (e != cudaSuccess) {
            state->last_error = "freqkv_gemm_kernel launch";
            return e;
        }
        const __nv_bfloat16* sk = prm.scratch;
        const __nv_bfloat16* sv = prm.scratch + (size_t)count * basis.n_keep * 128;
        e = launch_copy_back(view, FREQKV_BF16, p0, count, basis.n_keep, sink, sk, stream);
        if (e == cudaSuccess)
            e = launch_copy_back(view, FREQKV_BF16, view.mats_per_tensor + p0, count, basis.n_keep, sink, sv, stream);
        if (e != cudaSuccess) {
            state->last_error = "copy_back launch";
            return e;
        }
        state->kernels_last_call += 3;
    }
    return cudaSuccess;
}

void gemm_release(GemmState* state)
{
    if (state->scratch) cudaFree(state->scratch);
    state->scratch = nullptr;
    state->scratch_bytes = 0;
}

}  // namespace freqkv
