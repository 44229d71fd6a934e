// Attention of a chunk of incoming tokens over the bounded cache (Section 3.3: during training
// and prefilling the sequence is processed chunk-wise, attention interleaved with compression;
// first attention equation), with the position encoding of Section 3.4: keys are cached before
// RoPE and rotated to their row index inside the cache, each query to its own row index.
//
// The chunk's n tokens sit in cache rows [len - n, len).  Token i attends causally to rows
// [0, len - n + i].  Per (sequence, query head) this is a dense (n x len) x 128 contraction twice
// over -- the attention matrix of a chunk is (N - L - S) x N in the paper's count -- so it runs on
// the tcgen05 tensor cores:
//
//   pass 1 (CUDA cores, one read of the layer's keys and of the queries): rotate the keys of the
//     layer and the queries of the chunk, the queries also scaled by scale * log2(e), and round
//     them to fp16 into scratch (fp16 rather than bf16: three more mantissa bits keep the error of
//     the scores a quarter of bf16's).  Key rows from the length to the next multiple of the key
//     tile are written as zeros.
//   pass 2, one CTA per (sequence, query head, 128 queries), 192 threads, two CTAs per SM (each
//   holds half of the shared memory and of the tensor memory, so that one CTA's softmax overlaps
//   the other's tensor-core work); the query tiles with the most keys are scheduled first:
//     warp 0   TMA producer: the query tile once; per key tile of 64 rows the rotated keys and,
//              straight from the cache through a 5-D tensor map, the values (two-stage rings);
//     warp 1   MMA issuer: S = Q K_rot^T (fp16 in, fp32 in tensor memory, two S buffers so that
//              the next tile's scores are computed while this tile's softmax runs), then
//              O += P V (bf16 in; P is read from tensor memory, V is the MN-major operand, as
//              it lies in the cache);
//     warps 2-5 softmax, one query row per thread (tensor-memory lane = row): read the row of S,
//              causal mask on the diagonal tiles, running maximum and sum in base 2, weights rounded
//              to bf16 and written back over the first 32 columns of the same S buffer (two
//              per column, in key order: the A operand of the second product; the MMAs of one
//              thread execute in order, so the scores that later overwrite the buffer cannot
//              overtake the product that reads the weights).  O stays in tensor
//              memory; it is rescaled (read, multiplied, written back) only when a row's maximum
//              has grown by more than 2^8 since the reference was last moved -- the weights stay
//              below 2^8 meanwhile, and the final division by the running sum makes the result
//              independent of the reference.  Value rows past the cache length (stale cache
//              contents, possibly not finite) are zeroed in shared memory before they are used.
//     At the end the softmax threads read O, divide by the row sums and store bf16 rows.
// Every barrier wait is bounded in time; a wait that runs out sets a status bit and an abort flag
// that ends all roles, after which the CTA lets copies in flight land and frees its tensor memory.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "prefill.cuh"

namespace freqkv {
namespace {

constexpr int BQ = 128;             // queries per CTA
constexpr int BKV = 64;             // keys per tile
constexpr int Q_SLAB = BQ * 128;    // bytes: 128 rows x 64 two-byte values, one 128-byte swizzle row each
constexpr int Q_TILE = 2 * Q_SLAB;  // 128 queries x 128 channels
constexpr int KV_SLAB = BKV * 128;  // 64 rows x 64 channels
constexpr int KV_TILE = 2 * KV_SLAB;
constexpr int RING_K = 2, RING_V = 2;  // stages of the key ring and of the value ring (a third key stage measured no faster)
constexpr int OFF_Q = 0, OFF_K = Q_TILE, OFF_V = OFF_K + RING_K * KV_TILE, OFF_BAR = OFF_V + RING_V * KV_TILE;
constexpr int SMEM_USED = OFF_BAR + 256;
constexpr int SMEM_BYTES = SMEM_USED + 1024;  // + slack for aligning the base to 1024 bytes
static_assert(2 * (SMEM_BYTES + 1024) <= 233472, "two CTAs per SM (1 KB of each CTA's share is reserved)");
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 256;      // S buffers in columns 0..63 and 64..127, O in 128..255
constexpr unsigned long long LANDING_NS = 1000000ull;        // 1 ms
constexpr float NEG_INF = -INFINITY;
constexpr float RESCALE_STEP = 8.f;  // log2 of the largest weight the lazy reference allows

struct PrefillParams {
    int32_t n_new, kv_heads, g, layer, batch0, batch_count, q_tiles;
    __nv_bfloat16* out;  // [batch, kv_heads * g, n_new, 128]
    int32_t* status;
    unsigned long long wait_limit_ns;  // bound of every mbarrier wait
    int32_t len[PREFILL_MAX_BATCH];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
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
// Wait for the phase with the given parity.  Gives up when another role has raised the abort flag
// or after `limit_ns` (then it sets the status bit and raises the flag).  False = gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          unsigned long long limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) {
            atomicOr(status, PREFILL_ERR_WAIT);
            *abort_flag = 1;
            __threadfence_block();
            return false;
        }
    }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c0, int32_t c1, int32_t c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c0, int32_t c1, int32_t c2,
                                            int32_t c3, int32_t c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
// Shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte offsets
// (16-byte units), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptors, kind::f16, D fp32, M = 128.
// Scores (N = 64 keys): A and B fp16, both K-major.  Values (N = 128 channels): A and B bf16, A K-major, B MN-major.
constexpr uint32_t IDESC_QK = (1u << 4) | (0u << 7) | (0u << 10) | (0u << 15) | (0u << 16) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with the A operand in tensor memory: lane = row, 16-bit elements two per column in the
// order of the contraction index.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// When every MMA issued so far has finished, arrive on the barrier.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive columns of tensor memory <-> registers r[OFF .. OFF+31].
template <int OFF, int NREG>
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[NREG])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[OFF + 0]), "=r"(r[OFF + 1]), "=r"(r[OFF + 2]), "=r"(r[OFF + 3]), "=r"(r[OFF + 4]), "=r"(r[OFF + 5]),
          "=r"(r[OFF + 6]), "=r"(r[OFF + 7]), "=r"(r[OFF + 8]), "=r"(r[OFF + 9]), "=r"(r[OFF + 10]), "=r"(r[OFF + 11]),
          "=r"(r[OFF + 12]), "=r"(r[OFF + 13]), "=r"(r[OFF + 14]), "=r"(r[OFF + 15]), "=r"(r[OFF + 16]),
          "=r"(r[OFF + 17]), "=r"(r[OFF + 18]), "=r"(r[OFF + 19]), "=r"(r[OFF + 20]), "=r"(r[OFF + 21]),
          "=r"(r[OFF + 22]), "=r"(r[OFF + 23]), "=r"(r[OFF + 24]), "=r"(r[OFF + 25]), "=r"(r[OFF + 26]),
          "=r"(r[OFF + 27]), "=r"(r[OFF + 28]), "=r"(r[OFF + 29]), "=r"(r[OFF + 30]), "=r"(r[OFF + 31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
          "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
          "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
        : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// ---- pass 1: rotate and round to fp16 ----
//
// A half-warp per row; lane l16 holds the channel pairs (4 l16 + i, 64 + 4 l16 + i), i < 4.
// Rows [0, k_rows) of every (sequence, kv head) of the layer are key rows (zeros from the length
// on); the remaining jobs are the chunk's query rows.
struct RopeJob {
    const __nv_bfloat16* k;  // layer base of the key cache
    int64_t stride_batch, stride_head, stride_token;
    const __nv_bfloat16* q;  // [batch, heads_q, n_new, 128]
    __half* k_out;           // [batch * kv_heads][capacity][128]
    __half* q_out;           // [batch * heads_q][n_new][128]
    const float2* table;     // [capacity][64] or null
    float qscale;
    int32_t kv_heads, heads_q, n_new, capacity, k_rows, batch0, batch_count;
    int32_t len[PREFILL_MAX_BATCH];
};

__global__ void __launch_bounds__(256) prefill_rope_kernel(const RopeJob job)
{
    // blockIdx.y: a (sequence, kv head) slice of keys, then the (sequence, query head) slices of queries;
    // blockIdx.x: 64 consecutive rows of the slice, 4 per half-warp
    const int l16 = threadIdx.x % 16, c0 = 4 * l16;
    const int32_t k_slices = job.batch_count * job.kv_heads;
    const bool is_key = (int32_t)blockIdx.y < k_slices;
    const int32_t slice = is_key ? (int32_t)blockIdx.y : (int32_t)blockIdx.y - k_slices;
    const int32_t heads = is_key ? job.kv_heads : job.heads_q, b = slice / heads, hh = slice % heads;
    const int32_t rows = is_key ? job.k_rows : job.n_new, len = job.len[b];
    const __nv_bfloat16* src0;
    __half* dst0;
    int64_t src_stride;
    if (is_key) {
        src0 = job.k + (int64_t)(job.batch0 + b) * job.stride_batch + (int64_t)hh * job.stride_head;
        src_stride = job.stride_token;
        dst0 = job.k_out + ((int64_t)(job.batch0 + b) * job.kv_heads + hh) * job.capacity * 128;
    } else {
        const int64_t at = ((int64_t)(job.batch0 + b) * job.heads_q + hh) * job.n_new * 128;
        src0 = job.q + at;
        src_stride = 128;
        dst0 = job.q_out + at;
    }
    const float mul = is_key ? 1.f : job.qscale;
    const int32_t pos0 = is_key ? 0 : len - job.n_new;
#pragma unroll
    for (int i4 = 0; i4 < 4; ++i4) {
        const int32_t row = (int32_t)blockIdx.x * 64 + (threadIdx.x / 16) * 4 + i4;
        if (row >= rows) break;
        uint2 lo_out = make_uint2(0u, 0u), hi_out = make_uint2(0u, 0u);
        if (!(is_key && row >= len)) {  // key rows from the length on are written as zeros
            const __nv_bfloat16* src = src0 + (int64_t)row * src_stride;
            const uint2 ulo = __ldg(reinterpret_cast<const uint2*>(src + c0)), uhi = __ldg(reinterpret_cast<const uint2*>(src + 64 + c0));
            float lo[4] = {__uint_as_float(ulo.x << 16), __uint_as_float(ulo.x & 0xffff0000u), __uint_as_float(ulo.y << 16),
                           __uint_as_float(ulo.y & 0xffff0000u)};
            float hi[4] = {__uint_as_float(uhi.x << 16), __uint_as_float(uhi.x & 0xffff0000u), __uint_as_float(uhi.y << 16),
                           __uint_as_float(uhi.y & 0xffff0000u)};
            if (job.table) {
                const float4* t = reinterpret_cast<const float4*>(job.table + (int64_t)(pos0 + row) * 64 + c0);
                const float4 t0 = __ldg(t), t1 = __ldg(t + 1);
                const float cs[4] = {t0.x, t0.z, t1.x, t1.z}, sn[4] = {t0.y, t0.w, t1.y, t1.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float a = lo[i] * cs[i] - hi[i] * sn[i], bb = hi[i] * cs[i] + lo[i] * sn[i];
                    lo[i] = a;
                    hi[i] = bb;
                }
            }
            lo_out = make_uint2(pack_f16(lo[0] * mul, lo[1] * mul), pack_f16(lo[2] * mul, lo[3] * mul));
            hi_out = make_uint2(pack_f16(hi[0] * mul, hi[1] * mul), pack_f16(hi[2] * mul, hi[3] * mul));
        }
        __half* dst = dst0 + (int64_t)row * 128;
        *reinterpret_cast<uint2*>(dst + c0) = lo_out;
        *reinterpret_cast<uint2*>(dst + 64 + c0) = hi_out;
    }
}

// ---- pass 2 ----
__global__ void __launch_bounds__(THREADS, 2)
prefill_attend_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v, const PrefillParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzle atoms need 1024-byte alignment
    uint8_t* aligned = smem_raw + (base - raw);
    const uint32_t bar0 = base + OFF_BAR;
    // barriers: q_full, p_ready, o_full, s_full[2], s_free[2], then per ring stage k_full, k_empty, v_full, v_empty
    const uint32_t q_full = bar0, p_ready = bar0 + 8u, o_full = bar0 + 16u;
    auto s_full = [&](int s) { return bar0 + 8u * (3 + s); };
    auto s_free = [&](int s) { return bar0 + 8u * (5 + s); };
    auto k_full = [&](int s) { return bar0 + 8u * (7 + s); };
    auto k_empty = [&](int s) { return bar0 + 8u * (7 + RING_K + s); };
    auto v_full = [&](int s) { return bar0 + 8u * (7 + 2 * RING_K + s); };
    auto v_empty = [&](int s) { return bar0 + 8u * (7 + 2 * RING_K + RING_V + s); };
    constexpr int N_BARRIERS = 7 + 2 * RING_K + 2 * RING_V;
    static_assert(8 * N_BARRIERS + 8 <= 256, "barrier area");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aligned + OFF_BAR + 8 * N_BARRIERS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    // heaviest work first: the first blocks are the last query tiles (the most keys) of all heads
    const int32_t heads_q = prm.kv_heads * prm.g, units = heads_q * prm.batch_count;
    const int32_t q_tile = prm.q_tiles - 1 - (int32_t)blockIdx.x / units;
    const int32_t unit = (int32_t)blockIdx.x % units, b = unit / heads_q, hq = unit % heads_q, h = hq / prm.g;
    const int32_t q0 = q_tile * BQ;
    const int32_t len = prm.len[b], pos0 = len - prm.n_new;         // position of the chunk's first token
    const int32_t last_pos = pos0 + min(q0 + BQ, prm.n_new) - 1;    // of this tile's last valid query
    const int32_t n_tiles = last_pos / BKV + 1;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < RING_K; ++s) {
            mbar_init(k_full(s), 1);
            mbar_init(k_empty(s), 1);
        }
        for (int s = 0; s < RING_V; ++s) {
            mbar_init(v_full(s), 1);
            mbar_init(v_empty(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(s_full(s), 1);
            mbar_init(s_free(s), 4);  // lane 0 of each softmax warp
        }
        mbar_init(p_ready, 128);      // every softmax thread
        mbar_init(o_full, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 128;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const int32_t q_slice = (prm.batch0 + b) * heads_q + hq, k_slice = (prm.batch0 + b) * prm.kv_heads + h;
            // launched with programmatic stream serialization: the set-up above may run while pass 1 drains; its
            // output (read only through these loads) is complete and visible after this wait
            asm volatile("griddepcontrol.wait;" ::: "memory");
            mbar_expect_tx(q_full, Q_TILE);
            tma_load_3d(base + OFF_Q, &map_q, q_full, 0, q0, q_slice);
            tma_load_3d(base + OFF_Q + Q_SLAB, &map_q, q_full, 64, q0, q_slice);
            for (int32_t t = 0; t < n_tiles; ++t) {
                const int sk = t % RING_K, sv = t % RING_V;
                if (t >= RING_K && !mbar_wait(k_empty(sk), ((uint32_t)(t / RING_K) - 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) break;
                mbar_expect_tx(k_full(sk), KV_TILE);
                tma_load_3d(base + OFF_K + sk * KV_TILE, &map_k, k_full(sk), 0, t * BKV, k_slice);
                tma_load_3d(base + OFF_K + sk * KV_TILE + KV_SLAB, &map_k, k_full(sk), 64, t * BKV, k_slice);
                if (t >= RING_V && !mbar_wait(v_empty(sv), ((uint32_t)(t / RING_V) - 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) break;
                mbar_expect_tx(v_full(sv), KV_TILE);
                tma_load_5d(base + OFF_V + sv * KV_TILE, &map_v, v_full(sv), 0, t * BKV, h, prm.layer, prm.batch0 + b);
                tma_load_5d(base + OFF_V + sv * KV_TILE + KV_SLAB, &map_v, v_full(sv), 64, t * BKV, h, prm.layer, prm.batch0 + b);
            }
            if (*abort_flag) {  // let the copies in flight land before this CTA's shared memory goes away
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < LANDING_NS) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            bool alive = mbar_wait(q_full, 0, abort_flag, prm.status, prm.wait_limit_ns);
            auto issue_scores = [&](int32_t t) {
                const int s = t % RING_K;
                if (!mbar_wait(k_full(s), (uint32_t)(t / RING_K) & 1, abort_flag, prm.status, prm.wait_limit_ns)) return false;
                if (t >= 2 && !mbar_wait(s_free(t & 1), ((uint32_t)(t / 2) - 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) return false;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t qa = base + OFF_Q, ka = base + OFF_K + s * KV_TILE;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)  // 16 channels per instruction; 64-channel slabs, 32 bytes per step inside one
                    umma(tmem_base + (t & 1) * BKV, smem_desc(qa + (kk / 4) * Q_SLAB + (kk % 4) * 32, 16, 1024),
                         smem_desc(ka + (kk / 4) * KV_SLAB + (kk % 4) * 32, 16, 1024), IDESC_QK, kk != 0);
                umma_commit(s_full(t & 1));
                umma_commit(k_empty(s));
                return true;
            };
            if (alive) alive = issue_scores(0);
            for (int32_t t = 0; t < n_tiles && alive; ++t) {
                if (t + 1 < n_tiles && !issue_scores(t + 1)) break;
                const int s = t % RING_V;
                if (!mbar_wait(p_ready, t & 1, abort_flag, prm.status, prm.wait_limit_ns)) break;
                if (!mbar_wait(v_full(s), (uint32_t)(t / RING_V) & 1, abort_flag, prm.status, prm.wait_limit_ns)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t va = base + OFF_V + s * KV_TILE;
#pragma unroll
                for (int kk = 0; kk < BKV / 16; ++kk)  // 16 keys per instruction
                    // P: in tensor memory over the first 32 columns of this tile's S buffer, 8 columns per step.
                    // V: MN-major, 16 key rows = 2 KB per step, 64-channel slabs KV_SLAB apart.
                    umma_ts(tmem_o, tmem_base + (t & 1) * BKV + kk * 8, smem_desc(va + kk * 2048, KV_SLAB, 1024), IDESC_PV, (t | kk) != 0);
                umma_commit(o_full);
                umma_commit(v_empty(s));
            }
        }
    } else {
        // ---------------- softmax and epilogue: one query row per thread ----------------
        const int quarter = warp % 4, row = quarter * 32 + lane;     // tensor-memory lane = row of the tile
        const uint32_t lane_bits = (uint32_t)(quarter * 32) << 16;
        const int32_t my_pos = pos0 + q0 + row;                      // keys up to this index are visible
        const int32_t warp_pos = pos0 + q0 + quarter * 32;           // the smallest position in this warp
        float m_ref = NEG_INF, l_run = 0.f;
        bool alive = true;
        for (int32_t t = 0; t < n_tiles; ++t) {
            const int buf = t & 1, s = t % RING_V;
            const int32_t j0 = t * BKV;
            if (!mbar_wait(s_full(buf), (t / 2) & 1, abort_flag, prm.status, prm.wait_limit_ns)) { alive = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t sc[64];
            tmem_ld32<0>(tmem_base + lane_bits + buf * BKV + 0, sc);
            tmem_ld32<32>(tmem_base + lane_bits + buf * BKV + 32, sc);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(s_free(buf));

            if (j0 + BKV - 1 > warp_pos) {  // a tile on the diagonal: hide the keys after each row's own
#pragma unroll
                for (int j = 0; j < 64; ++j)
                    if (j0 + j > my_pos) sc[j] = __float_as_uint(NEG_INF);
            }
            float m4[4] = {NEG_INF, NEG_INF, NEG_INF, NEG_INF};  // four chains instead of one of 64
#pragma unroll
            for (int j = 0; j < 64; ++j) m4[j & 3] = fmaxf(m4[j & 3], __uint_as_float(sc[j]));
            const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
            // move the reference only when the maximum has outgrown it by more than RESCALE_STEP
            float factor = 1.f;
            const bool grow = mx > m_ref + RESCALE_STEP;   // true at the first tile (m_ref = -inf, key 0 is visible to every row)
            if (grow) {
                factor = ex2(m_ref - mx);                  // 0 at the first tile
                l_run *= factor;
                m_ref = mx;
            }
            uint32_t pk[32];
            float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float p0 = ex2(__uint_as_float(sc[2 * j]) - m_ref), p1 = ex2(__uint_as_float(sc[2 * j + 1]) - m_ref);
                s4[j & 3] += p0 + p1;
                pk[j] = pack_bf16(p0, p1);
            }
            l_run += (s4[0] + s4[1]) + (s4[2] + s4[3]);

            if (t > 0) {  // the previous tile's P V must have finished: P is free, O is at rest
                if (!mbar_wait(o_full, (t - 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) { alive = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (__any_sync(0xffffffffu, grow)) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t o[32];
                        tmem_ld32<0>(tmem_o + lane_bits + c * 32, o);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * factor);
                        tmem_st32(tmem_o + lane_bits + c * 32, o);
                    }
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            }
            // weights over the first 32 columns of this tile's S buffer (bf16 pairs): the A operand of P V.  The scores that
            // overwrite the buffer (tile t + 2) are issued behind that P V, and one thread's MMAs execute in order.
            tmem_st32(tmem_base + lane_bits + buf * BKV, pk);
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (j0 + BKV > len) {  // value rows past the cache length are stale: make them zeros
                if (!mbar_wait(v_full(s), (uint32_t)(t / RING_V) & 1, abort_flag, prm.status, prm.wait_limit_ns)) { alive = false; break; }
                if (row < BKV && j0 + row >= len) {
                    uint8_t* v_row = aligned + OFF_V + s * KV_TILE + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        *reinterpret_cast<uint4*>(v_row + c * 16) = make_uint4(0u, 0u, 0u, 0u);
                        *reinterpret_cast<uint4*>(v_row + KV_SLAB + c * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> the tensor core's reads
            }
            mbar_arrive(p_ready);
        }
        if (alive && mbar_wait(o_full, (n_tiles - 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const float inv = 1.f / l_run;
            const bool store = q0 + row < prm.n_new;
            uint4* out = reinterpret_cast<uint4*>(prm.out + ((((int64_t)(prm.batch0 + b) * heads_q + hq) * prm.n_new + q0 + row) * 128));
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tmem_ld32<0>(tmem_o + lane_bits + c * 32, o);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (store) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        out[c * 4 + j] = make_uint4(pack_bf16(__uint_as_float(o[8 * j]) * inv, __uint_as_float(o[8 * j + 1]) * inv),
                                                    pack_bf16(__uint_as_float(o[8 * j + 2]) * inv, __uint_as_float(o[8 * j + 3]) * inv),
                                                    pack_bf16(__uint_as_float(o[8 * j + 4]) * inv, __uint_as_float(o[8 * j + 5]) * inv),
                                                    pack_bf16(__uint_as_float(o[8 * j + 6]) * inv, __uint_as_float(o[8 * j + 7]) * inv));
                }
            }
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS));
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

// fp16 scratch as (channel, row, slice), read in boxes of 64 channels x box_rows rows; rows past the extent read as zeros.
bool encode_rows_map(CUtensorMap* map, void* base, int64_t rows, int64_t slices, uint32_t box_rows)
{
    const cuuint64_t dims[3] = {128, (cuuint64_t)rows, (cuuint64_t)slices};
    const cuuint64_t strides[2] = {256, (cuuint64_t)rows * 256};
    const cuuint32_t box[3] = {64, box_rows, 1};
    const cuuint32_t elem[3] = {1, 1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The value cache as (channel, token, kv_head, layer, batch); tokens past the capacity read as zeros.
bool encode_value_map(CUtensorMap* map, const freqkv_layout& l, const void* v)
{
    const cuuint64_t dims[5] = {128, (cuuint64_t)l.capacity, (cuuint64_t)l.kv_heads, (cuuint64_t)l.layers, (cuuint64_t)l.batch};
    const cuuint64_t row = (cuuint64_t)l.stride_token * 2;  // an axis of extent 1 is never stepped: any valid stride will do
    const cuuint64_t strides[4] = {row, l.kv_heads > 1 ? (cuuint64_t)l.stride_head * 2 : row,
                                   l.layers > 1 ? (cuuint64_t)l.stride_layer * 2 : row,
                                   l.batch > 1 ? (cuuint64_t)l.stride_batch * 2 : row};
    const cuuint32_t box[5] = {64, BKV, 1, 1, 1};
    const cuuint32_t elem[5] = {1, 1, 1, 1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(v), dims, strides, box, elem,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool prefill_supported(int32_t dtype, int32_t head_dim, int32_t q_heads_per_kv)
{
    return dtype == FREQKV_BF16 && head_dim == 128 && q_heads_per_kv >= 1 && q_heads_per_kv <= 64;
}

size_t prefill_key_scratch_bytes(const freqkv_layout& l) { return (size_t)l.batch * l.kv_heads * l.capacity * 256; }

size_t prefill_query_scratch_bytes(const freqkv_layout& l, int32_t q_heads_per_kv, int32_t n_new)
{
    return (size_t)l.batch * l.kv_heads * q_heads_per_kv * n_new * 256;
}

cudaError_t launch_prefill(const freqkv_layout& l, const void* k, const void* v, int32_t layer, const void* q, void* out,
                           int32_t g, int32_t n_new, const int32_t* lens_host, const float2* table, float scale,
                           void* key_scratch, void* query_scratch, int32_t* status, unsigned long long wait_limit_ns,
                           const char** error, int32_t* kernels_launched, cudaStream_t stream)
{
    *error = nullptr;
    if (!encode_fn()) {
        *error = "cuTensorMapEncodeTiled is not available from this driver";
        return cudaErrorNotSupported;
    }
    static PerDeviceOnce attrs;
    const cudaError_t attr_error = attrs.run([] {
        cudaError_t e = cudaFuncSetAttribute(prefill_attend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(prefill_attend_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        return e;
    });
    if (attr_error != cudaSuccess) return attr_error;
    const int32_t heads_q = l.kv_heads * g;
    CUtensorMap map_q, map_k, map_v;
    if (!encode_rows_map(&map_q, query_scratch, n_new, (int64_t)l.batch * heads_q, BQ) ||
        !encode_rows_map(&map_k, key_scratch, l.capacity, (int64_t)l.batch * l.kv_heads, BKV) || !encode_value_map(&map_v, l, v)) {
        *error = "cuTensorMapEncodeTiled rejected a tensor of the prefill attention";
        return cudaErrorInvalidValue;
    }
    // sequences per launch: their lengths travel as kernel arguments, and the pre-pass puts one slice per grid row
    const int32_t per_launch = std::max(1, std::min(PREFILL_MAX_BATCH, 65535 / (l.kv_heads + l.kv_heads * g)));
    for (int32_t b0 = 0; b0 < l.batch; b0 += per_launch) {
        const int32_t nb = std::min(per_launch, l.batch - b0);
        int32_t max_len = 0;
        RopeJob job;
        job.k = static_cast<const __nv_bfloat16*>(k) + (int64_t)layer * l.stride_layer;
        job.stride_batch = l.stride_batch;
        job.stride_head = l.stride_head;
        job.stride_token = l.stride_token;
        job.q = static_cast<const __nv_bfloat16*>(q);
        job.k_out = static_cast<__half*>(key_scratch);
        job.q_out = static_cast<__half*>(query_scratch);
        job.table = table;
        job.qscale = scale * 1.4426950408889634f;
        job.kv_heads = l.kv_heads;
        job.heads_q = heads_q;
        job.n_new = n_new;
        job.capacity = l.capacity;
        job.batch0 = b0;
        job.batch_count = nb;
        PrefillParams prm;
        for (int32_t i = 0; i < nb; ++i) {
            job.len[i] = prm.len[i] = lens_host[b0 + i];
            max_len = std::max(max_len, lens_host[b0 + i]);
        }
        job.k_rows = std::min(l.capacity, (max_len + BKV - 1) / BKV * BKV);
        const dim3 rope_grid((unsigned)((std::max(job.k_rows, n_new) + 63) / 64), (unsigned)(nb * (l.kv_heads + heads_q)));
        prefill_rope_kernel<<<rope_grid, 256, 0, stream>>>(job);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        prm.n_new = n_new;
        prm.kv_heads = l.kv_heads;
        prm.g = g;
        prm.layer = layer;
        prm.batch0 = b0;
        prm.batch_count = nb;
        prm.q_tiles = (n_new + BQ - 1) / BQ;
        prm.out = static_cast<__nv_bfloat16*>(out);
        prm.status = status;
        prm.wait_limit_ns = wait_limit_ns;
        const dim3 grid((unsigned)((int64_t)prm.q_tiles * heads_q * nb));
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(THREADS);
        cfg.dynamicSmemBytes = SMEM_BYTES;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;  // let the launch overlap the tail of pass 1
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, prefill_attend_kernel, map_q, map_k, map_v, prm);
        if (e != cudaSuccess) return e;
        *kernels_launched += 2;
    }
    return cudaSuccess;
}

}  // namespace freqkv
