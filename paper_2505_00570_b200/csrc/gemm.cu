// Tensor-core execution of the compression Y = P X (Section 3.3, Eq. 2-3 with the transforms
// of Appendix A folded into the basis P, see basis.cu) on the 5th-generation tensor cores of
// sm_100a: tcgen05.mma with accumulators in tensor memory, operands staged by TMA.
//
// Symmetry fold.  The DCT cosines are even or odd under n -> N-1-n (and m -> L-1-m) according to
// the parity of the frequency t, so with P = Pe + Po split into its even-t and odd-t parts
//     u_n = x_n + x_{N-1-n},   v_n = x_n - x_{N-1-n}            (n < ceil(N/2))
//     s_m = sum_n Pe[m][n] u_n,   d_m = sum_n Po[m][n] v_n      (m < ceil(L/2))
//     y_m = s_m + d_m,   y_{L-1-m} = s_m - d_m
// which is the same linear map with half the multiply-adds.  (For odd N the middle row enters u
// once and v as zero; for odd L the middle output row has d = 0 and is written once.)
// For even L the even part Pe is itself the basis of a compression of N/2 rows to L/2, so where N is a
// multiple of 4 it is folded once more (uu, uv; Pee, Peo; see MODE_FOLD2 and basis.cu): three quarters
// of these multiply-adds again.  The two-level form is what a plain compression of such lengths
// runs (the paper's 4092 -> 2046 and 4096 -> 2048); the description below is the one-level form, which
// serves every other length, retained bands, ragged batches and the power spectrum.
//
// Two kernels per call:
//   fold_kernel         reads every non-sink cache row once and writes U and V (bf16) to a scratch
//                       buffer, one plane of ceil(N/2) x 128 per (matrix, u|v); HBM-bound.
//   freqkv_gemm_kernel  persistent, one CTA per SM, CTAs paired into clusters of two that share
//                       every MMA (tcgen05 cta_group::2).  A cluster works on output tiles of 256
//                       folded rows x 256 columns (the K matrix and the V matrix of one (batch,
//                       layer, kv_head) side by side, so K and V share every instruction): CTA r
//                       of the pair holds rows 128 r .. 128 r + 127 of the basis slice and of the
//                       accumulators, and HALF of the input slice (r = 0: the K channels, r = 1: the
//                       V channels) -- the tensor cores of both SMs read both halves, so every
//                       byte of U / V is brought into shared memory once per 256 output rows.  Per
//                       tile the pair first accumulates S = Pe U, then D = Po V, in the two halves
//                       of tensor memory.  In each CTA:
//     warp 0      TMA producer: per 64-row slice of the contraction one box of Pe or Po (128 x 64)
//                 and 2 boxes of U or V (64 rows x 64 channels), 128-byte swizzled, into a ring
//                 of 6 stages of 32 KB; the bytes of both CTAs complete the leader's barrier;
//     warp 1      MMA issuer (leader CTA only): 4 tcgen05.mma (256 x 256 x 16) per stage, commits
//                 multicast to the barriers of both CTAs;
//     warps 2-9   epilogue: when S is complete they park it in registers (which frees that half
//                 of tensor memory for the next tile while D is still accumulating); when D is
//                 complete they form s + d and s - d, round to bf16 (nearest even) and store rows
//                 m and L-1-m straight into the cache.  Both steps overlap the MMAs of the
//                 neighbouring phases, so the tensor pipe never waits for the epilogue.
// The kernel reads only the scratch planes and the basis, so writing the cache in place is safe.
//
// Every wait on an mbarrier is bounded in time: a wait that runs out sets a bit in the status
// word, raises a CTA-wide abort flag that ends every other role's loop, the producer lets its
// copies in flight land, the two CTAs meet at a cluster barrier, tensor memory is freed and
// the kernel returns.
#include <cuda.h>

#include <algorithm>
#include <cstdio>
#include <vector>

#include "gemm.cuh"

namespace freqkv {
namespace {

constexpr int BM = 128;        // folded output rows per CTA and tile (the cluster's tile has 2 x 128); 256 columns: K | V
constexpr int BK = 64;         // contraction slice per stage (folded rows)
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK * 2;               // 16 KB: 128 rows x 64 bf16, 128 B per row
constexpr int B_CHUNK_BYTES = BK * 128;            // 8 KB: 64 rows x 64 channels
constexpr int B_BYTES = 2 * B_CHUNK_BYTES;         // 16 KB: this CTA's 128 of the 256 columns
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;     // 32 KB per CTA
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int NUM_THREADS = 320;                   // 10 warps
constexpr int EPI_WARPS = 8;
constexpr unsigned long long LANDING_NS = 1000000ull;        // 1 ms: far longer than any copy in flight needs

constexpr uint32_t ERR_FULL_WAIT = 1u, ERR_EMPTY_WAIT = 2u, ERR_ACC_FULL_WAIT = 4u, ERR_ACC_EMPTY_WAIT = 8u;

struct RaggedSeq {
    int32_t tile0, pair0, n_keep, rows_half, basis_rows_pad, k_steps, m_pairs, pad;
};

struct GemmParams {
    int32_t n_keep;             // L
    int32_t rows_half;          // ceil(L / 2): folded output rows
    int32_t basis_rows_pad;     // row offset of the Po plane inside the basis tensor map
    int32_t pair0, pair_count;  // (batch, layer, kv_head) triples covered by this launch
    int32_t m_pairs, k_steps;   // tiles of 256 folded rows per (batch, layer, kv_head); slices per phase
    // two-level fold only: ceil(L / 4) = twice-folded output rows, N / 4 = rows of uu (and of uv), slices of
    // the two short phases
    int32_t rows_quarter, n_quarter, k_steps_short;
    int32_t sink;
    int32_t mirror_sign;        // +1: y[L-1-m] = s - d;  -1: y[L-1-m] = d - s (a retained band that starts at an odd component)
    // power-spectrum mode only: per tensor [layers][kv_heads][n_in] sums, the weight of one squared value
    float* spectrum[2];
    float spectrum_scale;
    int32_t n_in;
    int32_t* status;
    unsigned long long wait_limit_ns;  // bound of every mbarrier wait
    // ragged mode only: per-sequence shapes (sorted by decreasing work, tile0 = running sum of tiles,
    // one entry past the end holds the total) and two tensor maps per sequence (basis, folded inputs)
    const RaggedSeq* seqs;
    const CUtensorMap* seq_maps;
    int32_t n_seqs;
};

// What one tile (256 folded output rows x K|V of one (batch, layer, kv_head)) works on.
struct TileCtx {
    const CUtensorMap* map_p;   // basis
    const CUtensorMap* map_x;   // folded inputs
    int32_t pair;               // (batch, layer, kv_head) triple inside the cache view
    int32_t pair_local;         // ... inside the scratch planes its tensor map covers
    int32_t m_tile;             // which 256 folded rows
    int32_t n_keep, rows_half, basis_rows_pad, k_steps;
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

// Address of the same shared-memory location in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Acquire at cluster scope: some of the arrivals these waits observe come from the peer CTA.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Wait for the phase with the given parity to complete.  Gives up when another role has raised
// the abort flag or after `limit_ns`; in the second case it records `err_bit` and raises the
// flag itself.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          uint32_t err_bit, unsigned long long limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) {
            atomicOr(status, (int32_t)err_bit);
            *abort_flag = 1;
            __threadfence_block();
            return false;
        }
    }
}

// TMA loads of a CTA pair: the data lands in this CTA's shared memory, the bytes are counted on
// the barrier `cluster_bar` of the leader CTA.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int32_t c0,
                                            int32_t c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int32_t c0,
                                            int32_t c1, int32_t c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int32_t c0,
                                            int32_t c1, int32_t c2, int32_t c3, int32_t c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
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

// Instruction descriptor, kind::f16: D fp32, A and B bf16, A K-major, B MN-major, M = 256 (128 rows
// in each CTA of the pair), N = 256.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((256u >> 3) << 17) |
                           ((256u >> 4) << 24);

// Issued by one thread of the leader CTA; both CTAs' tensor cores run it, each on its 128 rows of A
// and D, with B read from the shared memory of both.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(IDESC), "r"(accumulate)
        : "memory");
}

// When every MMA issued so far has finished, arrive on the barrier at this offset in BOTH CTAs.
__device__ __forceinline__ void umma_commit_both(uint32_t bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3)
        : "memory");
}

// 32 lanes x 32 consecutive columns of tensor memory into registers r[OFF .. OFF+31].
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

// 32 lanes x 16 consecutive columns.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// ---- fold: U = X + reversed X, V = X - reversed X, one 16-byte vector (8 channels) per item ----

__device__ __forceinline__ void fold8(const uint4& a, const uint4& b, uint4* u, uint4* v)
{
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    uint32_t uw[4], vw[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float a0 = __uint_as_float(aw[i] << 16), a1 = __uint_as_float(aw[i] & 0xffff0000u);
        const float b0 = __uint_as_float(bw[i] << 16), b1 = __uint_as_float(bw[i] & 0xffff0000u);
        uw[i] = pack_bf16(a0 + b0, a1 + b1);
        vw[i] = pack_bf16(a0 - b0, a1 - b1);
    }
    *u = make_uint4(uw[0], uw[1], uw[2], uw[3]);
    *v = make_uint4(vw[0], vw[1], vw[2], vw[3]);
}

// One fold job: the non-sink rows of `pair_count` (batch, layer, kv_head) triples starting at
// pair0, K and V, into the planes ((pair_local * 2 + tensor) * 2 + (0 = U, 1 = V)) of `dst`, each
// n_half rows x 128 channels (16 vectors of 16 bytes per row).
struct FoldJob {
    int32_t pair0, pair_count, n_in, n_half, sink;
    uint4* dst;
};

// Block (x, y): matrix x of the job (pair_local * 2 + tensor), y-th share of its n_half * 16 vectors.
// The matrix arithmetic is done once per thread; each thread then folds four vectors per round,
// all eight loads first.  Reads and writes are streaming (each byte is touched once).
__global__ void __launch_bounds__(256) fold_kernel(const CacheView view, const FoldJob job)
{
    const uint32_t pt = blockIdx.x;
    const char* x = static_cast<const char*>(tensor_base(view, pt & 1)) +
                    (matrix_offset(view, job.pair0 + (int32_t)(pt >> 1)) + (int64_t)job.sink * view.stride_token) * 2;
    const int64_t row_bytes = view.stride_token * 2;
    const uint32_t total = (uint32_t)job.n_half * 16u;
    uint4* u_plane = job.dst + (int64_t)pt * 2 * total;
    // a block works on chunks of 1024 consecutive vectors (64 rows and their 64 mirror rows)
    for (uint32_t c0 = blockIdx.y * 1024u; c0 < total; c0 += gridDim.y * 1024u) {
        uint4 a[4], b[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t i = c0 + j * 256u + threadIdx.x;
            if (i < total) {
                const int32_t n = (int32_t)(i >> 4), nr = job.n_in - 1 - n;
                a[j] = __ldcs(reinterpret_cast<const uint4*>(x + n * row_bytes) + (i & 15u));
                b[j] = __ldcs(reinterpret_cast<const uint4*>(x + nr * row_bytes) + (i & 15u));
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t i = c0 + j * 256u + threadIdx.x;
            if (i < total) {
                const int32_t n = (int32_t)(i >> 4);
                uint4 u, v;
                fold8(a[j], b[j], &u, &v);
                if (job.n_in - 1 - n == n) {  // middle row of an odd-length signal: u = x, v = 0
                    u = a[j];
                    v = make_uint4(0u, 0u, 0u, 0u);
                }
                __stcs(u_plane + i, u);
                __stcs(u_plane + total + i, v);
            }
        }
    }
}

// Two levels of folding at once (n_in a multiple of 4; see basis.cu): with N' = n_in / 2 and n < N' / 2 the
// four rows n, N-1-n, N'-1-n and N'+n give u_n, u_{N'-1-n}, v_n, v_{N'-1-n}, and from the two u's
// uu_n = u_n + u_{N'-1-n}, uv_n = u_n - u_{N'-1-n} (sums in fp32, rounded once).  Plane 0 of a matrix holds uu
// (rows 0 .. N'/2 - 1) followed by uv (rows N'/2 .. N' - 1), plane 1 holds v: the same bytes as one level.
__device__ __forceinline__ void fold8x2(const uint4& a, const uint4& b, const uint4& c, const uint4& d, uint4* uu, uint4* uv,
                                        uint4* v1, uint4* v2)
{
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w}, cw[4] = {c.x, c.y, c.z, c.w},
                   dw[4] = {d.x, d.y, d.z, d.w};
    uint32_t o[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float a0 = __uint_as_float(aw[i] << 16), a1 = __uint_as_float(aw[i] & 0xffff0000u);
        const float b0 = __uint_as_float(bw[i] << 16), b1 = __uint_as_float(bw[i] & 0xffff0000u);
        const float c0 = __uint_as_float(cw[i] << 16), c1 = __uint_as_float(cw[i] & 0xffff0000u);
        const float d0 = __uint_as_float(dw[i] << 16), d1 = __uint_as_float(dw[i] & 0xffff0000u);
        const float p0 = a0 + b0, p1 = a1 + b1, q0 = c0 + d0, q1 = c1 + d1;  // u_n, u_{N'-1-n}
        o[0][i] = pack_bf16(p0 + q0, p1 + q1);
        o[1][i] = pack_bf16(p0 - q0, p1 - q1);
        o[2][i] = pack_bf16(a0 - b0, a1 - b1);
        o[3][i] = pack_bf16(c0 - d0, c1 - d1);
    }
    *uu = make_uint4(o[0][0], o[0][1], o[0][2], o[0][3]);
    *uv = make_uint4(o[1][0], o[1][1], o[1][2], o[1][3]);
    *v1 = make_uint4(o[2][0], o[2][1], o[2][2], o[2][3]);
    *v2 = make_uint4(o[3][0], o[3][1], o[3][2], o[3][3]);
}

// Block (x, y) as in fold_kernel; job.n_half = N' rows per plane; a thread folds two vectors per round.
__global__ void __launch_bounds__(256) fold2_kernel(const CacheView view, const FoldJob job)
{
    const uint32_t pt = blockIdx.x;
    const char* x = static_cast<const char*>(tensor_base(view, pt & 1)) +
                    (matrix_offset(view, job.pair0 + (int32_t)(pt >> 1)) + (int64_t)job.sink * view.stride_token) * 2;
    const int64_t row_bytes = view.stride_token * 2;
    const int32_t n_quarter = job.n_half / 2;
    const uint32_t total = (uint32_t)n_quarter * 16u;                // vectors of uu (= of uv)
    uint4* plane0 = job.dst + (int64_t)pt * 2 * ((int64_t)job.n_half * 16);
    uint4* plane1 = plane0 + (int64_t)job.n_half * 16;
    for (uint32_t c0 = blockIdx.y * 512u; c0 < total; c0 += gridDim.y * 512u) {
        uint4 a[2], b[2], c[2], d[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const uint32_t i = c0 + j * 256u + threadIdx.x;
            if (i < total) {
                const int32_t n = (int32_t)(i >> 4);
                a[j] = __ldcs(reinterpret_cast<const uint4*>(x + n * row_bytes) + (i & 15u));
                b[j] = __ldcs(reinterpret_cast<const uint4*>(x + (job.n_in - 1 - n) * row_bytes) + (i & 15u));
                c[j] = __ldcs(reinterpret_cast<const uint4*>(x + (job.n_half - 1 - n) * row_bytes) + (i & 15u));
                d[j] = __ldcs(reinterpret_cast<const uint4*>(x + (job.n_half + n) * row_bytes) + (i & 15u));
            }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const uint32_t i = c0 + j * 256u + threadIdx.x;
            if (i < total) {
                const int32_t n = (int32_t)(i >> 4);
                uint4 uu, uv, v1, v2;
                fold8x2(a[j], b[j], c[j], d[j], &uu, &uv, &v1, &v2);
                __stcs(plane0 + i, uu);
                __stcs(plane0 + total + i, uv);
                __stcs(plane1 + i, v1);
                __stcs(plane1 + (int64_t)(job.n_half - 1 - n) * 16 + (i & 15u), v2);
            }
        }
    }
}

// The same for a ragged batch in one launch: every sequence has the same number of matrices, so
// block x belongs to job x / mats_per_seq.
__global__ void __launch_bounds__(256) fold_ragged_kernel(const CacheView view, const FoldJob* jobs, int32_t mats_per_seq)
{
    const FoldJob job = jobs[blockIdx.x / mats_per_seq];
    const uint32_t pt = blockIdx.x % mats_per_seq;
    const char* x = static_cast<const char*>(tensor_base(view, pt & 1)) +
                    (matrix_offset(view, job.pair0 + (int32_t)(pt >> 1)) + (int64_t)job.sink * view.stride_token) * 2;
    const int64_t row_bytes = view.stride_token * 2;
    const uint32_t total = (uint32_t)job.n_half * 16u;
    uint4* u_plane = job.dst + (int64_t)pt * 2 * total;
    for (uint32_t c0 = blockIdx.y * 1024u; c0 < total; c0 += gridDim.y * 1024u) {
        uint4 a[4], b[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t i = c0 + j * 256u + threadIdx.x;
            if (i < total) {
                const int32_t n = (int32_t)(i >> 4), nr = job.n_in - 1 - n;
                a[j] = __ldcs(reinterpret_cast<const uint4*>(x + n * row_bytes) + (i & 15u));
                b[j] = __ldcs(reinterpret_cast<const uint4*>(x + nr * row_bytes) + (i & 15u));
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t i = c0 + j * 256u + threadIdx.x;
            if (i < total) {
                const int32_t n = (int32_t)(i >> 4);
                uint4 u, v;
                fold8(a[j], b[j], &u, &v);
                if (job.n_in - 1 - n == n) {
                    u = a[j];
                    v = make_uint4(0u, 0u, 0u, 0u);
                }
                __stcs(u_plane + i, u);
                __stcs(u_plane + total + i, v);
            }
        }
    }
}

// MODE_FOLD: the compression above.
// MODE_RAGGED: MODE_FOLD over sequences of different lengths in one launch: a tile looks up its
//   sequence (shapes, basis and folded-input tensor maps) in a table built on the host.
// MODE_SPECTRUM: the basis holds the even and the odd rows of the plain N-point DCT-II instead of
//   Pe and Po, so S and D are the components z_2m and z_2m+1 themselves; the epilogue squares them,
//   sums over the 128 channels of its tensor and adds the sum to the power spectrum of its
//   (layer, kv head).  Nothing is written to the cache.
// MODE_DIRECT: for at most 256 kept rows (small retaining ratios) the fold pass would cost more
//   than it saves: the basis is the plain L x N matrix P, the input slices come straight from the
//   cache (map_x = K tensor, map_v = V tensor, 5-D maps over the non-sink rows), there is one
//   accumulator and one tile per (batch, layer, kv_head).  The tile's rows are stored only after
//   every slice of its matrices has been read, so writing in place is safe here too.
// MODE_FOLD2: two levels of the symmetry fold (n_in a multiple of 4, n_keep even).  A tile is 256
//   twice-folded rows m < ceil(L/4) and runs four phases: a = Pee uu and b = Peo uv (N/4 deep), then
//   d = Po v for rows m and d' = Po v for the mirrored rows L/2-1-m (N/2 deep), alternating between the
//   two halves of tensor memory.  The epilogue parks a, turns it with b into the pair s = a + b,
//   s' = a - b (kept as two bf16 in the register a occupied) and stores y_m = s + d, y_{L-1-m} = s - d,
//   y_{L/2-1-m} = s' + d', y_{L/2+m} = s' - d': three quarters of the multiply-adds of MODE_FOLD.
constexpr int MODE_FOLD = 0, MODE_SPECTRUM = 1, MODE_DIRECT = 2, MODE_RAGGED = 3, MODE_FOLD2 = 4;

// Ragged mode: a role walks its tiles in increasing order, so the sequence a tile belongs to is
// found by moving a cursor forward; the table is read only when a tile crosses into a new sequence.
struct SeqCursor {
    int32_t idx = -1, end_tile = 0;
    RaggedSeq s;
};

template <int MODE>
__device__ __forceinline__ TileCtx tile_ctx(const GemmParams& prm, int32_t tile, const CUtensorMap* map_p, const CUtensorMap* map_x,
                                            SeqCursor& cur)
{
    TileCtx t;
    if constexpr (MODE == MODE_RAGGED) {
        while (tile >= cur.end_tile) {
            ++cur.idx;
            cur.s = prm.seqs[cur.idx];
            cur.end_tile = __ldg(&prm.seqs[cur.idx + 1].tile0);
        }
        const RaggedSeq& s = cur.s;
        const int32_t lo = cur.idx;
        const int32_t local = tile - s.tile0;
        t.map_p = prm.seq_maps + 2 * lo;
        t.map_x = prm.seq_maps + 2 * lo + 1;
        t.pair_local = local / s.m_pairs;
        t.m_tile = local % s.m_pairs;
        t.pair = s.pair0 + t.pair_local;
        t.n_keep = s.n_keep;
        t.rows_half = s.rows_half;
        t.basis_rows_pad = s.basis_rows_pad;
        t.k_steps = s.k_steps;
    } else {
        t.map_p = map_p;
        t.map_x = map_x;
        t.pair_local = tile / prm.m_pairs;
        t.m_tile = tile % prm.m_pairs;
        t.pair = prm.pair0 + t.pair_local;
        t.n_keep = prm.n_keep;
        t.rows_half = prm.rows_half;
        t.basis_rows_pad = prm.basis_rows_pad;
        t.k_steps = prm.k_steps;
    }
    return t;
}

template <int MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
freqkv_gemm_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_x,
                   const __grid_constant__ CUtensorMap map_v, const CacheView view, const GemmParams prm)
{
    constexpr bool SPECTRUM = MODE == MODE_SPECTRUM;
    constexpr bool FOLD2 = MODE == MODE_FOLD2;
    constexpr int PHASES = MODE == MODE_DIRECT ? 1 : FOLD2 ? 4 : 2;
    constexpr int USES = FOLD2 ? 2 : 1;  // times a tile fills each half of tensor memory
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte swizzle atoms need 1024-byte alignment
    uint8_t* aligned = smem_raw + (base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(aligned + STAGES * STAGE_BYTES);
    const uint32_t bar0 = base + STAGES * STAGE_BYTES;
    // barrier slots (same offsets in both CTAs): full[0..S) -- used in the leader only --,
    // empty[S..2S), then s_full, s_empty, d_full, d_empty (the two *_empty used in the leader only)
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto acc_full_bar = [&](int eo) { return bar0 + 8u * (2 * STAGES + 2 * eo); };
    auto acc_empty_bar = [&](int eo) { return bar0 + 8u * (2 * STAGES + 2 * eo + 1); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_rank();  // 0 = leader of the pair
    const int32_t cluster = blockIdx.x / 2, n_clusters = gridDim.x / 2;
    // tiles of 256 folded rows x 256 columns
    const int32_t total_tiles = MODE == MODE_RAGGED ? prm.seqs[prm.n_seqs].tile0 : prm.pair_count * prm.m_pairs;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);   // the leader's producer arrives; both producers' bytes are counted
            mbar_init(empty_bar(s), 1);  // one multicast commit
        }
        for (int eo = 0; eo < 2; ++eo) {
            mbar_init(acc_full_bar(eo), 1);               // one multicast commit
            mbar_init(acc_empty_bar(eo), 2 * EPI_WARPS);  // the epilogue warps of both CTAs
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {  // tensor memory of the pair: all 512 columns in each CTA (S in 0..255, D in 256..511)
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            uint32_t it = 0;  // global slice counter: stage = it % STAGES, phase = it / STAGES
            bool alive = true;
            SeqCursor cursor;
            for (int32_t tile = cluster; tile < total_tiles && alive; tile += n_clusters) {
                const TileCtx tc = tile_ctx<MODE>(prm, tile, &map_p, &map_x, cursor);
                const int32_t pair_local = tc.pair_local;
                const int32_t m0 = (tc.m_tile * 2 + (int32_t)rank) * BM;
                const int32_t pair = tc.pair;  // direct mode: coordinates inside the cache tensor
                const int32_t head = pair % view.kv_heads, layer = (pair / view.kv_heads) % view.layers,
                              seq = pair / (view.kv_heads * view.layers);
                for (int eo = 0; eo < PHASES && alive; ++eo) {
                    // rank 0: K channels, rank 1: V.  Two-level fold: phases 0, 1 read uu and uv (both in plane 0,
                    // uv n_quarter rows down), phases 2, 3 read v (plane 1)
                    const int32_t plane = (pair_local * 2 + (int32_t)rank) * 2 + (FOLD2 ? eo >> 1 : eo);
                    const int32_t row0 = (FOLD2 && eo == 1) ? prm.n_quarter : 0;
                    const int32_t phase_steps = (FOLD2 && eo < 2) ? prm.k_steps_short : tc.k_steps;
                    for (int32_t ks = 0; ks < phase_steps; ++ks, ++it) {
                        const int s = it % STAGES;
                        if (it >= STAGES &&
                            !mbar_wait(empty_bar(s), ((it / STAGES) - 1) & 1, abort_flag, prm.status, ERR_EMPTY_WAIT, prm.wait_limit_ns)) {
                            alive = false;
                            break;
                        }
                        const uint32_t stage = base + s * STAGE_BYTES;
                        const uint32_t leader_full = cluster_addr(full_bar(s), 0);
                        if (rank == 0) mbar_expect_tx(full_bar(s), 2 * STAGE_BYTES);
                        const int32_t k0 = ks * BK;
                        tma_load_2d(stage, tc.map_p, leader_full, k0, eo * tc.basis_rows_pad + m0);
                        if constexpr (MODE == MODE_DIRECT) {
                            const CUtensorMap* cache = rank ? &map_v : &map_x;
                            tma_load_5d(stage + A_BYTES, cache, leader_full, 0, k0, head, layer, seq);
                            tma_load_5d(stage + A_BYTES + B_CHUNK_BYTES, cache, leader_full, 64, k0, head, layer, seq);
                        } else {
                            tma_load_3d(stage + A_BYTES, tc.map_x, leader_full, 0, row0 + k0, plane);
                            tma_load_3d(stage + A_BYTES + B_CHUNK_BYTES, tc.map_x, leader_full, 64, row0 + k0, plane);
                        }
                    }
                }
            }
            if (*abort_flag) {  // let the copies in flight land before this CTA's shared memory goes away
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < LANDING_NS) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, tile_no = 0;
            bool alive = true;
            SeqCursor cursor;
            for (int32_t tile = cluster; tile < total_tiles && alive; tile += n_clusters, ++tile_no) {
                const int32_t tile_steps = tile_ctx<MODE>(prm, tile, &map_p, &map_x, cursor).k_steps;
                for (int eo = 0; eo < PHASES && alive; ++eo) {
                    const int acc = eo & 1;                                   // half of tensor memory
                    const uint32_t use = tile_no * USES + (uint32_t)(eo >> 1);  // how often that half was filled before
                    const int32_t k_steps = (FOLD2 && eo < 2) ? prm.k_steps_short : tile_steps;
                    if (use > 0) {  // both CTAs' epilogues must have read what this half held last
                        if (!mbar_wait(acc_empty_bar(acc), (use - 1) & 1, abort_flag, prm.status, ERR_ACC_EMPTY_WAIT, prm.wait_limit_ns)) {
                            alive = false;
                            break;
                        }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    }
                    for (int32_t ks = 0; ks < k_steps; ++ks, ++it) {
                        const int s = it % STAGES;
                        if (!mbar_wait(full_bar(s), (it / STAGES) & 1, abort_flag, prm.status, ERR_FULL_WAIT, prm.wait_limit_ns)) {
                            alive = false;
                            break;
                        }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t a0 = base + s * STAGE_BYTES, b0 = a0 + A_BYTES;
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk) {
                            // A: 128 rows per CTA, 8-row groups 1 KB apart; 16 k-elements = 32 bytes inside the swizzled row
                            const uint64_t ad = smem_desc(a0 + kk * 32, 16, 1024);
                            // B: per CTA 2 chunks of 64 channels 8 KB apart (leading offset), 8-row groups 1 KB apart
                            const uint64_t bd = smem_desc(b0 + kk * 2048, B_CHUNK_BYTES, 1024);
                            umma_bf16(tmem_base + acc * 256, ad, bd, (ks | kk) != 0);
                        }
                        umma_commit_both(empty_bar(s));  // frees the stage in both CTAs when these MMAs have read it
                    }
                    if (alive) umma_commit_both(acc_full_bar(acc));
                }
            }
        }
    } else {
        // ---------------- epilogue (both CTAs, each on its own 128 rows) ----------------
        const int ew = warp - 2, quarter = warp % 4, tensor = ew / 4;  // tensor: 0 = K columns, 1 = V columns
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + tensor * 128;
        const uint32_t leader_s_empty = cluster_addr(acc_empty_bar(0), 0), leader_d_empty = cluster_addr(acc_empty_bar(1), 0);
        uint32_t tile_no = 0;
        SeqCursor cursor;
        if constexpr (MODE == MODE_DIRECT) {
            for (int32_t tile = cluster; tile < total_tiles; tile += n_clusters, ++tile_no) {
                if (!mbar_wait(acc_full_bar(0), tile_no & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT, prm.wait_limit_ns)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int32_t m = (int32_t)rank * BM + quarter * 32 + lane;
                __nv_bfloat16* mat = static_cast<__nv_bfloat16*>(tensor_base(view, tensor)) +
                                     matrix_offset(view, prm.pair0 + tile) + (int64_t)prm.sink * view.stride_token;
                uint4* out = reinterpret_cast<uint4*>(mat + (int64_t)m * view.stride_token);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t y[16];
                    tmem_ld16(lane_addr + c * 16, y);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (m < prm.n_keep) {
                        uint32_t p[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) p[j] = pack_bf16(__uint_as_float(y[2 * j]), __uint_as_float(y[2 * j + 1]));
                        out[2 * c] = make_uint4(p[0], p[1], p[2], p[3]);
                        out[2 * c + 1] = make_uint4(p[4], p[5], p[6], p[7]);
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(leader_s_empty);
            }
        } else if constexpr (SPECTRUM) {
            for (int32_t tile = cluster; tile < total_tiles; tile += n_clusters, ++tile_no) {
                const int32_t pair = prm.pair0 + tile / prm.m_pairs;
                const int32_t head = pair % view.kv_heads, layer = (pair / view.kv_heads) % view.layers;
                const int32_t m = ((tile % prm.m_pairs) * 2 + (int32_t)rank) * BM + quarter * 32 + lane;
                bool alive = true;
                for (int eo = 0; eo < 2; ++eo) {
                    if (!mbar_wait(acc_full_bar(eo), tile_no & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT, prm.wait_limit_ns)) {
                        alive = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    float sum = 0.f;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t r[32];
                        tmem_ld32<0>(lane_addr + eo * 256 + c * 32, r);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int j = 0; j < 32; ++j) sum = fmaf(__uint_as_float(r[j]), __uint_as_float(r[j]), sum);
                    }
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(eo ? leader_d_empty : leader_s_empty);
                    const int32_t t = 2 * m + eo;  // S holds the even components, D the odd ones
                    if (t < prm.n_in && prm.spectrum[tensor])
                        atomicAdd(prm.spectrum[tensor] + ((int64_t)layer * view.kv_heads + head) * prm.n_in + t,
                                  sum * prm.spectrum_scale);
                }
                if (!alive) break;
            }
        } else if constexpr (FOLD2) {
            const uint32_t leader_empty[2] = {leader_s_empty, leader_d_empty};
            auto release = [&](int acc) {
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(leader_empty[acc]);
            };
            for (int32_t tile = cluster; tile < total_tiles; tile += n_clusters, ++tile_no) {
                const uint32_t use = 2 * tile_no;
                // a = Pee uu: park this thread's row (128 columns) in registers
                if (!mbar_wait(acc_full_bar(0), use & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT, prm.wait_limit_ns)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                uint32_t s[128];
                tmem_ld32<0>(lane_addr + 0, s);
                tmem_ld32<32>(lane_addr + 32, s);
                tmem_ld32<64>(lane_addr + 64, s);
                tmem_ld32<96>(lane_addr + 96, s);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                release(0);
                // b = Peo uv: s = a + b (low half of the register) and s' = a - b (high half), both bf16
                if (!mbar_wait(acc_full_bar(1), use & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT, prm.wait_limit_ns)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t b[16];
                    tmem_ld16(lane_addr + 256 + c * 16, b);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float av = __uint_as_float(s[c * 16 + j]), bv = __uint_as_float(b[j]);
                        s[c * 16 + j] = pack_bf16(av + bv, av - bv);
                    }
                }
                release(1);

                const TileCtx tc = tile_ctx<MODE>(prm, tile, &map_p, &map_x, cursor);
                const int32_t m = (tc.m_tile * 2 + (int32_t)rank) * BM + quarter * 32 + lane;
                const int32_t mh = tc.rows_half - 1 - m;  // the row whose even part is s'
                const bool row_ok = m < prm.rows_quarter;
                __nv_bfloat16* mat = static_cast<__nv_bfloat16*>(tensor_base(view, tensor)) +
                                     matrix_offset(view, tc.pair) + (int64_t)prm.sink * view.stride_token;
                bool alive = true;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    // d = Po v of rows m (half 0) or of the mirrored rows L/2-1-m (half 1): rows r and L-1-r
                    if (!mbar_wait(acc_full_bar(half), (use + 1) & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT, prm.wait_limit_ns)) {
                        alive = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const int32_t r = half ? mh : m;
                    const bool store = row_ok && !(half && mh == m);  // the middle row of an odd L/2 comes out of half 0
                    uint4* out_p = reinterpret_cast<uint4*>(mat + (int64_t)r * view.stride_token);
                    uint4* out_m = reinterpret_cast<uint4*>(mat + (int64_t)(tc.n_keep - 1 - r) * view.stride_token);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint32_t d[16];
                        tmem_ld16(lane_addr + half * 256 + c * 16, d);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (store) {
                            uint32_t p[8], q[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const uint32_t w0 = s[c * 16 + 2 * j], w1 = s[c * 16 + 2 * j + 1];
                                const float s0 = __uint_as_float(half ? w0 & 0xffff0000u : w0 << 16);
                                const float s1 = __uint_as_float(half ? w1 & 0xffff0000u : w1 << 16);
                                const float d0 = __uint_as_float(d[2 * j]), d1 = __uint_as_float(d[2 * j + 1]);
                                p[j] = pack_bf16(s0 + d0, s1 + d1);
                                q[j] = pack_bf16(s0 - d0, s1 - d1);
                            }
                            out_p[2 * c] = make_uint4(p[0], p[1], p[2], p[3]);
                            out_p[2 * c + 1] = make_uint4(p[4], p[5], p[6], p[7]);
                            out_m[2 * c] = make_uint4(q[0], q[1], q[2], q[3]);
                            out_m[2 * c + 1] = make_uint4(q[4], q[5], q[6], q[7]);
                        }
                    }
                    release(half);
                }
                if (!alive) break;
            }
        } else
        for (int32_t tile = cluster; tile < total_tiles; tile += n_clusters, ++tile_no) {
            // S = Pe U: park this thread's row (128 columns) in registers, release that half
            if (!mbar_wait(acc_full_bar(0), tile_no & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT, prm.wait_limit_ns)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t s[128];
            tmem_ld32<0>(lane_addr + 0, s);
            tmem_ld32<32>(lane_addr + 32, s);
            tmem_ld32<64>(lane_addr + 64, s);
            tmem_ld32<96>(lane_addr + 96, s);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_s_empty);

            // D = Po V: combine and store rows m and L-1-m
            if (!mbar_wait(acc_full_bar(1), tile_no & 1, abort_flag, prm.status, ERR_ACC_FULL_WAIT, prm.wait_limit_ns)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const TileCtx tc = tile_ctx<MODE>(prm, tile, &map_p, &map_x, cursor);
            const int32_t m = (tc.m_tile * 2 + (int32_t)rank) * BM + quarter * 32 + lane;
            const int32_t mr = tc.n_keep - 1 - m;
            const bool row_ok = m < tc.rows_half;
            const float sgn = (float)prm.mirror_sign;
            __nv_bfloat16* mat = static_cast<__nv_bfloat16*>(tensor_base(view, tensor)) +
                                 matrix_offset(view, tc.pair) + (int64_t)prm.sink * view.stride_token;
            uint4* out_p = reinterpret_cast<uint4*>(mat + (int64_t)m * view.stride_token);
            uint4* out_m = reinterpret_cast<uint4*>(mat + (int64_t)mr * view.stride_token);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t d[16];
                tmem_ld16(lane_addr + 256 + c * 16, d);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row_ok) {
                    uint32_t p[8], q[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float s0 = __uint_as_float(s[c * 16 + 2 * j]), s1 = __uint_as_float(s[c * 16 + 2 * j + 1]);
                        const float d0 = __uint_as_float(d[2 * j]), d1 = __uint_as_float(d[2 * j + 1]);
                        p[j] = pack_bf16(s0 + d0, s1 + d1);
                        q[j] = pack_bf16(sgn * (s0 - d0), sgn * (s1 - d1));
                    }
                    out_p[2 * c] = make_uint4(p[0], p[1], p[2], p[3]);
                    out_p[2 * c + 1] = make_uint4(p[4], p[5], p[6], p[7]);
                    if (mr != m) {
                        out_m[2 * c] = make_uint4(q[0], q[1], q[2], q[3]);
                        out_m[2 * c + 1] = make_uint4(q[4], q[5], q[6], q[7]);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_d_empty);
        }
    }

    // Neither CTA may leave (its barriers and tensor memory are used by the other) before both are done.
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
    }
}

// One CTA, one thread: a wait of the kernels above on an mbarrier nothing ever arrives on, so
// that the give-up path (status bit, abort flag, return) can be exercised without stalling a
// real launch.  No TMA, no tensor memory, no cluster.
__global__ void bounded_wait_probe_kernel(int32_t* status, unsigned long long limit_ns)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0, &abort_flag, status, ERR_FULL_WAIT, limit_ns);
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

// Pe stacked over Po: a 2-D tensor of 2 * fold_rows_pad rows x fold_ld columns.
bool encode_basis_map(CUtensorMap* map, const Basis& basis)
{
    const cuuint64_t dims[2] = {(cuuint64_t)basis.fold_ld, (cuuint64_t)2 * basis.fold_rows_pad};
    const cuuint64_t strides[1] = {(cuuint64_t)basis.fold_ld * 2};
    const cuuint32_t box[2] = {BK, BM};
    const cuuint32_t elem[2] = {1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, basis.fold, dims, strides, box, elem,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The four planes of the twice-folded basis stacked: 4 * fold2_rows_pad rows x fold_ld columns.
bool encode_basis2_map(CUtensorMap* map, const Basis& basis)
{
    const cuuint64_t dims[2] = {(cuuint64_t)basis.fold_ld, (cuuint64_t)4 * basis.fold2_rows_pad};
    const cuuint64_t strides[1] = {(cuuint64_t)basis.fold_ld * 2};
    const cuuint32_t box[2] = {BK, BM};
    const cuuint32_t elem[2] = {1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, basis.fold2, dims, strides, box, elem,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The scratch planes as a 3-D tensor (channel, folded row, plane); rows past n_half read as zero.
bool encode_scratch_map(CUtensorMap* map, void* scratch, int32_t n_half, int32_t planes)
{
    const cuuint64_t dims[3] = {128, (cuuint64_t)n_half, (cuuint64_t)planes};
    const cuuint64_t strides[2] = {256, (cuuint64_t)n_half * 256};
    const cuuint32_t box[3] = {64, BK, 1};
    const cuuint32_t elem[3] = {1, 1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, scratch, dims, strides, box, elem,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t kRaggedScratchLimit = size_t(64) << 30;  // a ragged batch is folded whole: beyond this it goes sequence by sequence
constexpr size_t kFoldBufferBytes = size_t(2304) << 20;  // scratch for the folded inputs: a 7B-shaped cache of 4096 tokens fits in one pass

}  // namespace

bool gemm_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep)
{
    return dtype == FREQKV_BF16 && head_dim == 128 && n_in >= 1 && n_keep >= 1 && n_keep <= n_in;
}

// Everything a launch needs that is not a stream operation: kernel attributes, the count of
// resident CTA pairs, the scratch buffer for `pairs` (batch, layer, kv_head) triples of this basis
// (pairs = 0: none, the direct mode reads the cache itself).
// launch_gemm calls it itself; a caller that must not allocate later (stream capture) calls it first.
cudaError_t gemm_prepare(GemmState* state, int32_t pairs, const Basis& basis, int sm_count)
{
    state->last_error = nullptr;
    if (!encode_fn()) {
        state->last_error = "cuTensorMapEncodeTiled is not available from this driver";
        return cudaErrorNotSupported;
    }
    if (!state->attr_set) {
        cudaError_t e = cudaFuncSetAttribute(freqkv_gemm_kernel<MODE_FOLD>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(freqkv_gemm_kernel<MODE_SPECTRUM>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(freqkv_gemm_kernel<MODE_DIRECT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(freqkv_gemm_kernel<MODE_RAGGED>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(freqkv_gemm_kernel<MODE_FOLD2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) {
            state->last_error = "cudaFuncSetAttribute(max dynamic shared memory)";
            return e;
        }
        // how many CTA pairs the device can hold at once (one CTA per SM; SMs pair up inside a GPC)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * (sm_count / 2)));
        cfg.blockDim = dim3(NUM_THREADS);
        cfg.dynamicSmemBytes = SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        const cudaError_t q = cudaOccupancyMaxActiveClusters(&n, freqkv_gemm_kernel<MODE_FOLD>, &cfg);
        if (q != cudaSuccess || n < 1) {
            state->last_error = "cudaOccupancyMaxActiveClusters: no CTA pair fits on this device";
            return q != cudaSuccess ? q : cudaErrorLaunchOutOfResources;
        }
        state->max_clusters = std::min(n, sm_count / 2);
        state->attr_set = true;
    }
    const int32_t n_half = (basis.n_in + 1) / 2;
    const size_t per_pair = (size_t)4 * n_half * 128 * 2;  // K and V, U and V planes
    const int64_t fit = std::max<int64_t>(1, (int64_t)(kFoldBufferBytes / per_pair));
    const size_t need = (size_t)std::min<int64_t>(fit, pairs) * per_pair;
    if (need > state->scratch_bytes) {
        if (state->scratch) {
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) return e;
            cudaFree(state->scratch);
            state->scratch = nullptr;
            state->scratch_bytes = 0;
        }
        const cudaError_t e = cudaMalloc(&state->scratch, need);
        if (e != cudaSuccess) {
            state->last_error = "cudaMalloc(fold scratch)";
            return e;
        }
        state->scratch_bytes = need;
    }
    return cudaSuccess;
}

cudaError_t launch_gemm(GemmState* state, const CacheView& view, const Basis& basis, int32_t sink, int32_t* status_dev,
                        int sm_count, const LaunchHooks& hooks, cudaStream_t stream, const SpectrumOut* spectrum)
{
    state->kernels_last_call = 0;
    const cudaError_t prepared = gemm_prepare(state, view.mats_per_tensor, basis, sm_count);
    if (prepared != cudaSuccess) return prepared;
    const int32_t n_half = (basis.n_in + 1) / 2, rows_half = (basis.n_keep + 1) / 2;
    // two levels of folding where the basis has them (lengths that halve twice; not for the spectrum's basis)
    const int32_t rows_quarter = (rows_half + 1) / 2;
    const bool fold2 = basis.fold2 != nullptr && !spectrum && gemm_fold_levels(basis.n_in, basis.n_keep, basis.first) == 2;
    const int32_t m_pairs = ((fold2 ? rows_quarter : rows_half) + 2 * BM - 1) / (2 * BM);  // tiles of 256 folded rows
    const int32_t pairs = view.mats_per_tensor;
    const size_t per_pair = (size_t)4 * n_half * 128 * 2;
    // One pass when the folded inputs fit the scratch buffer, else several passes of `chunk` pairs.
    const int64_t chunk = std::min<int64_t>(std::max<int64_t>(1, (int64_t)(kFoldBufferBytes / per_pair)), pairs);
    CUtensorMap map_p;
    if (!(fold2 ? encode_basis2_map(&map_p, basis) : encode_basis_map(&map_p, basis))) {
        state->last_error = "tensor map encoding rejected the basis";
        return cudaErrorInvalidValue;
    }
    for (int64_t p0 = 0; p0 < pairs; p0 += chunk) {
        FoldJob job;
        job.pair0 = (int32_t)p0;
        job.pair_count = (int32_t)std::min<int64_t>(chunk, pairs - p0);
        job.n_in = basis.n_in;
        job.n_half = n_half;
        job.sink = sink;
        job.dst = static_cast<uint4*>(state->scratch);
        if (fold2) {
            const unsigned fold_y = (unsigned)std::min<int64_t>(((int64_t)(n_half / 2) * 16 + 511) / 512, 64);
            fold2_kernel<<<dim3((unsigned)job.pair_count * 2, fold_y), 256, 0, stream>>>(view, job);
        } else {
            const unsigned fold_y = (unsigned)std::min<int64_t>(((int64_t)n_half * 16 + 1023) / 1024, 64);
            fold_kernel<<<dim3((unsigned)job.pair_count * 2, fold_y), 256, 0, stream>>>(view, job);
        }
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) {
            state->last_error = "fold_kernel launch";
            return e;
        }
        CUtensorMap map_x;
        if (!encode_scratch_map(&map_x, state->scratch, n_half, job.pair_count * 4)) {
            state->last_error = "tensor map encoding rejected the scratch planes";
            return cudaErrorInvalidValue;
        }
        GemmParams prm;
        prm.n_keep = basis.n_keep;
        prm.rows_half = rows_half;
        prm.basis_rows_pad = fold2 ? basis.fold2_rows_pad : basis.fold_rows_pad;
        prm.rows_quarter = rows_quarter;
        prm.n_quarter = n_half / 2;
        prm.k_steps_short = (n_half / 2 + BK - 1) / BK;
        prm.pair0 = job.pair0;
        prm.pair_count = job.pair_count;
        prm.m_pairs = m_pairs;
        prm.k_steps = (n_half + BK - 1) / BK;
        prm.sink = sink;
        prm.mirror_sign = (basis.first & 1) ? -1 : 1;
        prm.spectrum[0] = spectrum ? spectrum->k : nullptr;
        prm.spectrum[1] = spectrum ? spectrum->v : nullptr;
        prm.spectrum_scale = spectrum ? spectrum->scale : 0.f;
        prm.n_in = basis.n_in;
        prm.status = status_dev;
        prm.wait_limit_ns = state->wait_limit_ns;
        prm.seqs = nullptr;
        prm.seq_maps = nullptr;
        prm.n_seqs = 0;
        const int32_t tiles = job.pair_count * m_pairs;
        const int clusters = std::min<int32_t>(tiles, state->max_clusters);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * clusters));
        cfg.blockDim = dim3(NUM_THREADS);
        cfg.dynamicSmemBytes = SMEM_BYTES;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (hooks.before) hooks.before(hooks.user, stream);
        e = spectrum ? cudaLaunchKernelEx(&cfg, freqkv_gemm_kernel<MODE_SPECTRUM>, map_p, map_x, map_x, view, prm)
            : fold2  ? cudaLaunchKernelEx(&cfg, freqkv_gemm_kernel<MODE_FOLD2>, map_p, map_x, map_x, view, prm)
                     : cudaLaunchKernelEx(&cfg, freqkv_gemm_kernel<MODE_FOLD>, map_p, map_x, map_x, view, prm);
        if (hooks.after) hooks.after(hooks.user, stream);
        if (e != cudaSuccess) {
            state->last_error = "freqkv_gemm_kernel launch";
            return e;
        }
        state->kernels_last_call += 2;
    }
    return cudaSuccess;
}

// A ragged batch in two launches: one fold pass and one tensor-core pass over every sequence,
// longest first.  Everything that can fail for lack of memory happens before the first launch.
cudaError_t launch_gemm_ragged(GemmState* state, const CacheView& view, const std::vector<RaggedItem>& items_in, int32_t sink,
                               int32_t* status_dev, int sm_count, const LaunchHooks& hooks, cudaStream_t stream)
{
    state->kernels_last_call = 0;
    if (items_in.empty()) return cudaSuccess;
    const cudaError_t prepared = gemm_prepare(state, 0, items_in[0].basis, sm_count);
    if (prepared != cudaSuccess) return prepared;
    const int32_t lh = view.layers * view.kv_heads;  // (layer, kv_head) pairs per sequence
    std::vector<RaggedItem> items = items_in;
    auto work = [](const RaggedItem& it) { return (int64_t)it.basis.n_in * it.basis.n_keep; };
    std::stable_sort(items.begin(), items.end(), [&](const RaggedItem& a, const RaggedItem& b) { return work(a) > work(b); });
    const size_t n = items.size();
    // scratch: the folded planes of every sequence, back to back
    std::vector<size_t> offset(n);
    size_t total = 0;
    int32_t max_half = 0;
    for (size_t i = 0; i < n; ++i) {
        const int32_t n_half = (items[i].basis.n_in + 1) / 2;
        offset[i] = total;
        total += (size_t)lh * 4 * n_half * 256;
        max_half = std::max(max_half, n_half);
    }
    if (total > kRaggedScratchLimit) {
        state->last_error = "folded inputs of the ragged batch exceed the scratch limit";
        return cudaErrorMemoryAllocation;
    }
    if (total > state->scratch_bytes) {
        if (state->scratch) {
            const cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) return e;
            cudaFree(state->scratch);
            state->scratch = nullptr;
            state->scratch_bytes = 0;
        }
        const cudaError_t e = cudaMalloc(&state->scratch, total);
        if (e != cudaSuccess) {
            state->last_error = "cudaMalloc(fold scratch of a ragged batch)";
            return e;
        }
        state->scratch_bytes = total;
    }
    // tables: two tensor maps, one shape record and one fold job per sequence
    const size_t maps_bytes = n * 2 * sizeof(CUtensorMap), seqs_bytes = (n + 1) * sizeof(RaggedSeq), jobs_bytes = n * sizeof(FoldJob);
    const size_t meta_bytes = maps_bytes + seqs_bytes + jobs_bytes;
    if (meta_bytes > state->ragged_meta_bytes) {
        if (state->ragged_meta) {
            const cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) return e;
            cudaFree(state->ragged_meta);
            state->ragged_meta = nullptr;
            state->ragged_meta_bytes = 0;
        }
        const cudaError_t e = cudaMalloc(&state->ragged_meta, meta_bytes);
        if (e != cudaSuccess) {
            state->last_error = "cudaMalloc(tables of a ragged batch)";
            return e;
        }
        state->ragged_meta_bytes = meta_bytes;
    }
    std::vector<CUtensorMap> maps(2 * n);
    std::vector<RaggedSeq> seqs(n + 1);
    std::vector<FoldJob> jobs(n);
    int64_t tiles = 0;
    for (size_t i = 0; i < n; ++i) {
        const Basis& b = items[i].basis;
        const int32_t n_half = (b.n_in + 1) / 2, rows_half = (b.n_keep + 1) / 2;
        char* planes = static_cast<char*>(state->scratch) + offset[i];
        if (!encode_basis_map(&maps[2 * i], b) || !encode_scratch_map(&maps[2 * i + 1], planes, n_half, lh * 4)) {
            state->last_error = "tensor map encoding rejected a sequence of the ragged batch";
            return cudaErrorInvalidValue;
        }
        RaggedSeq& s = seqs[i];
        s.tile0 = (int32_t)tiles;
        s.pair0 = items[i].batch_index * lh;
        s.n_keep = b.n_keep;
        s.rows_half = rows_half;
        s.basis_rows_pad = b.fold_rows_pad;
        s.k_steps = (n_half + BK - 1) / BK;
        s.m_pairs = (rows_half + 2 * BM - 1) / (2 * BM);
        s.pad = 0;
        tiles += (int64_t)lh * s.m_pairs;
        FoldJob& j = jobs[i];
        j.pair0 = s.pair0;
        j.pair_count = lh;
        j.n_in = b.n_in;
        j.n_half = n_half;
        j.sink = sink;
        j.dst = reinterpret_cast<uint4*>(planes);
    }
    if (tiles > 0x7fffffff || (int64_t)n * 2 * lh > 0x7fffffff) return cudaErrorInvalidValue;
    seqs[n] = RaggedSeq{(int32_t)tiles, 0, 0, 0, 0, 0, 1, 0};
    char* meta = static_cast<char*>(state->ragged_meta);
    // pageable sources: each copy has left its host buffer when the call returns
    cudaError_t e = cudaMemcpyAsync(meta, maps.data(), maps_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(meta + maps_bytes, seqs.data(), seqs_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(meta + maps_bytes + seqs_bytes, jobs.data(), jobs_bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return e;

    const unsigned fold_y = (unsigned)std::min<int64_t>(((int64_t)max_half * 16 + 1023) / 1024, 64);
    fold_ragged_kernel<<<dim3((unsigned)(n * 2 * lh), fold_y), 256, 0, stream>>>(
        view, reinterpret_cast<const FoldJob*>(meta + maps_bytes + seqs_bytes), 2 * lh);
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        state->last_error = "fold_ragged_kernel launch";
        return e;
    }
    GemmParams prm = {};
    prm.sink = sink;
    prm.mirror_sign = 1;
    prm.status = status_dev;
    prm.wait_limit_ns = state->wait_limit_ns;
    prm.seq_maps = reinterpret_cast<const CUtensorMap*>(meta);
    prm.seqs = reinterpret_cast<const RaggedSeq*>(meta + maps_bytes);
    prm.n_seqs = (int32_t)n;
    const int clusters = (int)std::min<int64_t>(tiles, state->max_clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (hooks.before) hooks.before(hooks.user, stream);
    e = cudaLaunchKernelEx(&cfg, freqkv_gemm_kernel<MODE_RAGGED>, maps[0], maps[1], maps[1], view, prm);
    if (hooks.after) hooks.after(hooks.user, stream);
    if (e != cudaSuccess) {
        state->last_error = "freqkv_gemm_kernel launch";
        return e;
    }
    state->kernels_last_call = 2;
    return cudaSuccess;
}

// The non-sink rows of one cache tensor as a 5-D tensor (channel, token, kv_head, layer, batch).
static bool encode_cache_map(CUtensorMap* map, const CacheView& view, int tensor, int32_t batch_count, int32_t n_in, int32_t sink)
{
    char* p = static_cast<char*>(tensor ? view.base[1] : view.base[0]) +
              ((int64_t)view.batch0 * view.stride_batch + (int64_t)sink * view.stride_token) * 2;
    const cuuint64_t dims[5] = {128, (cuuint64_t)n_in, (cuuint64_t)view.kv_heads, (cuuint64_t)view.layers,
                                (cuuint64_t)batch_count};
    // an axis of extent 1 is never stepped; give it a harmless stride
    const cuuint64_t row = (cuuint64_t)view.stride_token * 2;
    const cuuint64_t strides[4] = {row, view.kv_heads > 1 ? (cuuint64_t)view.stride_head * 2 : row,
                                   view.layers > 1 ? (cuuint64_t)view.stride_layer * 2 : row,
                                   batch_count > 1 ? (cuuint64_t)view.stride_batch * 2 : row};
    const cuuint32_t box[5] = {64, BK, 1, 1, 1};
    const cuuint32_t elem[5] = {1, 1, 1, 1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, p, dims, strides, box, elem,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool gemm_is_direct(int32_t n_keep) { return n_keep <= 2 * BM; }

// Levels of the symmetry fold a plain compression of these lengths runs: 0 = none (the direct mode), 2 where
// the lengths halve twice (n_in a multiple of 4, n_keep even, the lowest components kept) and the second level
// means fewer 64-row slices per matrix pair (tiles are 256 rows high: with few kept rows it can leave its
// last tile nearly empty and save nothing), else 1.
int32_t gemm_fold_levels(int32_t n_in, int32_t n_keep, int32_t first)
{
    if (gemm_is_direct(n_keep)) return 0;
    if (first != 0 || n_in % 4 != 0 || n_keep % 2 != 0) return 1;
    const int32_t n_half = n_in / 2, rows_half = n_keep / 2, rows_quarter = (rows_half + 1) / 2;
    const int64_t slices1 = (int64_t)((rows_half + 2 * BM - 1) / (2 * BM)) * 2 * ((n_half + BK - 1) / BK);
    const int64_t slices2 =
        (int64_t)((rows_quarter + 2 * BM - 1) / (2 * BM)) * 2 * ((n_half / 2 + BK - 1) / BK + (n_half + BK - 1) / BK);
    return slices2 < slices1 ? 2 : 1;
}

cudaError_t launch_gemm_direct(GemmState* state, const CacheView& view, const Basis& basis, int32_t sink,
                               int32_t* status_dev, int sm_count, const LaunchHooks& hooks, cudaStream_t stream)
{
    state->kernels_last_call = 0;
    const cudaError_t prepared = gemm_prepare(state, 0, basis, sm_count);
    if (prepared != cudaSuccess) return prepared;
    const int32_t pairs = view.mats_per_tensor;
    const int32_t batch_count = pairs / (view.layers * view.kv_heads);
    CUtensorMap map_p, map_k, map_v;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)basis.ld, (cuuint64_t)basis.dense_rows_pad};
        const cuuint64_t strides[1] = {(cuuint64_t)basis.ld * 2};
        const cuuint32_t box[2] = {BK, BM};
        const cuuint32_t elem[2] = {1, 1};
        if (encode_fn()(&map_p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, basis.dense, dims, strides, box, elem,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            state->last_error = "tensor map encoding rejected the basis";
            return cudaErrorInvalidValue;
        }
    }
    if (!encode_cache_map(&map_k, view, 0, batch_count, basis.n_in, sink) ||
        !encode_cache_map(&map_v, view, 1, batch_count, basis.n_in, sink)) {
        state->last_error = "tensor map encoding rejected this layout";
        return cudaErrorInvalidValue;
    }
    GemmParams prm = {};
    prm.n_keep = basis.n_keep;
    prm.rows_half = basis.n_keep;
    prm.basis_rows_pad = 0;
    prm.pair0 = 0;
    prm.pair_count = pairs;
    prm.m_pairs = 1;
    prm.k_steps = (basis.n_in + BK - 1) / BK;
    prm.sink = sink;
    prm.mirror_sign = 1;
    prm.n_in = basis.n_in;
    prm.status = status_dev;
    prm.wait_limit_ns = state->wait_limit_ns;
    const int clusters = std::min<int32_t>(pairs, state->max_clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (hooks.before) hooks.before(hooks.user, stream);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, freqkv_gemm_kernel<MODE_DIRECT>, map_p, map_k, map_v, view, prm);
    if (hooks.after) hooks.after(hooks.user, stream);
    if (e != cudaSuccess) {
        state->last_error = "freqkv_gemm_kernel launch";
        return e;
    }
    state->kernels_last_call = 1;
    return cudaSuccess;
}

cudaError_t launch_wait_probe(int32_t* status_dev, unsigned long long limit_ns, cudaStream_t stream)
{
    bounded_wait_probe_kernel<<<1, 32, 0, stream>>>(status_dev, limit_ns);
    return cudaGetLastError();
}

void gemm_release(GemmState* state)
{
    if (state->ragged_meta) cudaFree(state->ragged_meta);
    state->ragged_meta = nullptr;
    state->ragged_meta_bytes = 0;
    if (state->scratch) cudaFree(state->scratch);
    state->scratch = nullptr;
    state->scratch_bytes = 0;
}

}  // namespace freqkv
