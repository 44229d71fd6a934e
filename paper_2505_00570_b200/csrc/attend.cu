// Decode-time attention of one new token per sequence over the bounded cache (Section 3.4, the
// attention equation over sink tokens + compressed tokens + recent tokens).  Keys are cached
// before RoPE; here every cached key row j is rotated to position j -- its index inside the cache,
// not inside the original sequence -- and the query to position len - 1 (the new token's own key
// and value are row len - 1).  RoPE pairs channel c with channel c + 64 (head_dim 128), angle
// pos * base^(-2c/128).
//
// The work is one pass over the K and V rows of the layer: HBM-bound.  Kernel 1 splits the rows
// of every (sequence, kv head) over `splits` CTAs; inside a CTA each half-warp walks its own run
// of consecutive rows, four rows per round (all loads first): 16 lanes x 2 x 8 bytes cover the
// two halves of a bf16 key row, 16 lanes x 16 bytes a value row.  A lane keeps cos/sin of the
// current row's angle for its four channel pairs and steps them by one row with a fixed rotation
// (re-read from the fp64-built table every 32 rows), so the table costs almost no traffic; a
// round's rows are fetched while the previous round is computed.
// Scores of all G query heads of the kv head are reduced over the 16 lanes by shuffles and fed to
// a running softmax (base-2 exponent, scale * log2 e folded into the query).  Half-warps, then
// warps, merge their (max, sum, weighted values) and the CTA writes one partial per query head;
// kernel 2 merges the partials of the splits, normalises and rounds once to the cache dtype.
#include <algorithm>
#include <cmath>

#include <cuda_fp16.h>

#include "attend.cuh"

namespace freqkv {
namespace {

constexpr int THREADS = 256;
constexpr int RESYNC = 32;          // rows between two exact reloads of cos/sin
constexpr float NEG = -1.0e30f;     // "minus infinity" that stays finite under subtraction
constexpr int PART = 132;           // floats per partial: max, sum, 2 unused, 128 weighted channels

struct AttendParams {
    const void* k;
    const void* v;           // bases of the cache tensors, already moved to the layer
    int64_t stride_batch, stride_head, stride_token;  // elements
    int32_t kv_heads, splits, batch0;
    const void* q;           // [batch, kv_heads * G, 128]
    float* partial;          // [splits][batch][kv_heads * G][PART]
    const float2* table;     // [rows][64]: cos, sin of row * base^(-2c/128); null = no RoPE
    float qscale;            // scale * log2(e)
    int32_t total_batch;
    int32_t len[ATTEND_MAX_BATCH];
};

__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&o)[4])
{
    const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
    o[0] = __uint_as_float(u.x << 16); o[1] = __uint_as_float(u.x & 0xffff0000u);
    o[2] = __uint_as_float(u.y << 16); o[3] = __uint_as_float(u.y & 0xffff0000u);
}
__device__ __forceinline__ void load4(const float* p, float (&o)[4])
{
    const float4 u = __ldg(reinterpret_cast<const float4*>(p));
    o[0] = u.x; o[1] = u.y; o[2] = u.z; o[3] = u.w;
}
// One lane's share of a cache row as loaded: 4 + 4 key channels (c0.., 64 + c0..) and 8 value channels.
template <typename T>
struct RawRow;
template <>
struct RawRow<__nv_bfloat16> {
    uint2 klo, khi;
    uint4 v;
};
template <>
struct RawRow<float> {
    float4 klo, khi, v0, v1;
};

__device__ __forceinline__ void fetch(RawRow<__nv_bfloat16>& r, const __nv_bfloat16* krow, const __nv_bfloat16* vrow)
{
    r.klo = __ldg(reinterpret_cast<const uint2*>(krow));
    r.khi = __ldg(reinterpret_cast<const uint2*>(krow + 64));
    r.v = __ldg(reinterpret_cast<const uint4*>(vrow));
}
__device__ __forceinline__ void fetch(RawRow<float>& r, const float* krow, const float* vrow)
{
    r.klo = __ldg(reinterpret_cast<const float4*>(krow));
    r.khi = __ldg(reinterpret_cast<const float4*>(krow + 64));
    r.v0 = __ldg(reinterpret_cast<const float4*>(vrow));
    r.v1 = __ldg(reinterpret_cast<const float4*>(vrow) + 1);
}
__device__ __forceinline__ void unpack2(uint2 u, float (&o)[4])
{
    o[0] = __uint_as_float(u.x << 16); o[1] = __uint_as_float(u.x & 0xffff0000u);
    o[2] = __uint_as_float(u.y << 16); o[3] = __uint_as_float(u.y & 0xffff0000u);
}
__device__ __forceinline__ void unpack(const RawRow<__nv_bfloat16>& r, float (&klo)[4], float (&khi)[4], float (&v)[8])
{
    unpack2(r.klo, klo);
    unpack2(r.khi, khi);
    const uint32_t w[4] = {r.v.x, r.v.y, r.v.z, r.v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ void unpack(const RawRow<float>& r, float (&klo)[4], float (&khi)[4], float (&v)[8])
{
    klo[0] = r.klo.x; klo[1] = r.klo.y; klo[2] = r.klo.z; klo[3] = r.klo.w;
    khi[0] = r.khi.x; khi[1] = r.khi.y; khi[2] = r.khi.z; khi[3] = r.khi.w;
    v[0] = r.v0.x; v[1] = r.v0.y; v[2] = r.v0.z; v[3] = r.v0.w;
    v[4] = r.v1.x; v[5] = r.v1.y; v[6] = r.v1.z; v[7] = r.v1.w;
}

// 2^x on the special-function unit (2 ulp; the arguments here are <= 0).
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Rotate the pair (lo, hi) by the angle whose cosine and sine are cs.
__device__ __forceinline__ void rotate(float& lo, float& hi, float2 cs)
{
    const float a = lo * cs.x - hi * cs.y, b = hi * cs.x + lo * cs.y;
    lo = a;
    hi = b;
}

template <typename T, int G>
__global__ void __launch_bounds__(THREADS, (G <= 4 ? 2 : 1)) attend_partial_kernel(const AttendParams p)
{
    constexpr int ROWS = G >= 8 ? 2 : 4;  // rows per round and half-warp (fewer when many query heads need registers)
    __shared__ float sm_ml[8][G][2];
    __shared__ float sm_o[8][G][128];

    const int tid = threadIdx.x, warp = tid / 32, l16 = tid % 16, hw = tid / 16;
    const int32_t bh = blockIdx.y, b = bh / p.kv_heads, h = bh % p.kv_heads;
    const int32_t len = p.len[b];
    const int64_t mat = (int64_t)(p.batch0 + b) * p.stride_batch + (int64_t)h * p.stride_head;
    const T* K = static_cast<const T*>(p.k) + mat;
    const T* V = static_cast<const T*>(p.v) + mat;

    // rows of this CTA, then of this half-warp (runs of consecutive rows)
    const int32_t chunk = (len + p.splits - 1) / p.splits;
    const int32_t r0 = min(len, (int32_t)blockIdx.x * chunk), r1 = min(len, r0 + chunk);
    const int32_t per = (r1 - r0 + 15) / 16;
    const int32_t j0 = min(r1, r0 + hw * per), j1 = min(r1, j0 + per);
    const int c0 = 4 * l16;  // this lane's channel pairs: (c0 + i, 64 + c0 + i), i < 4

    // queries of the G heads, rotated to position len - 1 and scaled.  With many query heads they
    // live in shared memory (every half-warp needs the same values) to leave registers for rows in flight.
    constexpr bool Q_SHARED = G >= 4;
    __shared__ float4 sm_q[Q_SHARED ? G : 1][2][16];
    float qlo[G][4], qhi[G][4];
    {
        const T* Q = static_cast<const T*>(p.q) + ((int64_t)(p.batch0 + b) * p.kv_heads + h) * G * 128;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            load4(Q + g * 128 + c0, qlo[g]);
            load4(Q + g * 128 + 64 + c0, qhi[g]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (p.table) rotate(qlo[g][i], qhi[g][i], p.table[(int64_t)(len - 1) * 64 + c0 + i]);
                qlo[g][i] *= p.qscale;
                qhi[g][i] *= p.qscale;
            }
            if (Q_SHARED && hw == 0) {
                sm_q[g][0][l16] = make_float4(qlo[g][0], qlo[g][1], qlo[g][2], qlo[g][3]);
                sm_q[g][1][l16] = make_float4(qhi[g][0], qhi[g][1], qhi[g][2], qhi[g][3]);
            }
        }
    }
    if (Q_SHARED) __syncthreads();
    float2 step[4], cs[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        step[i] = p.table ? p.table[64 + c0 + i] : make_float2(1.f, 0.f);  // row 1: one position
        cs[i] = make_float2(1.f, 0.f);
    }

    float m[G], l[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = NEG;
        l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
    }

    const int32_t rounds = (per + ROWS - 1) / ROWS;  // the same for every half-warp: the shuffles below need whole warps
    RawRow<T> cur[ROWS], nxt[ROWS];
    auto fetch_round = [&](RawRow<T> (&dst)[ROWS], int32_t j) {
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const int32_t jr = max(0, min(j + r, j1 - 1));  // rows past the run re-read a valid row; their scores are discarded
            fetch(dst[r], K + (int64_t)jr * p.stride_token + c0, V + (int64_t)jr * p.stride_token + 8 * l16);
        }
    };
    fetch_round(cur, j0);
    for (int32_t it = 0; it < rounds; ++it) {
        const int32_t j = j0 + it * ROWS;
        if (it + 1 < rounds) fetch_round(nxt, j + ROWS);  // the next round's rows travel while this one is computed
        float klo[ROWS][4], khi[ROWS][4], vv[ROWS][8];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) unpack(cur[r], klo[r], khi[r], vv[r]);
        if (p.table && (j - j0) % RESYNC == 0) {  // exact cos / sin again (ROWS divides RESYNC)
#pragma unroll
            for (int i = 0; i < 4; ++i) cs[i] = p.table[(int64_t)max(0, min(j, j1 - 1)) * 64 + c0 + i];
        }
        float s[G][ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
#pragma unroll
            for (int i = 0; i < 4; ++i) rotate(klo[r][i], khi[r][i], cs[i]);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float acc = 0.f;
                if (Q_SHARED) {
                    const float4 a = sm_q[g][0][l16], b = sm_q[g][1][l16];
                    acc = fmaf(a.x, klo[r][0], fmaf(b.x, khi[r][0], acc));
                    acc = fmaf(a.y, klo[r][1], fmaf(b.y, khi[r][1], acc));
                    acc = fmaf(a.z, klo[r][2], fmaf(b.z, khi[r][2], acc));
                    acc = fmaf(a.w, klo[r][3], fmaf(b.w, khi[r][3], acc));
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc = fmaf(qlo[g][i], klo[r][i], fmaf(qhi[g][i], khi[r][i], acc));
                }
                s[g][r] = acc;
            }
            // angle of the next row
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float c = cs[i].x * step[i].x - cs[i].y * step[i].y, sn = cs[i].y * step[i].x + cs[i].x * step[i].y;
                cs[i] = make_float2(c, sn);
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int r = 0; r < ROWS; ++r) {
#pragma unroll
                for (int off = 8; off >= 1; off >>= 1) s[g][r] += __shfl_xor_sync(0xffffffffu, s[g][r], off);
                if (j + r >= j1) s[g][r] = NEG;
            }
            float mn = m[g];
#pragma unroll
            for (int r = 0; r < ROWS; ++r) mn = fmaxf(mn, s[g][r]);
            const float corr = ex2(m[g] - mn);
            m[g] = mn;
            float w[ROWS], sum = 0.f;
#pragma unroll
            for (int r = 0; r < ROWS; ++r) {
                w[r] = j + r < j1 ? ex2(s[g][r] - mn) : 0.f;
                sum += w[r];
            }
            l[g] = l[g] * corr + sum;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float acc = o[g][i] * corr;
#pragma unroll
                for (int r = 0; r < ROWS; ++r) acc = fmaf(w[r], vv[r][i], acc);
                o[g][i] = acc;
            }
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) cur[r] = nxt[r];
    }

    // merge the two half-warps of each warp, then the 8 warps through shared memory
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m[g], 16), l2 = __shfl_xor_sync(0xffffffffu, l[g], 16);
        const float mn = fmaxf(m[g], m2), ca = ex2(m[g] - mn), cb = ex2(m2 - mn);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float o2 = __shfl_xor_sync(0xffffffffu, o[g][i], 16);
            o[g][i] = o[g][i] * ca + o2 * cb;
        }
        l[g] = l[g] * ca + l2 * cb;
        m[g] = mn;
        if (tid % 32 < 16) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sm_o[warp][g][8 * l16 + i] = o[g][i];
            if (l16 == 0) {
                sm_ml[warp][g][0] = m[g];
                sm_ml[warp][g][1] = l[g];
            }
        }
    }
    __syncthreads();
    for (int idx = tid; idx < G * 128; idx += THREADS) {
        const int g = idx / 128, c = idx % 128;
        float mn = NEG;
#pragma unroll
        for (int w = 0; w < 8; ++w) mn = fmaxf(mn, sm_ml[w][g][0]);
        float sum = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const float f = ex2(sm_ml[w][g][0] - mn);
            sum = fmaf(sm_ml[w][g][1], f, sum);
            acc = fmaf(sm_o[w][g][c], f, acc);
        }
        float* out = p.partial + (((int64_t)blockIdx.x * p.total_batch + p.batch0 + b) * p.kv_heads * G + h * G + g) * PART;
        out[4 + c] = acc;
        if (c == 0) {
            out[0] = mn;
            out[1] = sum;
        }
    }
}

// ---- grouped-query variant on the tensor cores (bf16 caches, two or more query heads per KV head) ----
//
// With G query heads per KV head the CUDA-core kernel above spends its time on G dot products and
// G lane reductions per cache row.  Here a warp takes tiles of 16 cache rows and does both
// contractions with mma.sync (m16n8k16, fp32 accumulate), all heads at once (N = 8 heads, zero
// queries past G):
//   1. cp.async brings the 16 K rows and the 16 V rows of the warp's next tile into its own
//      two-stage ring of shared-memory tiles (16-byte chunks, XOR-swizzled by the row so that
//      ldmatrix meets no bank conflicts) while the current tile is processed;
//   2. the K tile is rotated in place (RoPE at the row's in-cache position, fp32 arithmetic,
//      cos/sin exact at the first row of each half-warp's 8 rows, fetched one round ahead, and
//      stepped from there) and rounded to fp16, not back to bf16: three more mantissa bits keep
//      the score error of a peaked softmax (large scale) a quarter of what bf16 keys would give.
//      Keys and scaled queries must therefore stay below 65504 in magnitude;
//   3. S = K_rot Q^T (fp16 in): A = the K tile through ldmatrix, B = the pre-rotated, pre-scaled
//      queries, kept in registers; a thread's accumulators are rows gq, gq + 8 x heads 2 tq, 2 tq + 1;
//   4. running softmax per head: the maximum over the tile's rows takes three shuffles over the
//      lanes of equal tq; each thread sums the weights of its own rows only (reduced once, at the end);
//   5. O^T += V^T P: the weights, rounded to bf16, become the B fragment through two 8x8 transposes
//      (movmatrix); A = the V tile through ldmatrix.trans; a thread's accumulators are channels
//      16 cb + gq, + 8 x heads 2 tq, 2 tq + 1, so the rescaling factors of step 4 apply as they are.
// 32 accumulators per thread instead of 64 (heads on M would waste half of them on padding) let
// three CTAs of four warps share an SM.  Warps, then splits, are merged as in the CUDA-core kernel.
constexpr int MMA_WARPS = 4, MMA_THREADS = 32 * MMA_WARPS, MMA_CTAS_PER_SM = 3;
constexpr int TILE_ROWS = 16;
constexpr int TILE_BYTES = TILE_ROWS * 256;                   // 16 rows x 128 two-byte values
constexpr int MMA_STAGES = 2;
constexpr int WARP_TILE_BYTES = MMA_STAGES * 2 * TILE_BYTES;  // stages of (K, V)
constexpr int MMA_SMEM_BYTES = MMA_WARPS * WARP_TILE_BYTES;   // 64 KB
static_assert(MMA_WARPS * 8 * (128 + 2) * 4 <= MMA_SMEM_BYTES, "the merge of the warps reuses the tile ring");

__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid)
{
    const int bytes = valid ? 16 : 0;  // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// 8x8 transpose of 16-bit values held one row per 4 lanes (the ldmatrix fragment layout).
__device__ __forceinline__ uint32_t transpose_8x8(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// D += A B, m16n8k16, A row-major, B column-major, fp32 accumulate; bf16 or fp16 operands.
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack2_f16(float lo, float hi)
{
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

template <int G>
__global__ void __launch_bounds__(MMA_THREADS, MMA_CTAS_PER_SM) attend_mma_kernel(const AttendParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int gq = lane / 4, tq = lane % 4;  // fragment coordinates
    const int32_t bh = blockIdx.y, b = bh / p.kv_heads, h = bh % p.kv_heads;
    const int32_t len = p.len[b];
    const int64_t mat = (int64_t)(p.batch0 + b) * p.stride_batch + (int64_t)h * p.stride_head;
    const __nv_bfloat16* K = static_cast<const __nv_bfloat16*>(p.k) + mat;
    const __nv_bfloat16* V = static_cast<const __nv_bfloat16*>(p.v) + mat;

    const int32_t chunk = (len + p.splits - 1) / p.splits;
    const int32_t r0 = min(len, (int32_t)blockIdx.x * chunk), r1 = min(len, r0 + chunk);
    const int32_t n_tiles = (r1 - r0 + TILE_ROWS - 1) / TILE_ROWS;

    const uint32_t warp_smem = (uint32_t)__cvta_generic_to_shared(smem) + warp * WARP_TILE_BYTES;
    auto k_tile = [&](int stage) { return warp_smem + stage * 2 * TILE_BYTES; };
    auto v_tile = [&](int stage) { return warp_smem + stage * 2 * TILE_BYTES + TILE_BYTES; };

    // queries as fp16 B fragments: head gq (zero past G), channels 16 kc + 2 tq (+1) and + 8
    uint32_t qb[8][2];
    {
        const __nv_bfloat16* Q = static_cast<const __nv_bfloat16*>(p.q) + (((int64_t)(p.batch0 + b) * p.kv_heads + h) * G + gq) * 128;
#pragma unroll
        for (int kc = 0; kc < 4; ++kc) {   // channel chunk kc pairs with chunk kc + 4 (channels + 64)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int c = 16 * kc + 8 * half + 2 * tq;
                float lo[2] = {0.f, 0.f}, hi[2] = {0.f, 0.f};
                if (gq < G) {
                    const uint32_t a = *reinterpret_cast<const uint32_t*>(Q + c), bq = *reinterpret_cast<const uint32_t*>(Q + 64 + c);
                    lo[0] = __uint_as_float(a << 16); lo[1] = __uint_as_float(a & 0xffff0000u);
                    hi[0] = __uint_as_float(bq << 16); hi[1] = __uint_as_float(bq & 0xffff0000u);
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        if (p.table) rotate(lo[i], hi[i], p.table[(int64_t)(len - 1) * 64 + c + i]);
                        lo[i] *= p.qscale;
                        hi[i] *= p.qscale;
                    }
                }
                qb[kc][half] = pack2_f16(lo[0], lo[1]);
                qb[kc + 4][half] = pack2_f16(hi[0], hi[1]);
            }
        }
    }

    // rotation roles: half-warp hw rotates rows 8 hw .. 8 hw + 7 of a tile, lane l16 the pairs 4 l16 .. 4 l16 + 3
    const int l16 = lane % 16, hw = lane / 16, c0 = 4 * l16;
    float2 step[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) step[i] = p.table ? p.table[64 + c0 + i] : make_float2(1.f, 0.f);

    // this thread's heads are 2 tq + j
    float m_run[2] = {NEG, NEG}, l_run[2] = {0.f, 0.f};
    float o[8][4];
#pragma unroll
    for (int cb = 0; cb < 8; ++cb)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[cb][i] = 0.f;

    auto prefetch = [&](int32_t tile, int stage) {
        const int32_t row0 = r0 + tile * TILE_ROWS;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int idx = lane + 32 * i, row = idx >> 4, ch = idx & 15;
            const bool ok = row0 + row < r1;
            const int64_t src = (int64_t)min(row0 + row, r1 - 1) * p.stride_token + ch * 8;
            cp_async16(k_tile(stage) + tile_off(row, ch), K + src, ok);
            cp_async16(v_tile(stage) + tile_off(row, ch), V + src, ok);
        }
    };
    // One group is committed per ring slot, empty past the last tile, so that "all but the newest
    // MMA_STAGES - 1 groups" always means "the current tile has landed".
#pragma unroll
    for (int j = 0; j < MMA_STAGES - 1; ++j) {
        if (warp + j * MMA_WARPS < n_tiles) prefetch(warp + j * MMA_WARPS, j);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    float2 cs_next[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        cs_next[i] = p.table ? p.table[(int64_t)min(r0 + warp * TILE_ROWS + 8 * hw, len - 1) * 64 + c0 + i] : make_float2(1.f, 0.f);
    const int mi = lane >> 3, lr = lane & 7;  // ldmatrix roles: lane supplies row lr of matrix mi
    int stage = 0;
    for (int32_t tile = warp; tile < n_tiles; tile += MMA_WARPS, stage = stage + 1 == MMA_STAGES ? 0 : stage + 1) {
        {
            const int ahead = stage == 0 ? MMA_STAGES - 1 : stage - 1;  // the slot processed in the previous round
            if (tile + (MMA_STAGES - 1) * MMA_WARPS < n_tiles) prefetch(tile + (MMA_STAGES - 1) * MMA_WARPS, ahead);
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group %0;" ::"n"(MMA_STAGES - 1) : "memory");
        }
        __syncwarp();
        const int32_t row0 = r0 + tile * TILE_ROWS;
        const uint32_t kt = k_tile(stage), vt = v_tile(stage);
        uint8_t* kt_ptr = smem + warp * WARP_TILE_BYTES + stage * 2 * TILE_BYTES;

        // 2. RoPE on the K tile, in place, bf16 -> fp16 (without RoPE: the conversion alone).  The
        // cos/sin of the tile's first rows were fetched one round ahead; fetch the next round's now.
        {
            float2 cs[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) cs[i] = cs_next[i];
            if (p.table) {
                const float2* t = p.table + (int64_t)min(row0 + MMA_WARPS * TILE_ROWS + 8 * hw, len - 1) * 64 + c0;
#pragma unroll
                for (int i = 0; i < 4; ++i) cs_next[i] = t[i];
            }
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const int row = 8 * hw + r;
                uint2* a_lo = reinterpret_cast<uint2*>(kt_ptr + tile_off(row, l16 >> 1) + (l16 & 1) * 8);
                uint2* a_hi = reinterpret_cast<uint2*>(kt_ptr + tile_off(row, 8 + (l16 >> 1)) + (l16 & 1) * 8);
                uint2 ulo = *a_lo, uhi = *a_hi;
                float lo[4], hi[4];
                unpack2(ulo, lo);
                unpack2(uhi, hi);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    rotate(lo[i], hi[i], cs[i]);
                    const float c = cs[i].x * step[i].x - cs[i].y * step[i].y, sn = cs[i].y * step[i].x + cs[i].x * step[i].y;
                    cs[i] = make_float2(c, sn);
                }
                ulo = make_uint2(pack2_f16(lo[0], lo[1]), pack2_f16(lo[2], lo[3]));
                uhi = make_uint2(pack2_f16(hi[0], hi[1]), pack2_f16(hi[2], hi[3]));
                *a_lo = ulo;
                *a_hi = uhi;
            }
            __syncwarp();
        }

        // 3. scores S[row][head]; two accumulators halve the chain of dependent MMAs
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const int krow = (mi & 1) * 8 + lr;
#pragma unroll
            for (int kc = 0; kc < 8; kc += 2) {
                uint32_t ka[4], kb[4];
                ldmatrix_x4(kt + tile_off(krow, 2 * kc + (mi >> 1)), ka);
                ldmatrix_x4(kt + tile_off(krow, 2 * kc + 2 + (mi >> 1)), kb);
                mma_f16(s0, ka, qb[kc][0], qb[kc][1]);
                mma_f16(s1, kb, qb[kc + 1][0], qb[kc + 1][1]);
            }
        }
        // 4. running softmax of heads 2 tq + j over the tile's rows (this thread: rows gq and gq + 8)
        const int32_t left = r1 - row0;  // valid rows in this tile
        const bool ok0 = gq < left, ok1 = gq + 8 < left;
        float corr[2], pw[2][2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float sa = s0[j] + s1[j], sb = s0[2 + j] + s1[2 + j];
            float mx = fmaxf(ok0 ? sa : NEG, ok1 ? sb : NEG);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float m_new = fmaxf(m_run[j], mx);
            corr[j] = ex2(m_run[j] - m_new);
            m_run[j] = m_new;
            pw[0][j] = ok0 ? ex2(sa - m_new) : 0.f;
            pw[1][j] = ok1 ? ex2(sb - m_new) : 0.f;
            l_run[j] = fmaf(l_run[j], corr[j], pw[0][j] + pw[1][j]);
        }
        // 5. O^T = O^T corr + V^T P
        const uint32_t pb0 = transpose_8x8(pack2_bf16(pw[0][0], pw[0][1])), pb1 = transpose_8x8(pack2_bf16(pw[1][0], pw[1][1]));
        {
            const int vrow = (mi >> 1) * 8 + lr;
#pragma unroll
            for (int cb = 0; cb < 8; ++cb) {
                uint32_t va[4];
                ldmatrix_x4_trans(vt + tile_off(vrow, 2 * cb + (mi & 1)), va);
                o[cb][0] *= corr[0];
                o[cb][1] *= corr[1];
                o[cb][2] *= corr[0];
                o[cb][3] *= corr[1];
                mma_bf16(o[cb], va, pb0, pb1);
            }
        }
        __syncwarp();  // the tile may be overwritten by the next prefetch
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 4);
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 8);
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 16);
    }

    // merge the warps through shared memory (the tiles are no longer needed)
    __syncthreads();
    float* sm_ml = reinterpret_cast<float*>(smem);                        // [warps][8 heads][2]
    float* sm_o = reinterpret_cast<float*>(smem) + MMA_WARPS * 8 * 2;     // [warps][8 heads][128]
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int head = warp * 8 + 2 * tq + j;
        if (gq == 0) {
            sm_ml[head * 2] = m_run[j];
            sm_ml[head * 2 + 1] = l_run[j];
        }
#pragma unroll
        for (int cb = 0; cb < 8; ++cb) {
            sm_o[head * 128 + 16 * cb + gq] = o[cb][j];
            sm_o[head * 128 + 16 * cb + 8 + gq] = o[cb][2 + j];
        }
    }
    __syncthreads();
    for (int idx = tid; idx < G * 128; idx += MMA_THREADS) {
        const int g = idx / 128, c = idx % 128;
        float mn = NEG;
#pragma unroll
        for (int w = 0; w < MMA_WARPS; ++w) mn = fmaxf(mn, sm_ml[(w * 8 + g) * 2]);
        float sum = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < MMA_WARPS; ++w) {
            const float f = ex2(sm_ml[(w * 8 + g) * 2] - mn);
            sum = fmaf(sm_ml[(w * 8 + g) * 2 + 1], f, sum);
            acc = fmaf(sm_o[(w * 8 + g) * 128 + c], f, acc);
        }
        float* out = p.partial + (((int64_t)blockIdx.x * p.total_batch + p.batch0 + b) * p.kv_heads * G + h * G + g) * PART;
        out[4 + c] = acc;
        if (c == 0) {
            out[0] = mn;
            out[1] = sum;
        }
    }
}

// One block per (sequence, query head): merge the partials of the splits in one pass, rescaling as
// the maximum grows (unrolled so that the loads of several splits are in flight), normalise and
// round once to the cache dtype.
template <typename T>
__global__ void __launch_bounds__(128) attend_merge_kernel(const float* __restrict__ partial, int32_t splits,
                                                           int64_t heads_total, T* __restrict__ out)
{
    const int64_t head = blockIdx.x;
    const int c = threadIdx.x;
    // launched with programmatic stream serialization: the blocks may start while the kernel that
    // writes the partials is still draining; wait here until that grid has completed and its writes are visible
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float mn = NEG, sum = 0.f, acc = 0.f;
#pragma unroll 8
    for (int s = 0; s < splits; ++s) {
        const float* pp = partial + (s * heads_total + head) * PART;
        const float m_s = pp[0], l_s = pp[1], o_s = pp[4 + c];
        const float m_new = fmaxf(mn, m_s), fa = ex2(mn - m_new), fb = ex2(m_s - m_new);
        sum = fmaf(sum, fa, l_s * fb);
        acc = fmaf(acc, fa, o_s * fb);
        mn = m_new;
    }
    const float y = acc / sum;
    if constexpr (sizeof(T) == 2)
        out[head * 128 + c] = __float2bfloat16_rn(y);
    else
        out[head * 128 + c] = y;
}

// cos / sin of pos * base^(-2c/128) in fp64, rounded once.
__global__ void rope_table_kernel(float2* table, int32_t rows, double base)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)rows * 64) return;
    const int32_t pos = (int32_t)(i / 64), c = (int32_t)(i % 64);
    const double angle = (double)pos * pow(base, -2.0 * c / 128.0);
    double sn, cs;
    sincos(angle, &sn, &cs);
    table[i] = make_float2((float)cs, (float)sn);
}

cudaError_t launch_mma(const AttendParams& prm, int32_t g, int32_t nb, cudaStream_t stream)
{
    static PerDeviceOnce attrs;
    const cudaError_t attr_error = attrs.run([] {
        const void* kernels[3] = {(const void*)attend_mma_kernel<2>, (const void*)attend_mma_kernel<4>, (const void*)attend_mma_kernel<8>};
        for (const void* f : kernels) {
            cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, MMA_SMEM_BYTES);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    });
    if (attr_error != cudaSuccess) return attr_error;
    const dim3 grid((unsigned)prm.splits, (unsigned)(nb * prm.kv_heads));
    switch (g) {
        case 2: attend_mma_kernel<2><<<grid, MMA_THREADS, MMA_SMEM_BYTES, stream>>>(prm); break;
        case 4: attend_mma_kernel<4><<<grid, MMA_THREADS, MMA_SMEM_BYTES, stream>>>(prm); break;
        case 8: attend_mma_kernel<8><<<grid, MMA_THREADS, MMA_SMEM_BYTES, stream>>>(prm); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_typed(const AttendParams& prm, int32_t g, int32_t nb, cudaStream_t stream)
{
    const dim3 grid((unsigned)prm.splits, (unsigned)(nb * prm.kv_heads));
    switch (g) {
        case 1: attend_partial_kernel<T, 1><<<grid, THREADS, 0, stream>>>(prm); break;
        case 2: attend_partial_kernel<T, 2><<<grid, THREADS, 0, stream>>>(prm); break;
        case 4: attend_partial_kernel<T, 4><<<grid, THREADS, 0, stream>>>(prm); break;
        case 8: attend_partial_kernel<T, 8><<<grid, THREADS, 0, stream>>>(prm); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

bool attend_supported(int32_t head_dim, int32_t q_heads_per_kv)
{
    return head_dim == 128 && (q_heads_per_kv == 1 || q_heads_per_kv == 2 || q_heads_per_kv == 4 || q_heads_per_kv == 8);
}

// Splits of the rows of one (sequence, kv head): the count, among those that leave a CTA at least
// 1024 rows, whose CTAs fill whole waves of the resident CTAs best (the smallest such count).
// Shorter chunks with fuller waves measured slower: the prologue (length, queries, table) and the
// partials weigh more than the idle CTA slots.
int32_t attend_splits(int32_t batch, int32_t kv_heads, int32_t max_len, int32_t q_heads_per_kv, int32_t dtype, int sm_count)
{
    const double groups = (double)batch * kv_heads;
    const bool tensor_cores = dtype == FREQKV_BF16 && q_heads_per_kv >= 2;
    const double resident = (double)sm_count * (tensor_cores ? MMA_CTAS_PER_SM : q_heads_per_kv <= 4 ? 2 : 1);
    const int32_t most = std::max(1, std::min(32, max_len / 1024));
    int32_t best = 1;
    double best_fill = 0.0;
    for (int32_t s = 1; s <= most; ++s) {
        const double waves = groups * s / resident, fill = waves / std::ceil(waves);
        if (fill > best_fill + 0.02) {
            best_fill = fill;
            best = s;
        }
    }
    return best;
}

size_t attend_partial_bytes(int32_t splits, int32_t batch, int32_t q_heads)
{
    return (size_t)splits * batch * q_heads * PART * sizeof(float);
}

cudaError_t launch_rope_table(float2* table, int32_t rows, double base, cudaStream_t stream)
{
    const int64_t n = (int64_t)rows * 64;
    rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(table, rows, base);
    return cudaGetLastError();
}

cudaError_t launch_attend(const freqkv_layout& l, const void* k, const void* v, int32_t layer, const void* q, void* out,
                          int32_t g, const int32_t* lens_host, const float2* table, float scale, int32_t splits,
                          float* partial, cudaStream_t stream)
{
    const size_t elt = dtype_size(l.dtype);
    AttendParams prm;
    prm.k = static_cast<const char*>(k) + (size_t)layer * l.stride_layer * elt;
    prm.v = static_cast<const char*>(v) + (size_t)layer * l.stride_layer * elt;
    prm.stride_batch = l.stride_batch;
    prm.stride_head = l.stride_head;
    prm.stride_token = l.stride_token;
    prm.kv_heads = l.kv_heads;
    prm.splits = splits;
    prm.q = q;
    prm.partial = partial;
    prm.table = table;
    prm.qscale = scale * 1.4426950408889634f;
    prm.total_batch = l.batch;
    for (int32_t b0 = 0; b0 < l.batch; b0 += ATTEND_MAX_BATCH) {
        const int32_t nb = std::min(ATTEND_MAX_BATCH, l.batch - b0);
        prm.batch0 = b0;
        for (int32_t i = 0; i < nb; ++i) prm.len[i] = lens_host[b0 + i];
        const cudaError_t e = l.dtype == FREQKV_F32 ? launch_typed<float>(prm, g, nb, stream)
                              : g >= 2             ? launch_mma(prm, g, nb, stream)   // grouped queries: tensor cores
                                                   : launch_typed<__nv_bfloat16>(prm, g, nb, stream);
        if (e != cudaSuccess) return e;
    }
    const int64_t heads_total = (int64_t)l.batch * l.kv_heads * g;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)heads_total);
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;  // let the launch overlap the tail of the kernel before it
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const float* partial_in = partial;
    if (l.dtype == FREQKV_F32)
        return cudaLaunchKernelEx(&cfg, attend_merge_kernel<float>, partial_in, splits, heads_total, static_cast<float*>(out));
    return cudaLaunchKernelEx(&cfg, attend_merge_kernel<__nv_bfloat16>, partial_in, splits, heads_total,
                              static_cast<__nv_bfloat16*>(out));
}

}  // namespace freqkv
