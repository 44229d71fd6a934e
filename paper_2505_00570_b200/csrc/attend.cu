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

// One block per (sequence, query head): merge the partials of the splits.
template <typename T>
__global__ void __launch_bounds__(128) attend_merge_kernel(const float* __restrict__ partial, int32_t splits,
                                                           int64_t heads_total, T* __restrict__ out)
{
    const int64_t head = blockIdx.x;
    const int c = threadIdx.x;
    float mn = NEG;
    for (int s = 0; s < splits; ++s) mn = fmaxf(mn, partial[(s * heads_total + head) * PART]);
    float sum = 0.f, acc = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float* pp = partial + (s * heads_total + head) * PART;
        const float f = ex2(pp[0] - mn);
        sum = fmaf(pp[1], f, sum);
        acc = fmaf(pp[4 + c], f, acc);
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
int32_t attend_splits(int32_t batch, int32_t kv_heads, int32_t max_len, int32_t q_heads_per_kv, int sm_count)
{
    const double groups = (double)batch * kv_heads;
    const double resident = (double)sm_count * (q_heads_per_kv <= 4 ? 2 : 1);
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
                                                    : launch_typed<__nv_bfloat16>(prm, g, nb, stream);
        if (e != cudaSuccess) return e;
    }
    const int64_t heads_total = (int64_t)l.batch * l.kv_heads * g;
    if (l.dtype == FREQKV_F32)
        attend_merge_kernel<float><<<(unsigned)heads_total, 128, 0, stream>>>(partial, splits, heads_total, static_cast<float*>(out));
    else
        attend_merge_kernel<__nv_bfloat16><<<(unsigned)heads_total, 128, 0, stream>>>(partial, splits, heads_total,
                                                                                  static_cast<__nv_bfloat16*>(out));
    return cudaGetLastError();
}

}  // namespace freqkv
