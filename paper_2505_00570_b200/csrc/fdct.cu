// Fast-transform execution of the compression (Section 3.3, Eq. 2-3) for power-of-two lengths:
// the O(N log N) route the paper points to (Appendix A: the DCT can be computed with the FFT).
//
// Two channels of a matrix are packed as the real and imaginary part of one complex sequence
// w_n (every step below is linear with real coefficients on each part, so the two channels
// never mix in the result).  For N input rows and L kept rows:
//
//   1. reorder  v_n = w_{2n},  v_{N-1-n} = w_{2n+1}                       (n < N/2)
//   2. V = FFT_N(v)                                                        (complex, forward)
//   3. DCT-II of both channels at once:  C_t = (phi_t V_t + conj(phi_t) V_{N-t}) / 2,
//      phi_t = exp(-i pi t / (2N));  the orthonormal factors of the DCT, of the L-point inverse
//      and the sqrt(L/N) rescale multiply to 2/N (1/N at t = 0):  g_t = 2 C_t / N,  g_0 = C_0 / N
//   4. keep t < L, and prepare the inverse:  U_0 = g_0,
//      U_t = psi_t (g_t - i g_{L-t}) / 2,  psi_t = exp(+i pi t / (2L))
//   5. r = inverse FFT_L(U) (unnormalised);  y_{2n} = r_n,  y_{2n+1} = r_{L-1-n}.
//
// One CTA owns 8192 complex points = P channel pairs of one matrix (P = 8192 / N), keeps them in
// shared memory for the whole chain and writes the L output rows over the input rows of its own
// channels: no other CTA touches those columns, so the transform is in place in global memory
// with no scratch.  Both FFTs run in place in shared memory, one radix-16 (8/4/2 for the odd
// factor) butterfly at a time per thread, held in registers: the forward one as decimation in
// time on digit-reversed input -- the load phase puts every element where that order wants it --
// the inverse one as decimation in frequency, whose digit-reversed output the store phase reads
// back in row order.  The twiddle of a butterfly is computed (sincospif of an exactly scaled
// index); the factors of the DCT spectrum and of the inverse's pre-twiddle come from fp64-built tables.
// Indices are padded (see pad()) so that the passes meet few shared-memory bank conflicts.
#include <cuda.h>

#include "fdct.cuh"

namespace freqkv {
namespace {

constexpr int POINTS = 8192;  // complex points per CTA
constexpr int THREADS = 256;

// One extra element per 16 and one more per 256: elements 1, 16 or 256 apart (the strides of the
// passes and of the digit-reversed placement) then fall into different shared-memory banks.
__host__ __device__ __forceinline__ int pad(int i) { return i + (i >> 4) + (i >> 8); }

__device__ __forceinline__ float2 cmul(float2 a, float2 b)
{
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 conjf2(float2 a) { return make_float2(a.x, -a.y); }

// exp(-+ 2 pi i q / 16), q = 0..7 (sign: forward -, inverse +)
template <int Q, bool INV>
__device__ __forceinline__ float2 mul_w16(float2 a)
{
    constexpr float C[8] = {1.f, 0.9238795325112867f, 0.7071067811865476f, 0.3826834323650898f,
                            0.f, -0.3826834323650898f, -0.7071067811865476f, -0.9238795325112867f};
    constexpr float S[8] = {0.f, 0.3826834323650898f, 0.7071067811865476f, 0.9238795325112867f,
                            1.f, 0.9238795325112867f, 0.7071067811865476f, 0.3826834323650898f};
    if constexpr (Q == 0) {
        return a;
    } else if constexpr (Q == 4) {  // -+ i
        return INV ? make_float2(-a.y, a.x) : make_float2(a.y, -a.x);
    } else {
        constexpr float c = C[Q], s = INV ? S[Q] : -S[Q];
        return make_float2(fmaf(a.x, c, -a.y * s), fmaf(a.x, s, a.y * c));
    }
}

// In-register R-point DFT, natural order in and out (decimation in time).
template <int R, bool INV>
struct SmallFft {
    template <int K>
    static __device__ __forceinline__ void combine(float2 (&v)[R], const float2 (&e)[R / 2], const float2 (&o)[R / 2])
    {
        if constexpr (K < R / 2) {
            const float2 t = mul_w16<K * (16 / R), INV>(o[K]);
            v[K] = cadd(e[K], t);
            v[K + R / 2] = csub(e[K], t);
            combine<K + 1>(v, e, o);
        }
    }
    static __device__ __forceinline__ void run(float2 (&v)[R])
    {
        float2 e[R / 2], o[R / 2];
#pragma unroll
        for (int i = 0; i < R / 2; ++i) {
            e[i] = v[2 * i];
            o[i] = v[2 * i + 1];
        }
        SmallFft<R / 2, INV>::run(e);
        SmallFft<R / 2, INV>::run(o);
        combine<0>(v, e, o);
    }
};
template <bool INV>
struct SmallFft<1, INV> {
    static __device__ __forceinline__ void run(float2 (&)[1]) {}
};

// One transform is a sequence of in-place passes, each with a radix R = 2^log_r and a stride
// S = 2^log_s (the product of the radices of the passes below it): radix-16 passes with strides
// 1, 16, 256, ..., then, when log2 of the length is not a multiple of 4, one pass of radix 8, 4 or 2
// on top.  (Lengths are at least 16, so pass 0 always has radix 16.)
struct Passes {
    int32_t count;
    int32_t log_r[4], log_s[4];
};

// Where element n of the natural order sits in the digit-reversed order that goes with `passes`:
// the lowest digit of n (radix of the last pass) selects the block of the largest stride, and so on.
__device__ __forceinline__ int digit_pos(int n, const Passes& ps)
{
    int pos = 0;
#pragma unroll
    for (int p = 3; p >= 0; --p) {
        if (p < ps.count) {
            pos += (n & ((1 << ps.log_r[p]) - 1)) << ps.log_s[p];
            n >>= ps.log_r[p];
        }
    }
    return pos;
}

// v[q] *= w^q, q = 1 .. R-1.
template <int R>
__device__ __forceinline__ void twiddle_all(float2 (&v)[R], float2 w1)
{
    v[1] = cmul(v[1], w1);
    if constexpr (R >= 4) {
        const float2 w2 = cmul(w1, w1), w3 = cmul(w2, w1);
        v[2] = cmul(v[2], w2);
        v[3] = cmul(v[3], w3);
        if constexpr (R >= 8) {
            const float2 w4 = cmul(w2, w2);
            v[4] = cmul(v[4], w4);
            v[5] = cmul(v[5], cmul(w4, w1));
            v[6] = cmul(v[6], cmul(w4, w2));
            v[7] = cmul(v[7], cmul(w4, w3));
            if constexpr (R >= 16) {
                const float2 w8 = cmul(w4, w4), w12 = cmul(w8, w4);
                v[8] = cmul(v[8], w8);
                v[9] = cmul(v[9], cmul(w8, w1));
                v[10] = cmul(v[10], cmul(w8, w2));
                v[11] = cmul(v[11], cmul(w8, w3));
                v[12] = cmul(v[12], w12);
                v[13] = cmul(v[13], cmul(w12, w1));
                v[14] = cmul(v[14], cmul(w12, w2));
                v[15] = cmul(v[15], cmul(w12, w3));
            }
        }
    }
}

// One in-place pass over `pairs` sequences of 2^log_n points stored at s[pair * stride + pad(i)].
// Butterfly g of a sequence (2^(log_n - log_r) of them) works on the R elements base + q S,
// base = (g / S) S R + k, k = g mod S.  A thread does its butterflies one after the other.
//   forward (decimation in time, input digit-reversed, output natural):
//     element q is multiplied by w^(q k), w = exp(-2 pi i / (S R)), then the R-point DFT;
//   inverse (decimation in frequency, input natural, output digit-reversed):
//     the R-point inverse DFT, then output r is multiplied by conj(w)^(r k).
// W[j] = exp(-2 pi i j / 2^log_table).
// The stride is 1, 16, 256 or 4096 (see make_passes), for which the padded position of element q
// is pad(base) + q * STEP with a constant STEP: S = 1: consecutive (base is a multiple of R);
// S = 16: base + 16 q stays inside one group of 256, so only the per-16 padding grows, by one per q;
// S a multiple of 256: both paddings grow by whole amounts.
template <int R, int LOG_S, bool INV>
__device__ __forceinline__ void fft_pass(float2* s, int log_n, int seq_stride, int pairs, const float2* __restrict__ W,
                                         int log_table, int tid)
{
    constexpr int log_r = R == 16 ? 4 : R == 8 ? 3 : R == 4 ? 2 : 1;
    constexpr int S = 1 << LOG_S;
    constexpr int STEP = LOG_S == 0 ? 1 : LOG_S == 4 ? 17 : S + (S >> 4) + (S >> 8);
    const int log_bf = log_n - log_r;  // butterflies per sequence
    const int total = pairs << log_bf;
    for (int g = tid; g < total; g += THREADS) {
        const int pair = g >> log_bf, j = g & ((1 << log_bf) - 1), k = j & (S - 1);
        float2* x = s + pair * seq_stride + pad(((j >> LOG_S) << (LOG_S + log_r)) + k);
        float2 v[R];
#pragma unroll
        for (int q = 0; q < R; ++q) v[q] = x[q * STEP];
        if constexpr (LOG_S > 0) {
            // w^q for q = 1 .. R-1 from one table entry: w^2 and w^3 by products, the rest as
            // w^(4a+b) = (w^4)^a w^b, so that no power is more than three products away from the table
            // w = exp(-2 pi i k / (S R)), computed (an exact power-of-two scaling of k, then sincospif): a table
            // entry per butterfly would cost one scattered 8-byte global load per lane on the load/store pipe
            float2 w1;
            sincospif(-(float)k * (2.0f / (float)(S << log_r)), &w1.y, &w1.x);
            if (INV) w1.y = -w1.y;
            if (!INV) twiddle_all<R>(v, w1);
            SmallFft<R, INV>::run(v);
            if (INV) twiddle_all<R>(v, w1);
        } else {
            SmallFft<R, INV>::run(v);
        }
#pragma unroll
        for (int q = 0; q < R; ++q) x[q * STEP] = v[q];
    }
    __syncthreads();
}

template <int LOG_S, bool INV>
__device__ __forceinline__ void fft_pass_radix(int log_r, float2* s, int log_n, int seq_stride, int pairs,
                                               const float2* __restrict__ W, int log_table, int tid)
{
    switch (log_r) {
        case 4: fft_pass<16, LOG_S, INV>(s, log_n, seq_stride, pairs, W, log_table, tid); break;
        case 3: fft_pass<8, LOG_S, INV>(s, log_n, seq_stride, pairs, W, log_table, tid); break;
        case 2: fft_pass<4, LOG_S, INV>(s, log_n, seq_stride, pairs, W, log_table, tid); break;
        default: fft_pass<2, LOG_S, INV>(s, log_n, seq_stride, pairs, W, log_table, tid); break;
    }
}

// All passes of one transform, in the order the direction needs: forward from stride 1 up,
// inverse from the largest stride down.
template <bool INV>
__device__ __forceinline__ void fft_all(float2* s, int log_n, int seq_stride, int pairs, const Passes& ps,
                                        const float2* __restrict__ W, int log_table, int tid)
{
    // (constant indices into the pass list: it lives in the kernel's parameter space)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int p = INV ? 3 - i : i;
        if (p >= ps.count) continue;
        switch (ps.log_s[p]) {
            case 0: fft_pass<16, 0, INV>(s, log_n, seq_stride, pairs, W, log_table, tid); break;  // stride 1 is always radix 16
            case 4: fft_pass_radix<4, INV>(ps.log_r[p], s, log_n, seq_stride, pairs, W, log_table, tid); break;
            case 8: fft_pass_radix<8, INV>(ps.log_r[p], s, log_n, seq_stride, pairs, W, log_table, tid); break;
            default: fft_pass_radix<12, INV>(ps.log_r[p], s, log_n, seq_stride, pairs, W, log_table, tid); break;
        }
    }
}

template <typename T>
__device__ __forceinline__ float2 load_pair(const T* p);
template <>
__device__ __forceinline__ float2 load_pair<float>(const float* p)
{
    return *reinterpret_cast<const float2*>(p);
}
template <>
__device__ __forceinline__ float2 load_pair<__nv_bfloat16>(const __nv_bfloat16* p)
{
    const uint32_t u = *reinterpret_cast<const uint32_t*>(p);
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}
// Two neighbouring pairs (four channels) with one load.
__device__ __forceinline__ void load_two_pairs(const float* p, float2& a, float2& b)
{
    const float4 u = *reinterpret_cast<const float4*>(p);
    a = make_float2(u.x, u.y);
    b = make_float2(u.z, u.w);
}
__device__ __forceinline__ void load_two_pairs(const __nv_bfloat16* p, float2& a, float2& b)
{
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    a = make_float2(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
    b = make_float2(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
}
__device__ __forceinline__ void store_pair(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
__device__ __forceinline__ void store_pair(__nv_bfloat16* p, float2 v)
{
    const __nv_bfloat162 b = __floats2bfloat162_rn(v.x, v.y);
    *reinterpret_cast<uint32_t*>(p) = *reinterpret_cast<const uint32_t*>(&b);
}
__device__ __forceinline__ void store_two_pairs(float* p, float2 a, float2 b)
{
    *reinterpret_cast<float4*>(p) = make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ void store_two_pairs(__nv_bfloat16* p, float2 a, float2 b)
{
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(b.x, b.y);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}

struct FdctParams {
    int32_t log_n, log_l;     // N = 2^log_n input rows, L = 2^log_l kept rows
    int32_t log_pairs;        // P = 2^log_pairs channel pairs per CTA (P * N = POINTS)
    int32_t groups_per_mat;   // head_dim / (2 P)
    int32_t sink;
    Passes fwd, inv;          // pass lists of the N-point and of the L-point transform
    const float2* W;          // exp(-2 pi i q / N), q < N
    const float2* phi;        // exp(-i pi t / (2N)) / N, t <= L
    const float2* psi;        // exp(+i pi t / (2L)) / 2, t <= L
};

template <typename T>
__global__ void __launch_bounds__(THREADS, 3) fdct_kernel(CacheView view, FdctParams prm)
{
    extern __shared__ float2 s[];
    const int tid = threadIdx.x;
    const int N = 1 << prm.log_n, L = 1 << prm.log_l, P = 1 << prm.log_pairs;
    const int ps = pad(N) + 1;  // sequence stride in shared memory

    const int32_t mat = blockIdx.x / prm.groups_per_mat, group = blockIdx.x % prm.groups_per_mat;
    const int32_t tensor = mat / view.mats_per_tensor;
    T* x = static_cast<T*>(tensor_base(view, tensor)) + matrix_offset(view, mat % view.mats_per_tensor) +
           (int64_t)prm.sink * view.stride_token + group * 2 * P;

    // 1. load, reorder (row m -> v index m/2 for even m, N-1-(m-1)/2 for odd m) and place every
    //    element where the in-place forward transform wants it (digit-reversed)
    if (P >= 2) {
        const int half = P >> 1, log_half = prm.log_pairs - 1;
        for (int idx = tid; idx < (N << log_half); idx += THREADS) {
            const int m = idx >> log_half, p2 = idx & (half - 1);
            float2 a, b;
            load_two_pairs(x + (int64_t)m * view.stride_token + 4 * p2, a, b);
            const int vi = (m & 1) ? N - 1 - (m >> 1) : (m >> 1);
            const int at = pad(digit_pos(vi, prm.fwd));
            s[(2 * p2) * ps + at] = a;
            s[(2 * p2 + 1) * ps + at] = b;
        }
    } else {
        for (int m = tid; m < N; m += THREADS) {
            const int vi = (m & 1) ? N - 1 - (m >> 1) : (m >> 1);
            s[pad(digit_pos(vi, prm.fwd))] = load_pair<T>(x + (int64_t)m * view.stride_token);
        }
    }
    __syncthreads();

    // 2. forward FFT of length N on every pair (natural order out)
    fft_all<false>(s, prm.log_n, ps, P, prm.fwd, prm.W, prm.log_n, tid);

    // 3-4. spectrum of the DCT, truncation, and the pre-twiddle of the inverse, in place in [0, L)
    {
        const int half = L >> 1;  // items t = 1 .. L/2 per pair, partner L - t
        const int log_half = prm.log_l - 1;
        const int items = P << log_half;
        for (int idx = tid; idx < items; idx += THREADS) {
            const int p = idx >> log_half, t = (idx & (half - 1)) + 1, u = L - t;
            float2* q = s + p * ps;
            const float2 vt = q[pad(t)], vnt = q[pad(N - t)], vu = q[pad(u)], vnu = q[pad(N - u)];
            const float2 ft = __ldg(prm.phi + t), fu = __ldg(prm.phi + u);
            const float2 gt = cadd(cmul(ft, vt), cmul(conjf2(ft), vnt));
            const float2 gu = cadd(cmul(fu, vu), cmul(conjf2(fu), vnu));
            // U_t = psi_t (g_t - i g_u), U_u = psi_u (g_u - i g_t);  -i (a + ib) = b - ia
            const float2 ut = cmul(__ldg(prm.psi + t), make_float2(gt.x + gu.y, gt.y - gu.x));
            const float2 uu = cmul(__ldg(prm.psi + u), make_float2(gu.x + gt.y, gu.y - gt.x));
            q[pad(t)] = ut;
            q[pad(u)] = uu;
        }
        if (tid < P) {  // t = 0: U_0 = g_0 = V_0 / N  (phi[0] = 1/N)
            float2* q = s + tid * ps;
            const float2 v0 = q[0];
            q[0] = make_float2(v0.x * prm.phi[0].x, v0.y * prm.phi[0].x);
        }
    }
    __syncthreads();

    // 5. inverse FFT of length L (digit-reversed order out), then un-reorder and store over rows [sink, sink + L)
    fft_all<true>(s, prm.log_l, ps, P, prm.inv, prm.W, prm.log_n, tid);

    if (P >= 2) {
        const int half = P >> 1, log_half = prm.log_pairs - 1;
        for (int idx = tid; idx < (L << log_half); idx += THREADS) {
            const int m = idx >> log_half, p2 = idx & (half - 1);
            const int ri = (m & 1) ? L - 1 - (m >> 1) : (m >> 1);
            const int at = pad(digit_pos(ri, prm.inv));
            store_two_pairs(x + (int64_t)m * view.stride_token + 4 * p2, s[(2 * p2) * ps + at], s[(2 * p2 + 1) * ps + at]);
        }
    } else {
        for (int m = tid; m < L; m += THREADS) {
            const int ri = (m & 1) ? L - 1 - (m >> 1) : (m >> 1);
            store_pair(x + (int64_t)m * view.stride_token, s[pad(digit_pos(ri, prm.inv))]);
        }
    }
}

// exp tables in fp64: W[q] = exp(-2 pi i q / N); phi[t] = exp(-i pi t/(2N)) / N; psi[t] = exp(i pi t/(2L)) / 2.
__global__ void fdct_tables_kernel(float2* W, float2* phi, float2* psi, int32_t N, int32_t L)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) {
        double sn, cs;
        sincospi(2.0 * (double)i / (double)N, &sn, &cs);
        W[i] = make_float2((float)cs, (float)-sn);
    }
    if (i <= L) {
        double sn, cs;
        sincospi((double)i / (2.0 * (double)N), &sn, &cs);
        phi[i] = make_float2((float)(cs / N), (float)(-sn / N));
        sincospi((double)i / (2.0 * (double)L), &sn, &cs);
        psi[i] = make_float2((float)(cs * 0.5), (float)(sn * 0.5));
    }
}

int ilog2(int32_t x)
{
    int l = 0;
    while ((1 << l) < x) ++l;
    return l;
}

Passes make_passes(int log_len)
{
    Passes ps = {};
    int log_s = 0;
    for (int i = 0; i < log_len / 4; ++i) {
        ps.log_r[ps.count] = 4;
        ps.log_s[ps.count++] = log_s;
        log_s += 4;
    }
    if (log_len % 4) {
        ps.log_r[ps.count] = log_len % 4;
        ps.log_s[ps.count++] = log_s;
    }
    return ps;
}

size_t smem_bytes(int32_t N)
{
    const int P = POINTS / N;
    return (size_t)P * (pad(N) + 1) * sizeof(float2);
}

}  // namespace

bool fdct_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep)
{
    if (dtype != FREQKV_BF16 && dtype != FREQKV_F32) return false;
    if (n_in < 128 || n_in > POINTS || (n_in & (n_in - 1))) return false;
    if (n_keep < 16 || n_keep > n_in / 2 || (n_keep & (n_keep - 1))) return false;
    const int P = POINTS / n_in;
    return head_dim % (2 * P) == 0;
}

cudaError_t fdct_make_plan(int32_t n_in, int32_t n_keep, cudaStream_t stream, FdctPlan* out)
{
    float2* buf = nullptr;
    const size_t count = (size_t)n_in + 2 * ((size_t)n_keep + 1);
    cudaError_t e = cudaMalloc(&buf, count * sizeof(float2));
    if (e != cudaSuccess) return e;
    float2* W = buf;
    float2* phi = buf + n_in;
    float2* psi = phi + n_keep + 1;
    fdct_tables_kernel<<<(n_in + 255) / 256, 256, 0, stream>>>(W, phi, psi, n_in, n_keep);
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        cudaFree(buf);
        return e;
    }
    out->twiddle = buf;
    out->n_in = n_in;
    out->n_keep = n_keep;
    return cudaSuccess;
}

void fdct_free_plan(FdctPlan* plan)
{
    if (plan->twiddle) cudaFree(plan->twiddle);
    plan->twiddle = nullptr;
}

cudaError_t launch_fdct(const CacheView& view, int32_t dtype, int32_t n_mat, const FdctPlan& plan, int32_t sink,
                        cudaStream_t stream)
{
    static PerDeviceOnce attrs;
    const size_t smem = smem_bytes(plan.n_in);
    const cudaError_t attr_error = attrs.run([] {
        const size_t max_smem = smem_bytes(128);  // the largest footprint (most pairs, most padding rows)
        cudaError_t e = cudaFuncSetAttribute(fdct_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(fdct_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
        return e;
    });
    if (attr_error != cudaSuccess) return attr_error;
    FdctParams prm;
    prm.log_n = ilog2(plan.n_in);
    prm.log_l = ilog2(plan.n_keep);
    const int P = POINTS / plan.n_in;
    prm.log_pairs = ilog2(P);
    prm.groups_per_mat = view.head_dim / (2 * P);
    prm.sink = sink;
    prm.fwd = make_passes(prm.log_n);
    prm.inv = make_passes(prm.log_l);
    prm.W = plan.twiddle;
    prm.phi = plan.twiddle + plan.n_in;
    prm.psi = prm.phi + plan.n_keep + 1;
    const unsigned grid = (unsigned)n_mat * (unsigned)prm.groups_per_mat;
    if (dtype == FREQKV_F32)
        fdct_kernel<float><<<grid, THREADS, smem, stream>>>(view, prm);
    else
        fdct_kernel<__nv_bfloat16><<<grid, THREADS, smem, stream>>>(view, prm);
    return cudaGetLastError();
}

}  // namespace freqkv
