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
// with no scratch.  FFT passes are Stockham radix-16 (remainder 8/4/2) butterflies held in
// registers; a thread reads all its inputs, the CTA synchronises, then it writes.  Indices are
// padded by one element per 16 so the stride-16 writes of the first pass are conflict-free.
#include <cuda.h>

#include "fdct.cuh"

namespace freqkv {
namespace {

constexpr int POINTS = 8192;  // complex points per CTA
constexpr int THREADS = 256;
constexpr int PPT = POINTS / THREADS;  // 32 points per thread in a forward pass

__device__ __forceinline__ int pad(int i) { return i + (i >> 4); }

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

// One Stockham pass of radix R over `pairs` sequences of length n stored at s[pair * ps + pad(i)].
// Butterfly j (of n/R per sequence) reads x[j + r n/R], multiplies by w^(r k) with k = j mod ns and
// w = exp(-+ 2 pi i / (ns R)), transforms, and writes y[(j - k) R + k + r ns].
template <int R, int B, bool INV>
__device__ __forceinline__ void fft_pass(float2* s, int log_n, int ps, int pairs, int log_ns, const float2* __restrict__ W,
                                         int log_table, int tid)
{
    float2 v[B][R];
    int dst[B];  // pair << 20 | first output index; -1 when this slot has no butterfly
    constexpr int log_r = R == 16 ? 4 : R == 8 ? 3 : R == 4 ? 2 : 1;
    const int log_bf = log_n - log_r;  // butterflies per sequence
    const int total = pairs << log_bf;
    const int span = 1 << log_bf, ns = 1 << log_ns;
#pragma unroll
    for (int b = 0; b < B; ++b) {
        const int g = tid + b * THREADS;
        dst[b] = -1;
        if (g < total) {
            const int pair = g >> log_bf, j = g & (span - 1), k = j & (ns - 1);
            const float2* x = s + pair * ps;
#pragma unroll
            for (int r = 0; r < R; ++r) v[b][r] = x[pad(j + r * span)];
            if (log_ns > 0) {
                float2 w1 = W[k << (log_table - log_r - log_ns)];  // exp(-2 pi i k / (ns R))
                if (INV) w1.y = -w1.y;
                float2 w = w1;
#pragma unroll
                for (int r = 1; r < R; ++r) {
                    v[b][r] = cmul(v[b][r], w);
                    if (r + 1 < R) w = cmul(w, w1);
                }
            }
            SmallFft<R, INV>::run(v[b]);
            dst[b] = (pair << 20) | ((j - k) * R + k);
        }
    }
    __syncthreads();
#pragma unroll
    for (int b = 0; b < B; ++b) {
        if (dst[b] >= 0) {
            float2* y = s + (dst[b] >> 20) * ps;
            const int j0 = dst[b] & ((1 << 20) - 1);
#pragma unroll
            for (int r = 0; r < R; ++r) y[pad(j0 + r * ns)] = v[b][r];
        }
    }
    __syncthreads();
}

// All passes of one transform of length 2^log_n over `pairs` sequences.  PPT_ = points per thread
// (32 forward, fewer for the shorter inverse); a radix-R pass gives each thread max(1, PPT_/R)
// butterflies, guarded by the butterfly count.
template <bool INV, int PPT_>
__device__ __forceinline__ void fft_all(float2* s, int log_n, int ps, int pairs, const float2* __restrict__ W,
                                        int log_table, int tid)
{
    int log_ns = 0, left = log_n;
    while (left > 0) {
        if (left >= 4) {
            fft_pass<16, (PPT_ >= 16 ? PPT_ / 16 : 1), INV>(s, log_n, ps, pairs, log_ns, W, log_table, tid);
            log_ns += 4, left -= 4;
        } else if (left == 3) {
            fft_pass<8, (PPT_ >= 8 ? PPT_ / 8 : 1), INV>(s, log_n, ps, pairs, log_ns, W, log_table, tid);
            log_ns += 3, left -= 3;
        } else if (left == 2) {
            fft_pass<4, (PPT_ >= 4 ? PPT_ / 4 : 1), INV>(s, log_n, ps, pairs, log_ns, W, log_table, tid);
            log_ns += 2, left -= 2;
        } else {
            fft_pass<2, (PPT_ >= 2 ? PPT_ / 2 : 1), INV>(s, log_n, ps, pairs, log_ns, W, log_table, tid);
            log_ns += 1, left -= 1;
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
__device__ __forceinline__ void store_pair(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
__device__ __forceinline__ void store_pair(__nv_bfloat16* p, float2 v)
{
    const __nv_bfloat162 b = __floats2bfloat162_rn(v.x, v.y);
    *reinterpret_cast<uint32_t*>(p) = *reinterpret_cast<const uint32_t*>(&b);
}

struct FdctParams {
    int32_t log_n, log_l;     // N = 2^log_n input rows, L = 2^log_l kept rows
    int32_t log_pairs;        // P = 2^log_pairs channel pairs per CTA (P * N = POINTS)
    int32_t groups_per_mat;   // head_dim / (2 P)
    int32_t sink;
    const float2* W;          // exp(-2 pi i q / N), q < N
    const float2* phi;        // exp(-i pi t / (2N)) / N, t <= L
    const float2* psi;        // exp(+i pi t / (2L)) / 2, t <= L
};

template <typename T>
__global__ void __launch_bounds__(THREADS, 2) fdct_kernel(CacheView view, FdctParams prm)
{
    extern __shared__ float2 s[];
    const int tid = threadIdx.x;
    const int N = 1 << prm.log_n, L = 1 << prm.log_l, P = 1 << prm.log_pairs;
    const int ps = pad(N) + 1;  // sequence stride in shared memory (odd multiple keeps pairs on different banks)

    const int32_t mat = blockIdx.x / prm.groups_per_mat, group = blockIdx.x % prm.groups_per_mat;
    const int32_t tensor = mat / view.mats_per_tensor;
    T* x = static_cast<T*>(tensor_base(view, tensor)) + matrix_offset(view, mat % view.mats_per_tensor) +
           (int64_t)prm.sink * view.stride_token + group * 2 * P;

    // 1. load and reorder: row m -> v index m/2 (m even) or N-1-(m-1)/2 (m odd)
#pragma unroll 4
    for (int i = 0; i < PPT; ++i) {
        const int idx = tid + i * THREADS;
        const int m = idx >> prm.log_pairs, p = idx & (P - 1);
        const float2 w = load_pair<T>(x + (int64_t)m * view.stride_token + 2 * p);
        const int vi = (m & 1) ? N - 1 - (m >> 1) : (m >> 1);
        s[p * ps + pad(vi)] = w;
    }
    __syncthreads();

    // 2. forward FFT of length N on every pair
    fft_all<false, PPT>(s, prm.log_n, ps, P, prm.W, prm.log_n, tid);

    // 3-4. spectrum of the DCT, truncation, and the pre-twiddle of the inverse, in place in [0, L)
    {
        const int half = L >> 1;  // items t = 1 .. L/2 per pair, partner L - t
        const int log_half = prm.log_l - 1;
        const int items = P << log_half;
        for (int idx = tid; idx < items; idx += THREADS) {
            const int p = idx >> log_half, t = (idx & (half - 1)) + 1, u = L - t;
            float2* q = s + p * ps;
            const float2 vt = q[pad(t)], vnt = q[pad(N - t)], vu = q[pad(u)], vnu = q[pad(N - u)];
            const float2 ft = prm.phi[t], fu = prm.phi[u];
            const float2 gt = cadd(cmul(ft, vt), cmul(conjf2(ft), vnt));
            const float2 gu = cadd(cmul(fu, vu), cmul(conjf2(fu), vnu));
            // U_t = psi_t (g_t - i g_u), U_u = psi_u (g_u - i g_t);  -i (a + ib) = b - ia
            const float2 ut = cmul(prm.psi[t], make_float2(gt.x + gu.y, gt.y - gu.x));
            const float2 uu = cmul(prm.psi[u], make_float2(gu.x + gt.y, gu.y - gt.x));
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

    // 5. inverse FFT of length L, then un-reorder and store over rows [sink, sink + L)
    switch (prm.log_n - prm.log_l) {  // points per thread of the inverse = 32 L / N
        case 1: fft_all<true, 16>(s, prm.log_l, ps, P, prm.W, prm.log_n, tid); break;
        case 2: fft_all<true, 8>(s, prm.log_l, ps, P, prm.W, prm.log_n, tid); break;
        case 3: fft_all<true, 4>(s, prm.log_l, ps, P, prm.W, prm.log_n, tid); break;
        case 4: fft_all<true, 2>(s, prm.log_l, ps, P, prm.W, prm.log_n, tid); break;
        default: fft_all<true, 1>(s, prm.log_l, ps, P, prm.W, prm.log_n, tid); break;
    }

    const int out_items = P << prm.log_l;
    for (int idx = tid; idx < out_items; idx += THREADS) {
        const int m = idx >> prm.log_pairs, p = idx & (P - 1);
        const int ri = (m & 1) ? L - 1 - (m >> 1) : (m >> 1);
        store_pair(x + (int64_t)m * view.stride_token + 2 * p, s[p * ps + pad(ri)]);
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

size_t smem_bytes(int32_t N)
{
    const int P = POINTS / N;
    return (size_t)P * ((N + (N >> 4)) + 1) * sizeof(float2);
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
    static bool attr_set[2] = {false, false};
    const size_t smem = smem_bytes(plan.n_in);
    if (!attr_set[dtype == FREQKV_F32]) {
        const size_t max_smem = smem_bytes(128);  // the largest footprint (most pairs, most padding rows)
        const cudaError_t e =
            dtype == FREQKV_F32
                ? cudaFuncSetAttribute(fdct_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem)
                : cudaFuncSetAttribute(fdct_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)max_smem);
        if (e != cudaSuccess) return e;
        attr_set[dtype == FREQKV_F32] = true;
    }
    FdctParams prm;
    prm.log_n = ilog2(plan.n_in);
    prm.log_l = ilog2(plan.n_keep);
    const int P = POINTS / plan.n_in;
    prm.log_pairs = ilog2(P);
    prm.groups_per_mat = view.head_dim / (2 * P);
    prm.sink = sink;
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
