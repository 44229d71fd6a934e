// Projection basis of one compression (Section 3.3, Eq. 2-3 with the transforms of
// Appendix A).  DCT-II of length N, truncation to L components, L-point inverse DCT and the
// sqrt(L/N) rescale are one linear map Y = P X with
//
//   P[m][n] = (1/N) * [ 1 + 2 * sum_{t=1}^{L-1} cos(pi t (2m+1)/(2L)) * cos(pi t (2n+1)/(2N)) ].
//
// The product of cosines splits into cosines of the sum and difference angle, and each of the
// two cosine series sums to a Dirichlet kernel:
//
//   P[m][n] = (1/(2N)) * [ D(a+) + D(a-) ],   a± = (2m+1) N ± (2n+1) L   (integers),
//   D(a) = sin((2L-1) pi a / (4LN)) / sin(pi a / (4LN)),   D(0) = 2L-1.
//
// 0 < a+ < 4LN and |a-| < 2LN, so the denominator vanishes only at a- = 0.  The numerator's
// phase is reduced exactly in 64-bit integers modulo 8LN before sinpi, so every entry is
// accurate to a few fp64 ulps; it is rounded once to fp32 and once to bf16.
#include <algorithm>

#include "common.cuh"

namespace freqkv {
namespace {

__device__ inline double dirichlet(int64_t a, int64_t L, int64_t LN4)
{
    if (a < 0) a = -a;  // D is even
    if (a == 0) return (double)(2 * L - 1);
    const int64_t r = ((2 * L - 1) * a) % (2 * LN4);
    return sinpi((double)r / (double)LN4) / sinpi((double)a / (double)LN4);
}

// Retaining components t0 .. t0 + L - 1 instead of the lowest L (the paper's high/low-frequency
// ablation; t0 >= 1 here).  With A = pi (2m+1) / (2L), B = pi (2n+1) / (2N) the orthonormal weights
// give  P[m][n] = (sqrt 2 / N) [ cos(B t0) + sqrt 2 * sum_{t'=1}^{L-1} cos(A t') cos(B (t0 + t')) ],
// and each of the two cosine series the product splits into sums in closed form:
//   sum_{t'=1}^{L-1} cos(theta t' + phi) = sin((L-1) theta / 2) / sin(theta / 2) * cos(L theta / 2 + phi),
// (L - 1) cos(phi) at theta = 0.  All phases are integer multiples of pi / (4LN) and are reduced
// exactly modulo 8LN before sinpi / cospi.
__device__ inline double cos_units(int64_t k, int64_t LN4)
{
    const int64_t period = 2 * LN4;
    k = ((k % period) + period) % period;
    return cospi((double)k / (double)LN4);
}
__device__ inline double sin_units(int64_t k, int64_t LN4)
{
    const int64_t period = 2 * LN4;
    k = ((k % period) + period) % period;
    return sinpi((double)k / (double)LN4);
}
__device__ inline double cosine_series(int64_t a, int64_t phi, int64_t L, int64_t LN4)
{
    if (a == 0) return (double)(L - 1) * cos_units(phi, LN4);
    return sin_units((L - 1) * a, LN4) / sin_units(a, LN4) * cos_units(L * a + phi, LN4);
}

// P[m][n] of the map that keeps components t0 .. t0 + L - 1 of an N-point signal.
__device__ inline double basis_entry(int64_t m, int64_t n, int64_t N, int64_t L, int64_t t0)
{
    const int64_t LN4 = 4 * L * N;
    const int64_t u = (2 * m + 1) * N, w = (2 * n + 1) * L;
    if (t0 == 0) return (dirichlet(u + w, L, LN4) + dirichlet(u - w, L, LN4)) / (double)(2 * N);
    const int64_t phi = (2 * n + 1) * t0 * 2 * L;
    const double series = 0.5 * (cosine_series(u + w, phi, L, LN4) + cosine_series(u - w, -phi, L, LN4));
    return 1.4142135623730951 / (double)N * (cos_units(phi, LN4) + 1.4142135623730951 * series);
}

__global__ void build_basis_kernel(float* __restrict__ p_f32, __nv_bfloat16* __restrict__ p_bf16, int32_t n_in,
                                   int32_t n_keep, int32_t first, int32_t ld, int32_t rows_pad)
{
    const int64_t total = (int64_t)rows_pad * ld;
    const int64_t N = n_in, L = n_keep;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t m = i / ld, n = i % ld;
        double p = 0.0;
        if (m < L && n < N) p = basis_entry(m, n, N, L, first);
        if (p_f32) p_f32[i] = (float)p;
        if (p_bf16) p_bf16[i] = __double2bfloat16(p);
    }
}

// Folded basis for the tensor-core path.  The cosines of the DCT are symmetric or antisymmetric
// under n -> N-1-n and m -> L-1-m according to the parity of the frequency index t, so
// P[m][N-1-n] = Pe[m][n] - Po[m][n] and P[L-1-m][n] = Pe[m][n] - Po[m][n], where Pe (Po) is the part
// of the sum over even (odd) t:  Pe = (P[m][n] + P[m][N-1-n]) / 2,  Po = (P[m][n] - P[m][N-1-n]) / 2.
// Only m < ceil(L/2), n < ceil(N/2) are stored: plane 0 = Pe, plane 1 = Po, each rows_pad x ld,
// zero padded.  For odd N the middle column of Po is zero and that of Pe is P itself, for odd L the
// middle row of Po is zero: the formulas above give exactly that.
// When a band starting at an odd component t0 is retained, the parity of the inverse's index t'
// is opposite to that of t = t0 + t': Pe is then antisymmetric and Po symmetric under m -> L-1-m,
// which only changes a sign in the tensor-core kernel's epilogue.
__global__ void build_folded_basis_kernel(__nv_bfloat16* __restrict__ out, int32_t n_in, int32_t n_keep, int32_t first,
                                          int32_t ld, int32_t rows_pad)
{
    const int64_t plane = (int64_t)rows_pad * ld;
    const int64_t N = n_in, L = n_keep;
    const int64_t Nh = (N + 1) / 2, Lh = (L + 1) / 2;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < plane; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t m = i / ld, n = i % ld;
        double pe = 0.0, po = 0.0;
        if (m < Lh && n < Nh) {
            const double a = basis_entry(m, n, N, L, first), b = basis_entry(m, N - 1 - n, N, L, first);
            pe = 0.5 * (a + b);
            po = 0.5 * (a - b);
        }
        out[i] = __double2bfloat16(pe);
        out[plane + i] = __double2bfloat16(po);
    }
}

// Second fold.  For even L the even-t part Pe is, up to a factor, the basis of the compression of
// N/2 rows to L/2 (t = 2t': cos(pi t' (2m+1) / (2 (L/2))) cos(pi t' (2n+1) / (2 (N/2)))), so it has the same
// symmetries one level down: with N' = N/2, L' = L/2, n < N'/2, m < ceil(L'/2)
//     Pee[m][n] = (Pe[m][n] + Pe[m][N'-1-n]) / 2,   Peo[m][n] = (Pe[m][n] - Pe[m][N'-1-n]) / 2,
//     s_m = Pee uu + Peo uv,   s_{L'-1-m} = Pee uu - Peo uv,     uu_n = u_n + u_{N'-1-n},  uv_n = u_n - u_{N'-1-n}.
// Planes: 0 = Pee, 1 = Peo (columns n < N'/2), 2 = Po[m][.], 3 = Po[L'-1-m][.] (columns n < N'), rows m < ceil(L'/2).
__global__ void build_folded2_basis_kernel(__nv_bfloat16* __restrict__ out, int32_t n_in, int32_t n_keep, int32_t ld,
                                           int32_t rows_pad)
{
    const int64_t plane = (int64_t)rows_pad * ld;
    const int64_t N = n_in, L = n_keep, Nh = N / 2, Lh = L / 2, Nq = Nh / 2, Lq = (Lh + 1) / 2;
    auto pe = [&](int64_t m, int64_t n) { return 0.5 * (basis_entry(m, n, N, L, 0) + basis_entry(m, N - 1 - n, N, L, 0)); };
    auto po = [&](int64_t m, int64_t n) { return 0.5 * (basis_entry(m, n, N, L, 0) - basis_entry(m, N - 1 - n, N, L, 0)); };
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < plane; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t m = i / ld, n = i % ld;
        double pee = 0.0, peo = 0.0, p_lo = 0.0, p_hi = 0.0;
        if (m < Lq && n < Nq) {
            const double a = pe(m, n), b = pe(m, Nh - 1 - n);
            pee = 0.5 * (a + b);
            peo = 0.5 * (a - b);
        }
        if (m < Lq && n < Nh) {
            p_lo = po(m, n);
            p_hi = po(Lh - 1 - m, n);
        }
        out[i] = __double2bfloat16(pee);
        out[plane + i] = __double2bfloat16(peo);
        out[2 * plane + i] = __double2bfloat16(p_lo);
        out[3 * plane + i] = __double2bfloat16(p_hi);
    }
}

// The plain orthonormal DCT-II of length N, folded the same way (power-spectrum analysis): plane 0
// holds the even rows C[2m][n], plane 1 the odd rows C[2m+1][n], n < ceil(N/2); applied to
// u_n = x_n + x_{N-1-n} and v_n = x_n - x_{N-1-n} they give the components z_2m and z_2m+1 (for odd N the
// middle column meets u = x once; the odd rows vanish there).  C[t][n] = alpha_t cos(pi t (2n+1) / (2N)),
// the phase t (2n+1) reduced exactly modulo 4N.
__global__ void build_dct_folded_kernel(__nv_bfloat16* __restrict__ out, int32_t n_in, int32_t ld, int32_t rows_pad)
{
    const int64_t plane = (int64_t)rows_pad * ld;
    const int64_t N = n_in, Nh = (N + 1) / 2;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < 2 * plane; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t eo = i / plane, j = i % plane, m = j / ld, n = j % ld, t = 2 * m + eo;
        double c = 0.0;
        if (t < N && n < Nh) {
            const int64_t k = (t * (2 * n + 1)) % (4 * N);
            c = (t == 0 ? sqrt(1.0 / (double)N) : sqrt(2.0 / (double)N)) * cospi((double)k / (double)(2 * N));
        }
        out[i] = __double2bfloat16(c);
    }
}

}  // namespace

cudaError_t launch_build_dct_folded(__nv_bfloat16* out, int32_t n_in, int32_t ld, int32_t rows_pad, cudaStream_t stream)
{
    const int64_t total = (int64_t)2 * rows_pad * ld;
    int64_t blocks = std::min<int64_t>((total + 255) / 256, 148 * 32);
    build_dct_folded_kernel<<<(unsigned)std::max<int64_t>(blocks, 1), 256, 0, stream>>>(out, n_in, ld, rows_pad);
    return cudaGetLastError();
}

cudaError_t launch_build_folded2_basis(__nv_bfloat16* out, int32_t n_in, int32_t n_keep, int32_t ld, int32_t rows_pad,
                                       cudaStream_t stream)
{
    const int64_t total = (int64_t)rows_pad * ld;
    const int64_t blocks = std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, 148 * 32));
    build_folded2_basis_kernel<<<(unsigned)blocks, 256, 0, stream>>>(out, n_in, n_keep, ld, rows_pad);
    return cudaGetLastError();
}

cudaError_t launch_build_folded_basis(__nv_bfloat16* out, int32_t n_in, int32_t n_keep, int32_t first, int32_t ld,
                                      int32_t rows_pad, cudaStream_t stream)
{
    const int64_t total = (int64_t)rows_pad * ld;
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (blocks < 1) blocks = 1;
    build_folded_basis_kernel<<<(unsigned)blocks, threads, 0, stream>>>(out, n_in, n_keep, first, ld, rows_pad);
    return cudaGetLastError();
}

cudaError_t launch_build_basis(float* p_f32, __nv_bfloat16* p_bf16, int32_t n_in, int32_t n_keep, int32_t first,
                               int32_t ld, int32_t rows_pad, cudaStream_t stream)
{
    const int64_t total = (int64_t)rows_pad * ld;
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (blocks < 1) blocks = 1;
    build_basis_kernel<<<(unsigned)blocks, threads, 0, stream>>>(p_f32, p_bf16, n_in, n_keep, first, ld, rows_pad);
    return cudaGetLastError();
}

}  // namespace freqkv
