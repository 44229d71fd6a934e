// Fast transform on the tensor cores.
//
// The compression of one channel (Section 3.3, Eq. 2-3: DCT-II of N rows, keep L components,
// L-point inverse, rescale by sqrt(L/N)) is computed the way Appendix A points to -- "the DCT can
// be computed using the FFT", O(N log N) instead of the O(L N) of a dense projection -- with the
// FFT's factors executed as small dense matrix products on the tcgen05 tensor cores:
//
//   forward, N = N1 N2     v = reordered input (v_p = x_2p, v_{N-1-p} = x_{2p+1}),  p = N2 n1 + n2
//     stage 1  (over n1)   A[t1, n2] = sum_n1 exp(-2 pi i n1 t1 / N1) v[n1, n2],   t1 <= N1/2 (real input:
//                          the other half is the conjugate)
//     twiddle              A~ = A * exp(-i pi t1 (4 n2 + 1) / (2N))          (CUDA cores, fp32)
//     stage 2  (over n2)   U_t = exp(-i pi t2 / (2 N2)) sum_n2 exp(-2 pi i n2 t2 / N2) A~[t1, n2],  t = t1 + N1 t2;
//                          the DCT components are  z_t = Re U_t  and  z_{N-t} = -Im U_t
//   keep t < L; all normalisations (orthonormal DCT and inverse, sqrt(L/N)) multiply to 2/N
//   inverse, L = L1 L2     r = Re IDFT_L(h_t exp(i pi t / (2L))) in Hermitian form, t = t1 + L1 t2, j = L2 j1 + j2
//     stage 3  (over t2)   C[t1, j2] = sum_t2 g[j2, t2] (h_{t1 + L1 t2} - i h_{L - t1 - L1 t2}),  t1 <= L1/2,
//                          g = exp(i pi t2 / (2 L2)) exp(2 pi i j2 t2 / L2) / 2
//     twiddle              C~ = C * exp(i pi t1 (4 j2 + 1) / (2L))
//     stage 4  (over t1)   r[j1, j2] = sum_t1 w_t1 Re(exp(2 pi i j1 t1 / L1) C~[t1, j2]),  y_{2j} = r_j, y_{2j+1} = r_{L-1-j}
//
// The above is the Cooley-Tukey family: any factors, complex intermediate values, a twiddle pass
// after stages 1 and 3.  Where the lengths split into coprime factors, N = N1 N2 and L = L1 L2 with
// N2, L2 odd, the prime-factor family needs neither complex values nor twiddles.  A DCT sum over the
// odd numbers m = 2n + 1 modulo 4N, cos(2 pi m k / (4N)), separates by the Chinese remainder theorem
// into residues modulo 4 N1 and modulo N2:
//     z_k = sigma(k) D[c(k), e(k)],   D[c, e] = sum_{n1, b} x[n1, b] cos(pi (2 n1 + 1) c / (2 N1) + 2 pi b e / N2),
// (n1, b) a permutation of the rows (m or its mirror 4N - m reduced to 1 <= m mod 4 N1 < 2 N1), c in
// [0, N1], e modulo N2, sigma a sign.  cos(theta + phi) = cos cos - sin sin makes it two real stages:
//     stage 1  (over b)    Pc[e, n1] = sum_b cos(2 pi b e / N2) x[n1, b],  Ps[e, n1] likewise with sin,  0 <= e <= (N2 - 1) / 2
//     stage 2  (over n1)   D[c, +-e] = sum_n1 cos(theta) Pc[e, n1] -+ sin(theta) Ps[e, n1]      (rows (c, +) and (c, -))
// and the L-point inverse is the same sum with the roles of input and output exchanged:
//     stage 3  (over e')   P'c[b, c'] = sum_e' cos(2 pi b e' / L2) H[c', e'],  P's likewise,   H = the retained z_k (k = 0 halved),
//                          signed and placed by the residues of k modulo 4 L1 and L2
//     stage 4  (over c')   y[j1, +-b] = sum_c' cos(theta') P'c[b, c'] -+ sin(theta') P's[b, c']
// Between the stages the values are only rounded and moved; the pass after stage 2 places each
// retained component by a host-built table (destination, sign).
//
// Each stage is D = F B with F a real matrix of at most 128 rows (the real and imaginary parts of
// a complex stage are separate rows) and B the data: contraction index down the rows, (outer
// index, channel) along the columns.  Work is cut into slabs of one matrix x 8 channels (one
// 16-byte piece of every row): a slab's N x 8 values stay in shared memory through all four
// stages and its L output rows are written over its own input rows, so the transform is in place
// in global memory with no scratch -- no other CTA touches those channels.
//
// One persistent CTA per SM:
//   warps 0-15  after every stage move the accumulators from tensor memory to the next stage's
//               operand in shared memory (twiddle, round to bf16, re-index) or, after stage 4, to
//               the cache; warp w works on TMEM lanes 32 (w % 4) .. +31 and on 64-column group
//               w / 4 of every chunk;
//   warp 16     issues the tcgen05.mma instructions (M 128, N up to 256, K 16; bf16 in, fp32 out)
//               of one 256-column chunk at a time into one of two halves of tensor memory, so
//               that the products of a chunk overlap the movement of the previous one;
//   warps 17-24 load: cp.async, each 16-byte piece of a row placed where stage 1 wants it (table
//               built on the host).  The next slab's copies are issued as soon as stage 3 has
//               consumed the buffer they go to and run while the other warps finish the slab.
//               (A warp keeps about one such instruction of 32 scattered pieces in flight, so the
//               number of loading warps sets the load rate: the 16 moving warps doing it
//               themselves cost them 5 k cycles per slab, four loading warps were too few.)
// The four matrices F stay resident in shared memory (copied once per CTA from a pre-swizzled
// image).  Two data buffers alternate between stages.  Every barrier wait is bounded in time.
#include <cuda.h>

#include <algorithm>
#include <cmath>
#include <cstring>

#include "dctmm.cuh"

namespace freqkv {
namespace {

constexpr int EPI_WARPS = 16;                // four per TMEM lane quarter: one atom of a chunk each
constexpr int EPI_THREADS = EPI_WARPS * 32;
constexpr int LOAD_WARPS = 8;                // warps that only load the next slab
constexpr int LOAD_THREADS = LOAD_WARPS * 32;
constexpr int THREADS = EPI_THREADS + 32 + LOAD_THREADS;
constexpr int CHUNK_ATOMS = 4;                 // 4 x 64 columns = N 256 per instruction
constexpr int TMEM_COLS = 512;
constexpr int SMEM_LIMIT = 232448 - 1024;      // opt-in maximum minus alignment slack
constexpr int MAX_N = 4608;                  // rows of a transform (what shared memory can hold at all)

struct DctmmParams {
    DctmmPlan plan;
    // prime-factor output map: row (j1, +-) and column b of stage 4 hold token j with
    // 2j + 1 or its mirror = ((2 j1 + 1) out_a +- b out_w) mod 4L
    int32_t out_a, out_w;
    int32_t sink, slabs_per_matrix, total_slabs;
    int32_t* status;
    unsigned long long wait_limit_ns;
};

// ---------------------------------------------------------------------------------- device helpers

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
// The same, but the thread may be suspended for up to `hint_ns` while the phase is incomplete
// (it is woken when the phase completes): a waiting warp then leaves the issue slots to the others.
__device__ __forceinline__ bool mbar_try_wait_suspend(uint32_t bar, uint32_t parity, uint32_t hint_ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Wait for the phase with the given parity; gives up when another thread has raised the abort
// flag or after limit_ns (then it sets the status bit and raises the flag).  False = gave up.
// The global timer is read rarely: its reads are slow and many warps wait at once.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          unsigned long long limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait_suspend(bar, parity, 20000u)) return true;
        if ((spins & 63u) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns) {
                atomicOr(status, DCTMM_ERR_WAIT);
                *abort_flag = 1;
                __threadfence_block();
                return false;
            }
        }
    }
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
// Instruction descriptor, kind::f16: D fp32, A and B bf16, A K-major, B MN-major, M = 128, N = n.
__device__ __forceinline__ uint32_t idesc_for(uint32_t n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 16 consecutive columns, issued without waiting; the registers may be read only after
// tmem_ld_wait16 on the same array (which names them as operands, so that no use is scheduled before it).
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&u)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
          "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait16(uint32_t (&u)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(u[0]), "+r"(u[1]), "+r"(u[2]), "+r"(u[3]), "+r"(u[4]), "+r"(u[5]), "+r"(u[6]), "+r"(u[7]), "+r"(u[8]),
                   "+r"(u[9]), "+r"(u[10]), "+r"(u[11]), "+r"(u[12]), "+r"(u[13]), "+r"(u[14]), "+r"(u[15])
                 :
                 : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint4 pack8(const float* v)
{
    return make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
__device__ __forceinline__ uint4 pack8u(const uint32_t* u)
{
    return make_uint4(pack_bf16(__uint_as_float(u[0]), __uint_as_float(u[1])), pack_bf16(__uint_as_float(u[2]), __uint_as_float(u[3])),
                      pack_bf16(__uint_as_float(u[4]), __uint_as_float(u[5])), pack_bf16(__uint_as_float(u[6]), __uint_as_float(u[7])));
}
__device__ __forceinline__ void st_shared_16(uint32_t addr, const uint4& v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// Byte offset, inside a stage's B buffer, of the 16-byte piece (contraction index k, outer index o):
// 64-column groups ("atoms", 8 outer values x 8 channels) are k_pad rows of 128 bytes each; the
// eight pieces of a row are permuted by the row number (128-byte swizzle).
__host__ __device__ __forceinline__ uint32_t b_piece(uint32_t k, uint32_t o, uint32_t k_pad)
{
    return (o >> 3) * (k_pad * 128u) + k * 128u + (((o & 7u) ^ (k & 7u)) << 4);
}

// cos and sin of pi * num / den for integers 0 <= num < 2 den.
__device__ __forceinline__ void sincos_ratio(int32_t num, int32_t den, float* s, float* c)
{
    sincospif((float)num / (float)den, s, c);
}

// ---------------------------------------------------------------------------------- the kernel

template <int FAMILY>
__global__ void __launch_bounds__(THREADS, 1) freqkv_dctmm_kernel(const CacheView view, const DctmmParams prm)
{
    constexpr bool PF = FAMILY == DCTMM_PRIME_FACTOR;
    extern __shared__ uint8_t smem_raw[];
    const DctmmPlan& P = prm.plan;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* aligned = smem_raw + (base - raw);
    // barriers: ready[0..3] (stage s operand complete), acc_full[0..1], acc_empty[0..1], x_free (every
    // product of stage 3 has read its operand: the buffer it shares with stage 1's takes the next slab)
    const uint32_t bar0 = base + P.bar_off;
    auto ready_bar = [&](int s) { return bar0 + 8u * s; };
    auto full_bar = [&](int b) { return bar0 + 8u * (4 + b); };
    auto empty_bar = [&](int b) { return bar0 + 8u * (6 + b); };
    const uint32_t x_free_bar = bar0 + 8u * 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aligned + P.bar_off + 96);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

    if (threadIdx.x == 0) {
        mbar_init(ready_bar(0), LOAD_THREADS);
        for (int s = 1; s < 4; ++s) mbar_init(ready_bar(s), EPI_THREADS);
        mbar_init(x_free_bar, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(full_bar(b), 1);
            mbar_init(empty_bar(b), EPI_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == EPI_WARPS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    // the matrices F and the destination table of the second pass: plain copies of the host-built
    // image; both data buffers start as zeros (never-written padding must not hold NaN bit
    // patterns: it meets zero entries of F)
    {
        const uint4* img = static_cast<const uint4*>(P.image);
        uint4* dst = reinterpret_cast<uint4*>(aligned);
        const int32_t n_f = P.f_bytes / 16, n_data = P.tab_off / 16, n_tab = P.tab_bytes / 16;  // table: rows, then the zero list
        for (int32_t i = threadIdx.x; i < n_f; i += THREADS) dst[i] = img[i];
        for (int32_t i = n_f + threadIdx.x; i < n_data; i += THREADS) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        for (int32_t i = threadIdx.x; i < n_tab; i += THREADS) dst[n_data + i] = img[n_f + i];
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const int32_t n_iter = prm.total_slabs > (int32_t)blockIdx.x
                               ? (prm.total_slabs - (int32_t)blockIdx.x + (int32_t)gridDim.x - 1) / (int32_t)gridDim.x
                               : 0;

    if (warp == EPI_WARPS) {
        // ------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            uint32_t q = 0;  // chunk counter: tensor-memory half q & 1
            bool alive = true;
            for (int32_t it = 0; it < n_iter && alive; ++it) {
                for (int s = 0; s < 4 && alive; ++s) {
                    const DctmmStage& st = P.st[s];
                    if (!mbar_wait(ready_bar(s), it & 1, abort_flag, prm.status, prm.wait_limit_ns)) {
                        alive = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t b_base = base + st.b_off, lbo = (uint32_t)st.k_pad * 128u;
                    const int32_t k_steps = st.k_pad / 16;
                    for (int32_t a0 = 0; a0 < st.atoms; a0 += CHUNK_ATOMS, ++q) {
                        const uint32_t buf = q & 1u;
                        if (q >= 2 && !mbar_wait(empty_bar(buf), ((q >> 1) - 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) {
                            alive = false;
                            break;
                        }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t n_atoms = (uint32_t)min(CHUNK_ATOMS, st.atoms - a0);
                        const uint32_t idesc = idesc_for(64u * n_atoms);
                        for (int32_t ks = 0; ks < k_steps; ++ks) {
                            const uint64_t ad = smem_desc(base + (uint32_t)st.a_tile[ks >> 2] + (uint32_t)(ks & 3) * 32u, 16, 1024);
                            const uint64_t bd = smem_desc(b_base + (uint32_t)a0 * lbo + (uint32_t)ks * 2048u, lbo, 1024);
                            umma(tmem_base + buf * 256u, ad, bd, idesc, ks != 0);
                        }
                        umma_commit(full_bar(buf));
                        if (s == 2 && a0 + CHUNK_ATOMS >= st.atoms) umma_commit(x_free_bar);
                    }
                }
            }
            if (*abort_flag) {  // products may still be in flight: let them finish before tensor memory is freed
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 1000000ull) __nanosleep(1000);
            }
        }
    } else if (warp > EPI_WARPS) {
        // ------------------------------------------------------------ loading warps
        // Row n of the slab goes, as one 16-byte piece, where stage 1 contracts it (host-built table of
        // piece numbers).  The copies of a slab are issued as soon as stage 3 of the slab before has read
        // the buffer, and run while the other warps finish that slab.
        const int ltid = threadIdx.x - (EPI_THREADS + 32);
        const int32_t N = P.n_in;
        const int64_t row_bytes = view.stride_token * 2;
        const uint16_t* load_tab = reinterpret_cast<const uint16_t*>(static_cast<const uint8_t*>(P.image) + P.f_bytes + P.tab_bytes);
        const DctmmStage& st0 = P.st[0];
        const uint32_t x_base = base + st0.b_off;
        for (int32_t it = 0; it < n_iter; ++it) {
            const int32_t slab = (int32_t)blockIdx.x + it * (int32_t)gridDim.x;
            if (it > 0 && !mbar_wait(x_free_bar, (it - 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) break;
            const int32_t mat = slab / prm.slabs_per_matrix, piece = slab - mat * prm.slabs_per_matrix;
            const int32_t tensor = mat / view.mats_per_tensor;
            const char* src = static_cast<const char*>(tensor_base(view, tensor)) +
                              (matrix_offset(view, mat - tensor * view.mats_per_tensor) + (int64_t)prm.sink * view.stride_token) * 2 + piece * 16;
            for (int32_t n0 = ltid; n0 < N; n0 += 4 * LOAD_THREADS) {
                uint32_t dst[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[j] = n0 + j * LOAD_THREADS < N ? __ldg(load_tab + n0 + j * LOAD_THREADS) : 0u;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (n0 + j * LOAD_THREADS < N) cp_async_16(x_base + dst[j] * 16u, src + (int64_t)(n0 + j * LOAD_THREADS) * row_bytes);
            }
            // rows k .. k_pad-1 of the operand are contraction padding: zero for every outer value
            for (int32_t i = ltid; i < (st0.k_pad - st0.k) * st0.atoms * 8; i += LOAD_THREADS) {
                const int32_t k = st0.k + i / (st0.atoms * 8), o = i % (st0.atoms * 8);
                st_shared_16(x_base + b_piece((uint32_t)k, (uint32_t)o, (uint32_t)st0.k_pad), make_uint4(0u, 0u, 0u, 0u));
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(ready_bar(0));
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else {
        // ------------------------------------------------------------ move / store warps
        const int tid = threadIdx.x;            // 0 .. EPI_THREADS - 1
        const int quarter = warp & 3, group = warp >> 2;  // group g takes atom g of every 4-atom chunk
        const int row = quarter * 32 + lane;    // TMEM lane = row of D this thread reads
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int32_t N = P.n_in, L = P.n_keep, L2 = P.l2, T1 = P.t1;
        const int ri = (row >> 4) & 1;                       // stages 1 and 3: rows 16..31 of a warp are imaginary parts
        const int32_t cidx = (row >> 5) * 16 + (row & 15);   // t1 (stage 1) or j2 (stage 3) of this row
        const int32_t hL = (L + 1) / 2;
        const int64_t row_bytes = view.stride_token * 2;

        // Twiddles of the two complex passes, by recurrence: this thread's value at the first outer
        // index of its first atom (o = 8 * group), the factor from o to o + 1, and the factor over
        // the 24 outer values of the other groups' atoms in between.
        // stage 1: exp(-i pi t1 (4 o + 1) / (2N));  stage 3: exp(+i pi (4 j2 + 1) o / (2L)).
        float2 tw_start[2], tw_step1[2], tw_jump[2];
        uint32_t swz[4];  // stages 1, 3 write row k = 2 o + ri, piece cidx % 8 of its atom: the swizzled piece for o % 4 = j
#pragma unroll
        for (int j = 0; j < 4; ++j) swz[j] = ((((uint32_t)cidx & 7u) ^ ((uint32_t)(2 * j + ri) & 7u)) << 4) + (uint32_t)ri * 128u;
#pragma unroll
        for (int i = 0; i < 2 && !PF; ++i) {
            const int32_t den = i == 0 ? 2 * N : 2 * L;         // angles are pi * num / den, num taken modulo 2 den
            const int32_t fac = i == 0 ? cidx : 4 * cidx + 1;   // the row's own factor of the phase
            const int32_t per_o = i == 0 ? 4 : 1;               // phase units per step of o
            const int32_t first = i == 0 ? 4 * (8 * group) + 1 : 8 * group;
            auto unit = [&](int32_t mult) {
                float sn, cs;
                sincos_ratio((int32_t)(((int64_t)fac * mult) % (2 * den)), den, &sn, &cs);
                return make_float2(cs, i == 0 ? -sn : sn);
            };
            tw_start[i] = unit(first);
            tw_step1[i] = unit(per_o);
            tw_jump[i] = unit(24 * per_o);
        }
        const bool row2_ok = row < P.rows2;  // rows of stage 2 that exist: the table has no others
        const uint32_t* dest_tab = reinterpret_cast<const uint32_t*>(aligned + P.tab_off) + (row2_ok ? row : 0) * (P.st[1].atoms * 8);
        // prime-factor family: 16-bit entries (piece number, bit 13 = negate, bit 14 = halve, 0xffff = nowhere),
        // and after the rows the numbers of the pieces of stage 3's operand that stay zero
        const uint16_t* dest_tab16 = reinterpret_cast<const uint16_t*>(aligned + P.tab_off) + (row2_ok ? row : 0) * (P.st[1].atoms * 8);
        const uint16_t* zero_list = reinterpret_cast<const uint16_t*>(aligned + P.tab_off) + P.rows2 * (P.st[1].atoms * 8);
        // prime-factor output map: this row's odd number m at the first column of its first atom, its
        // change per column (+- out_w) and over the 24 columns of the other groups' atoms, all modulo 4L
        int32_t out_first = 0, out_step = 0, out_jump = 0;
        if (PF) {
            const int64_t L4 = 4 * (int64_t)L;
            const int64_t a0 = ((int64_t)(2 * (row >> 1) + 1) * prm.out_a) % L4;
            out_step = (row & 1) ? (int32_t)(L4 - prm.out_w) : prm.out_w;
            out_first = (int32_t)((a0 + (int64_t)out_step * (8 * group)) % L4);
            out_jump = (int32_t)(((int64_t)out_step * 24) % L4);
        }

        auto slab_base = [&](int32_t slab) -> char* {
            const int32_t mat = slab / prm.slabs_per_matrix, piece = slab - mat * prm.slabs_per_matrix;
            const int32_t tensor = mat / view.mats_per_tensor;
            return static_cast<char*>(tensor_base(view, tensor)) +
                   (matrix_offset(view, mat - tensor * view.mats_per_tensor) + (int64_t)prm.sink * view.stride_token) * 2 +
                   piece * 16;
        };
        // Rows k .. k_pad-1 of a B buffer are contraction padding: zero for every outer value
        // (thread: outer value tid % 64, rows tid / 64, + 8, ...; at most 64 outer values per buffer...)
        auto zero_pad_rows = [&](const DctmmStage& st) {
            const int32_t cols = st.atoms * 8;
            const uint32_t dst = base + st.b_off;
            for (int32_t o = tid & 63; o < cols; o += 64)
                for (int32_t k = st.k + (tid >> 6); k < st.k_pad; k += EPI_THREADS / 64)
                    st_shared_16(dst + b_piece((uint32_t)k, (uint32_t)o, (uint32_t)st.k_pad), make_uint4(0u, 0u, 0u, 0u));
        };

        uint32_t q = 0;
        bool alive = true;
        for (int32_t it = 0; it < n_iter && alive; ++it) {
            const int32_t slab = (int32_t)blockIdx.x + it * (int32_t)gridDim.x;
            char* cur_base = slab_base(slab);

            for (int s = 0; s < 4 && alive; ++s) {
                const DctmmStage& st = P.st[s];
                const DctmmStage& nx = P.st[(s + 1) & 3];
                const uint32_t nb = base + nx.b_off, nk_pad = (uint32_t)nx.k_pad;
                if (s < 3) zero_pad_rows(nx);
                if (PF && s == 1)
                    for (int32_t i = tid; i < P.n_zero; i += EPI_THREADS) st_shared_16(nb + (uint32_t)zero_list[i] * 16u, make_uint4(0u, 0u, 0u, 0u));
                int32_t out_m = out_first;
                const bool quarter_active = quarter * 32 < st.rows;  // rows past the stage's own are never read
                float wr = tw_start[s >> 1].x, wi = tw_start[s >> 1].y;
                for (int32_t a0 = 0; a0 < st.atoms && alive; a0 += CHUNK_ATOMS, ++q) {
                    const uint32_t buf = q & 1u;
                    if (!mbar_wait(full_bar(buf), (q >> 1) & 1, abort_flag, prm.status, prm.wait_limit_ns)) {
                        alive = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if (quarter_active && a0 + group < st.atoms) {
                        const uint32_t taddr = lane_taddr + buf * 256u + (uint32_t)(group * 64);
                        const int32_t o_atom = (a0 + group) * 8;  // first outer value of this thread's atom
                        // The atom's 64 columns come out of tensor memory 16 at a time (two outer values);
                        // the load of the next 16 is in flight while these are worked on.
                        uint32_t ua[16], ub[16];
                        tmem_ld16_issue(taddr, ua);
                        if (PF && (s == 0 || s == 2)) {
                            // rows are cosine sums (index e = row) then sine sums (e = row - rows / 2) of the
                            // contracted index; the next stage contracts (part, this stage's outer index) for outer e
                            const int32_t half_rows = st.rows >> 1;
                            const int32_t sine = row >= half_rows ? 1 : 0;
                            const uint32_t e = (uint32_t)(row - sine * half_rows), e7 = e & 7u;
                            const uint32_t k0 = (uint32_t)(sine * st.outer + o_atom);
                            const uint32_t dst0 = nb + (e >> 3) * (nk_pad * 128u);
                            const bool mine = row < st.rows;
#pragma unroll
                            for (int part = 0; part < 4; ++part) {
                                uint32_t(&u)[16] = (part & 1) ? ub : ua;
                                tmem_ld_wait16(u);
                                if (part < 3) tmem_ld16_issue(taddr + (part + 1) * 16, (part & 1) ? ua : ub);
#pragma unroll
                                for (int jj = 0; jj < 2; ++jj) {
                                    const uint32_t k = k0 + (uint32_t)(part * 2 + jj);
                                    if (mine && o_atom + part * 2 + jj < st.outer)
                                        st_shared_16(dst0 + (k << 7) + (((e7 ^ k) & 7u) << 4), pack8u(&u[jj * 8]));
                                }
                            }
                        } else if (s == 0 || s == 2) {
                            // complex twiddle: this row holds one part, the row 16 lanes away the other
                            const int32_t count = (s == 0) ? T1 : L2;
                            const float sr = tw_step1[s >> 1].x, si = tw_step1[s >> 1].y;
                            const bool mine = cidx < count;
                            const uint32_t dst0 = nb + ((uint32_t)cidx >> 3) * (nk_pad * 128u) + (uint32_t)o_atom * 256u;
#pragma unroll
                            for (int part = 0; part < 4; ++part) {
                                uint32_t(&u)[16] = (part & 1) ? ub : ua;
                                tmem_ld_wait16(u);
                                if (part < 3) tmem_ld16_issue(taddr + (part + 1) * 16, (part & 1) ? ua : ub);
#pragma unroll
                                for (int jj = 0; jj < 2; ++jj) {
                                    const int j = (part & 1) * 2 + jj;  // o % 4
                                    float out[8];
                                    const float swi = ri ? wi : -wi;
#pragma unroll
                                    for (int c = 0; c < 8; ++c) {
                                        const float val = __uint_as_float(u[jj * 8 + c]);
                                        const float other = __shfl_xor_sync(0xffffffffu, val, 16);
                                        out[c] = fmaf(val, wr, other * swi);
                                    }
                                    if (mine && o_atom + part * 2 + jj < st.outer)
                                        st_shared_16(dst0 + (uint32_t)(part * 2 + jj) * 256u + swz[j], pack8(out));
                                    const float nr = fmaf(wr, sr, -wi * si), ni = fmaf(wr, si, wi * sr);
                                    wr = nr;
                                    wi = ni;
                                }
                            }
                            {   // now at o_atom + 8: skip the other groups' atoms, on to o_atom + 32
                                const float jr = tw_jump[s >> 1].x, ji = tw_jump[s >> 1].y;
                                const float nr = fmaf(wr, jr, -wi * ji), ni = fmaf(wr, ji, wi * jr);
                                wr = nr;
                                wi = ni;
                            }
                        } else if (PF && s == 1) {
                            // a retained component goes, signed, to the one place where stage 3 contracts it
#pragma unroll
                            for (int part = 0; part < 4; ++part) {
                                uint32_t(&u)[16] = (part & 1) ? ub : ua;
                                tmem_ld_wait16(u);
                                if (part < 3) tmem_ld16_issue(taddr + (part + 1) * 16, (part & 1) ? ua : ub);
                                const uint32_t dd = *reinterpret_cast<const uint32_t*>(dest_tab16 + o_atom + part * 2);
#pragma unroll
                                for (int jj = 0; jj < 2; ++jj) {
                                    const uint32_t ent = jj ? dd >> 16 : dd & 0xffffu;
                                    if (row2_ok && ent != 0xffffu) {
                                        uint4 val;
                                        if (ent & 0x4000u) {
                                            float half[8];
#pragma unroll
                                            for (int c = 0; c < 8; ++c) half[c] = 0.5f * __uint_as_float(u[jj * 8 + c]);
                                            val = pack8(half);
                                        } else {
                                            val = pack8u(&u[jj * 8]);
                                        }
                                        const uint32_t flip = (ent & 0x2000u) ? 0x80008000u : 0u;
                                        val.x ^= flip;
                                        val.y ^= flip;
                                        val.z ^= flip;
                                        val.w ^= flip;
                                        st_shared_16(nb + (ent & 0x1fffu) * 16u, val);
                                    }
                                }
                            }
                        } else if (s == 1) {
                            // retained spectrum values go where stage 3 contracts them: up to two places
                            // each, from the host-built table (16-bit piece numbers, 0xffff = nowhere)
#pragma unroll
                            for (int part = 0; part < 4; ++part) {
                                uint32_t(&u)[16] = (part & 1) ? ub : ua;
                                tmem_ld_wait16(u);
                                if (part < 3) tmem_ld16_issue(taddr + (part + 1) * 16, (part & 1) ? ua : ub);
                                const uint2 dd = *reinterpret_cast<const uint2*>(dest_tab + o_atom + part * 2);
                                const uint32_t d[2] = {dd.x, dd.y};
#pragma unroll
                                for (int jj = 0; jj < 2; ++jj) {
                                    const uint32_t da = d[jj] & 0xffffu, db = d[jj] >> 16;
                                    if (row2_ok && d[jj] != 0xffffffffu) {
                                        const uint4 val = pack8u(&u[jj * 8]);
                                        if (da != 0xffffu) st_shared_16(nb + da * 16u, val);
                                        if (db != 0xffffu) st_shared_16(nb + db * 16u, val);
                                    }
                                }
                            }
                            // h_L = 0: the partner of component 0 in the Hermitian form
                            if (row == 0 && o_atom == 0) st_shared_16(nb + b_piece((uint32_t)L2, 0u, nk_pad), make_uint4(0u, 0u, 0u, 0u));
                        } else if (PF) {
                            // output rows: row (j1, +-) and column b hold the token whose odd number 2j + 1, or
                            // its mirror 4L - (2j + 1), is out_m; (j1, -) at b = 0 repeats (j1, +)
                            const int32_t L4 = 4 * L;
#pragma unroll
                            for (int part = 0; part < 4; ++part) {
                                uint32_t(&u)[16] = (part & 1) ? ub : ua;
                                tmem_ld_wait16(u);
                                if (part < 3) tmem_ld16_issue(taddr + (part + 1) * 16, (part & 1) ? ua : ub);
#pragma unroll
                                for (int jj = 0; jj < 2; ++jj) {
                                    const int32_t o = o_atom + part * 2 + jj;
                                    if (row < st.rows && o < st.outer && !((row & 1) && o == 0)) {
                                        const int32_t j_out = (out_m < 2 * L ? out_m - 1 : L4 - out_m - 1) >> 1;
                                        *reinterpret_cast<uint4*>(cur_base + (int64_t)j_out * row_bytes) = pack8u(&u[jj * 8]);
                                    }
                                    out_m += out_step;
                                    if (out_m >= L4) out_m -= L4;
                                }
                            }
                            out_m += out_jump;
                            if (out_m >= L4) out_m -= L4;
                        } else {
                            // output rows: r_j = y_2j for j < ceil(L/2), r_{L-1-j} = y_{2j+1}
#pragma unroll
                            for (int part = 0; part < 4; ++part) {
                                uint32_t(&u)[16] = (part & 1) ? ub : ua;
                                tmem_ld_wait16(u);
                                if (part < 3) tmem_ld16_issue(taddr + (part + 1) * 16, (part & 1) ? ua : ub);
                                if (row < P.l1) {
#pragma unroll
                                    for (int jj = 0; jj < 2; ++jj) {
                                        const int32_t o = o_atom + part * 2 + jj;
                                        if (o < L2) {
                                            const int32_t j_out = L2 * row + o;
                                            const int32_t m = j_out < hL ? 2 * j_out : 2 * (L - 1 - j_out) + 1;
                                            *reinterpret_cast<uint4*>(cur_base + (int64_t)m * row_bytes) = pack8u(&u[jj * 8]);
                                        }
                                    }
                                }
                            }
                        }
                    }
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_bar(buf));
                }
                if (s < 3 && alive) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_arrive(ready_bar(s + 1));
                }
            }
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == EPI_WARPS) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS));
    }
}

// ---------------------------------------------------------------------------------- host side

inline int32_t round_up(int32_t x, int32_t m) { return (x + m - 1) / m * m; }

uint16_t to_bf16(double x)
{
    const float f = (float)x;
    uint32_t u;
    std::memcpy(&u, &f, 4);
    const uint32_t rounded = u + 0x7fffu + ((u >> 16) & 1u);  // nearest even (inputs are finite)
    return (uint16_t)(rounded >> 16);
}

int64_t gcd64(int64_t a, int64_t b)
{
    while (b) {
        const int64_t t = a % b;
        a = b;
        b = t;
    }
    return a;
}
// x with a x = 1 (mod m), for coprime a and m (m small: by search over the residues)
int64_t inverse_mod(int64_t a, int64_t m)
{
    if (m == 1) return 0;
    a %= m;
    for (int64_t x = 1; x < m; ++x)
        if (a * x % m == 1) return x;
    return 0;
}

// Shared-memory layout common to both families, from the stages' k, rows and outer counts: the
// matrices F as 64-wide tiles of 128-byte rows (a last tile narrower than 64 may share its rows
// with another stage's: each takes its own byte columns), two data buffers, the table, the
// barriers.  False when a limit is exceeded.
bool layout_plan(DctmmPlan* p, const int32_t k[4], const int32_t rows[4], const int32_t outer[4], int32_t tab_bytes)
{
    int32_t off = 0, b_bytes[4];
    for (int s = 0; s < 4; ++s) {
        DctmmStage& st = p->st[s];
        if (rows[s] < 1 || rows[s] > 128 || outer[s] < 1 || k[s] < 1) return false;
        st.k = k[s];
        st.k_pad = round_up(k[s], 16);
        if (st.k_pad > 64 * 8) return false;
        st.rows = rows[s];
        st.rows8 = round_up(rows[s], 8);
        st.outer = outer[s];
        st.atoms = (outer[s] + 7) / 8;
        for (int t = 0; t < 8; ++t) st.a_tile[t] = 0;
        for (int t = 0; t < st.k_pad / 64; ++t) {
            st.a_tile[t] = off;
            off += st.rows8 * 128;
        }
        b_bytes[s] = st.atoms * st.k_pad * 128;
    }
    // the narrow last tiles, widest first, each into the first shared tile with room
    struct Shared { int32_t off, used, rows8; };
    std::vector<Shared> shared;
    int order[4] = {0, 1, 2, 3};
    std::stable_sort(order, order + 4, [&](int a, int b) { return p->st[a].k_pad % 64 > p->st[b].k_pad % 64; });
    std::vector<std::pair<int, int>> placed;  // (stage, shared tile)
    for (int idx = 0; idx < 4; ++idx) {
        const int s = order[idx];
        const int32_t bytes = (p->st[s].k_pad % 64) * 2;
        if (bytes == 0) continue;
        size_t t = 0;
        while (t < shared.size() && shared[t].used + bytes > 128) ++t;
        if (t == shared.size()) shared.push_back({0, 0, 0});
        p->st[s].a_tile[p->st[s].k_pad / 64] = shared[t].used;  // byte column for now; the tile's offset is added below
        shared[t].used += bytes;
        shared[t].rows8 = std::max(shared[t].rows8, p->st[s].rows8);
        placed.push_back({s, (int)t});
    }
    for (Shared& t : shared) {
        t.off = off;
        off += t.rows8 * 128;
    }
    for (const auto& pl : placed) p->st[pl.first].a_tile[p->st[pl.first].k_pad / 64] += shared[pl.second].off;
    p->f_bytes = off;
    const int32_t x = std::max(b_bytes[0], b_bytes[2]), y = std::max(b_bytes[1], b_bytes[3]);
    p->st[0].b_off = p->st[2].b_off = off;
    p->st[1].b_off = p->st[3].b_off = off + x;
    // an instruction reads 128 rows of a tile of F whatever `rows` is: keep that inside the allocation
    p->bar_off = std::max(off + x + y, off + 128 * 128);
    p->tab_off = round_up(p->bar_off, 16);
    p->tab_bytes = round_up(tab_bytes, 16);
    p->bar_off = p->tab_off + p->tab_bytes;
    p->smem_bytes = p->bar_off + 128 + 1024;  // barriers, tensor-memory slot, abort flag; alignment slack
    return p->smem_bytes <= SMEM_LIMIT;
}

// Cooley-Tukey family: stage shapes of one factor choice; false when a limit is exceeded.
bool shape_plan(int32_t N, int32_t L, int32_t n1, int32_t n2, int32_t l1, int32_t l2, DctmmPlan* p, std::vector<DctmmRow2>* rows2)
{
    const int32_t t1 = n1 / 2 + 1, t3 = l1 / 2 + 1;
    if (t1 > 64 || l2 > 64 || l1 > 128) return false;
    // stage-2 rows: real parts (t = t1 + n1 t2 < L) and negated imaginary parts (t = N - t1 - n1 t2 < L,
    // only for t1 whose mirror is not computed as a real part: 1 <= t1 < ceil(n1 / 2))
    rows2->clear();
    for (int32_t t2 = 0; t2 < n2 && n1 * t2 < L; ++t2) rows2->push_back({n1 * t2, +1, 0, std::min(t1, L - n1 * t2)});
    const int32_t hi = (n1 + 1) / 2;
    for (int32_t t2 = 0; t2 < n2; ++t2) {
        const int32_t lo = std::max(1, N - n1 * t2 - L + 1);
        if (lo < hi) rows2->push_back({N - n1 * t2, -1, lo, hi});
    }
    if ((int32_t)rows2->size() > 128 || rows2->empty()) return false;
    *p = DctmmPlan();
    p->family = DCTMM_COOLEY_TUKEY;
    p->n_in = N; p->n_keep = L; p->n1 = n1; p->n2 = n2; p->l1 = l1; p->l2 = l2; p->t1 = t1; p->t3 = t3;
    p->rows2 = (int32_t)rows2->size();
    const int32_t k[4] = {n1, 2 * n2, 2 * l2, 2 * t3};
    const int32_t rows[4] = {32 * ((t1 + 15) / 16), p->rows2, 32 * ((l2 + 15) / 16), l1};
    const int32_t outer[4] = {n2, t1, t3, l2};
    // destination table of the second pass: one 32-bit entry per (row, outer value of stage 2)
    return layout_plan(p, k, rows, outer, p->rows2 * ((t1 + 7) / 8) * 8 * 4);
}

// Prime-factor family: N = n1 n2 and L = l1 l2 with 4 n1, n2 coprime and 4 l1, l2 coprime.
bool shape_plan_pf(int32_t N, int32_t L, int32_t n1, int32_t n2, int32_t l1, int32_t l2, DctmmPlan* p)
{
    if (n2 < 3 || l2 < 3 || gcd64(4 * (int64_t)n1, n2) != 1 || gcd64(4 * (int64_t)l1, l2) != 1) return false;
    const int32_t h = (n2 - 1) / 2, hl = (l2 - 1) / 2;
    if (n1 > 64 || h + 1 > 64 || l1 + 1 > 64 || hl + 1 > 64) return false;
    *p = DctmmPlan();
    p->family = DCTMM_PRIME_FACTOR;
    p->n_in = N; p->n_keep = L; p->n1 = n1; p->n2 = n2; p->l1 = l1; p->l2 = l2;
    p->rows2 = 2 * (n1 + 1);
    p->n_zero = l2 * (l1 + 1) - L;
    const int32_t k[4] = {n2, 2 * n1, l2, 2 * (l1 + 1)};
    const int32_t rows[4] = {2 * (h + 1), 2 * (n1 + 1), 2 * (hl + 1), 2 * l1};
    const int32_t outer[4] = {n1, h + 1, l1 + 1, hl + 1};
    if (!layout_plan(p, k, rows, outer, (p->rows2 * ((h + 1 + 7) / 8) * 8 + p->n_zero) * 2)) return false;
    // 13 bits of a table entry number the 16-byte pieces of stage 3's operand
    return p->st[2].atoms * p->st[2].k_pad * 8 <= 0x2000;
}

// Rough cycles per slab of a factor choice: 2 k_pad per 64-column atom on the tensor pipe, about
// 20 per outer value in the passes that move the accumulators.  (Measured on B200, the Cooley-Tukey
// choices that fit shared memory for 4092 -> 2046 and 4096 -> 2048 all land within 4 % of each other.)
int64_t plan_cost(const DctmmPlan& p)
{
    int64_t c = 0;
    for (int s = 0; s < 4; ++s) c += 2 * (int64_t)p.st[s].k_pad * p.st[s].atoms + 20 * (int64_t)p.st[s].outer;
    return c;
}

std::vector<int32_t> divisors(int32_t n)
{
    std::vector<int32_t> d;
    for (int32_t i = 1; (int64_t)i * i <= n; ++i)
        if (n % i == 0) {
            d.push_back(i);
            if (i != n / i) d.push_back(n / i);
        }
    std::sort(d.begin(), d.end());
    return d;
}

// The cheapest factor choice of the family that meets every limit; false if there is none.
bool choose_factors(int32_t N, int32_t L, int32_t family, DctmmPlan* plan, std::vector<DctmmRow2>* rows2_out)
{
    if (N < 16 || N > MAX_N || L < 2 || L >= N) return false;
    int64_t best = -1;
    DctmmPlan cand;
    std::vector<DctmmRow2> rows2;
    const std::vector<int32_t> dn = divisors(N), dl = divisors(L);
    for (int32_t n1 : dn) {
        if (family == DCTMM_COOLEY_TUKEY && n1 / 2 + 1 > 64) continue;
        for (int32_t l1 : dl) {
            const bool ok = family == DCTMM_PRIME_FACTOR ? shape_plan_pf(N, L, n1, N / n1, l1, L / l1, &cand)
                                                         : shape_plan(N, L, n1, N / n1, l1, L / l1, &cand, &rows2);
            if (!ok) continue;
            const int64_t c = plan_cost(cand);
            if (best < 0 || c < best) {
                best = c;
                *plan = cand;
                *rows2_out = rows2;
            }
        }
    }
    return best >= 0;
}

// Prime-factor index maps.  Row n: m = 2n + 1 -> (n1, b).  Component k -> (c, e, sign) with
// z_k = sign D[c, e]  (forward) and the same for the inverse's input with (l1, l2).
void pf_row_map(int32_t n, int32_t n1, int32_t n2, int32_t* i1, int32_t* b)
{
    const int32_t m = 2 * n + 1;
    int32_t a = m % (4 * n1);
    *b = m % n2;
    if (a > 2 * n1) {
        a = 4 * n1 - a;
        *b = *b ? n2 - *b : 0;
    }
    *i1 = a / 2;
}
void pf_component_map(int32_t k, int32_t n1, int32_t n2, int32_t* c, int32_t* e, int32_t* sign)
{
    // k / (4 n1 n2) = q1 (k mod 4 n1) / (4 n1) + q2 (k mod n2) / n2 modulo 1
    const int64_t q1 = inverse_mod(n2, 4 * (int64_t)n1), q2 = inverse_mod(4 * (int64_t)n1, n2);
    const int32_t cc = (int32_t)(q1 * (k % (4 * n1)) % (4 * n1)), ee = (int32_t)(q2 * (k % n2) % n2);
    // cos(pi (2 n1 + 1) cc / (2 n1) + phi) = sign cos(pi (2 n1 + 1) c / (2 n1) + rho phi), 0 <= c <= n1
    int32_t rho;
    if (cc <= n1) { *c = cc; *sign = 1; rho = 1; }
    else if (cc <= 2 * n1) { *c = 2 * n1 - cc; *sign = -1; rho = -1; }
    else if (cc < 3 * n1) { *c = cc - 2 * n1; *sign = -1; rho = 1; }
    else { *c = 4 * n1 - cc; *sign = 1; rho = -1; }
    *e = rho > 0 ? ee : (ee ? n2 - ee : 0);
}

void build_pf(DctmmHostPlan* out)
{
    const DctmmPlan& p = out->plan;
    const int32_t N = p.n_in, L = p.n_keep, n1 = p.n1, n2 = p.n2, l1 = p.l1, l2 = p.l2;
    const int32_t h = (n2 - 1) / 2, hl = (l2 - 1) / 2;
    const double pi = 3.14159265358979323846;
    auto cs = [&](int64_t a, int64_t b, double* c, double* s) {  // of 2 pi a / b, a reduced first
        a %= b;
        *c = std::cos(2.0 * pi * (double)a / (double)b);
        *s = std::sin(2.0 * pi * (double)a / (double)b);
    };
    for (int s = 0; s < 4; ++s) out->f[s].assign((size_t)p.st[s].rows8 * p.st[s].k_pad, 0.0);
    // F1 / F3: rows e = 0 .. h of cos(2 pi b e / n2), then the same of sin (its row e = 0 is zero)
    for (int which = 0; which < 2; ++which) {
        const int32_t len = which ? l2 : n2, half = which ? hl : h;
        const DctmmStage& st = p.st[which ? 2 : 0];
        for (int32_t e = 0; e <= half; ++e)
            for (int32_t b = 0; b < len; ++b) {
                double c, s;
                cs((int64_t)e * b, len, &c, &s);
                out->f[which ? 2 : 0][(size_t)e * st.k_pad + b] = c;
                out->f[which ? 2 : 0][(size_t)(half + 1 + e) * st.k_pad + b] = s;
            }
    }
    // F2: rows (c, +) = [cos theta | -sin theta], (c, -) = [cos theta | +sin theta] over columns (part, n1),
    // theta = pi (2 n1 + 1) c / (2 N1), times 2/N.  F4: rows (j1, +-) over columns (part, c'), theta' = pi (2 j1 + 1) c' / (2 L1).
    for (int32_t c = 0; c <= n1; ++c)
        for (int32_t i = 0; i < n1; ++i) {
            double co, si;
            cs((int64_t)(2 * i + 1) * c, 4 * (int64_t)n1, &co, &si);
            double* plus = &out->f[1][(size_t)(2 * c) * p.st[1].k_pad], *minus = plus + p.st[1].k_pad;
            plus[i] = minus[i] = 2.0 / N * co;
            plus[n1 + i] = -2.0 / N * si;
            minus[n1 + i] = 2.0 / N * si;
        }
    for (int32_t j = 0; j < l1; ++j)
        for (int32_t c = 0; c <= l1; ++c) {
            double co, si;
            cs((int64_t)(2 * j + 1) * c, 4 * (int64_t)l1, &co, &si);
            double* plus = &out->f[3][(size_t)(2 * j) * p.st[3].k_pad], *minus = plus + p.st[3].k_pad;
            plus[c] = minus[c] = co;
            plus[l1 + 1 + c] = -si;
            minus[l1 + 1 + c] = si;
        }
    // table of the pass after stage 2: row (c, +-), column e of stage 2 -> piece of stage 3's operand
    const int32_t cols = p.st[1].atoms * 8, k3_pad = p.st[2].k_pad;
    out->table.assign((size_t)p.rows2 * cols + p.n_zero, 0xffffu);
    std::vector<char> filled((size_t)l2 * (l1 + 1), 0);
    for (int32_t k = 0; k < L; ++k) {
        int32_t c, e, sf, ci, ei, si;
        pf_component_map(k, n1, n2, &c, &e, &sf);
        pf_component_map(k, l1, l2, &ci, &ei, &si);
        const int32_t r = e <= h ? 2 * c : 2 * c + 1, o = e <= h ? e : n2 - e;
        uint16_t ent = (uint16_t)(b_piece((uint32_t)ei, (uint32_t)ci, (uint32_t)k3_pad) / 16);
        if (sf * si < 0) ent |= 0x2000u;
        if (k == 0) ent |= 0x4000u;
        out->table[(size_t)r * cols + o] = ent;
        filled[(size_t)ei * (l1 + 1) + ci] = 1;
    }
    size_t z = (size_t)p.rows2 * cols;
    for (int32_t ei = 0; ei < l2; ++ei)
        for (int32_t ci = 0; ci <= l1; ++ci)
            if (!filled[(size_t)ei * (l1 + 1) + ci]) out->table[z++] = (uint16_t)(b_piece((uint32_t)ei, (uint32_t)ci, (uint32_t)k3_pad) / 16);
}

// The two numbers of the prime-factor output map (see DctmmParams): the odd number m modulo 4L with
// m = a (mod 4 L1) and m = b (mod L2) is (a out_a + b out_w) mod 4L.
void pf_output_map(const DctmmPlan& p, int32_t* out_a, int32_t* out_w)
{
    const int64_t L4 = 4 * (int64_t)p.n_keep, m1 = 4 * (int64_t)p.l1;
    *out_a = (int32_t)(p.l2 * inverse_mod(p.l2, m1) % L4);
    *out_w = (int32_t)(m1 * inverse_mod(m1, p.l2) % L4);
}

void build_ct(DctmmHostPlan* out)
{
    const DctmmPlan& p = out->plan;
    const int32_t N = p.n_in, n1 = p.n1, n2 = p.n2, l1 = p.l1, l2 = p.l2, t1 = p.t1, t3 = p.t3;
    const double pi = 3.14159265358979323846;
    // exact angle reduction: cos / sin of 2 pi a / b with the integer a reduced modulo b first
    auto cs = [&](int64_t a, int64_t b, double* c, double* s) {
        a %= b;
        if (a < 0) a += b;
        *c = std::cos(2.0 * pi * (double)a / (double)b);
        *s = std::sin(2.0 * pi * (double)a / (double)b);
    };
    for (int s = 0; s < 4; ++s) out->f[s].assign((size_t)p.st[s].rows8 * p.st[s].k_pad, 0.0);
    // F1: rows (t1, part) in the lane order of the twiddle pass: within every 32 rows, 16 real parts then
    // the 16 imaginary parts of the same t1.  exp(-2 pi i n1 t1 / N1)
    for (int32_t r = 0; r < p.st[0].rows; ++r) {
        const int32_t part = (r >> 4) & 1, t = (r >> 5) * 16 + (r & 15);
        if (t >= t1) continue;
        for (int32_t k = 0; k < n1; ++k) {
            double c, s;
            cs((int64_t)k * t, n1, &c, &s);
            out->f[0][(size_t)r * p.st[0].k_pad + k] = part ? -s : c;
        }
    }
    // F2: row (part, t2), columns (n2, re | im) interleaved.  c = (2/N) exp(-i pi t2 / (2 N2)) exp(-2 pi i n2 t2 / N2)
    // = (2/N) exp(-2 pi i t2 (4 n2 + 1) / (4 N2));  real part of c A: cr Ar - ci Ai;  minus imaginary part: -ci Ar - cr Ai
    for (int32_t r = 0; r < p.rows2; ++r) {
        const DctmmRow2& m = out->rows2[r];
        const int32_t t2 = m.dir > 0 ? m.t_start / n1 : (N - m.t_start) / n1;
        for (int32_t k = 0; k < n2; ++k) {
            double c, s;
            cs((int64_t)t2 * (4 * k + 1), 4 * (int64_t)n2, &c, &s);
            const double cr = 2.0 / N * c, ci = -2.0 / N * s;
            double* row = &out->f[1][(size_t)r * p.st[1].k_pad];
            if (m.dir > 0) {
                row[2 * k] = cr;
                row[2 * k + 1] = -ci;
            } else {
                row[2 * k] = -ci;
                row[2 * k + 1] = -cr;
            }
        }
    }
    // F3: rows (j2, part) in the lane order of the twiddle pass; columns (a | b, t2).
    // g = exp(i pi t2 / (2 L2)) exp(2 pi i j2 t2 / L2) / 2 = exp(2 pi i t2 (4 j2 + 1) / (4 L2)) / 2;
    // (a - i b) g: real part a gr + b gi, imaginary part a gi - b gr
    for (int32_t r = 0; r < p.st[2].rows; ++r) {
        const int32_t part = (r >> 4) & 1, j2 = (r >> 5) * 16 + (r & 15);
        if (j2 >= l2) continue;
        double* row = &out->f[2][(size_t)r * p.st[2].k_pad];
        for (int32_t k = 0; k < l2; ++k) {
            double c, s;
            cs((int64_t)k * (4 * j2 + 1), 4 * (int64_t)l2, &c, &s);
            const double gr = 0.5 * c, gi = 0.5 * s;
            row[k] = part ? gi : gr;
            row[l2 + k] = part ? -gr : gi;
        }
    }
    // F4: row j1, columns (t1, re | im) interleaved: w (cos(2 pi j1 t1 / L1) Cr - sin(2 pi j1 t1 / L1) Ci),
    // w = 1 for the self-conjugate t1 (0, and L1/2 when L1 is even), 2 otherwise
    for (int32_t r = 0; r < l1; ++r) {
        double* row = &out->f[3][(size_t)r * p.st[3].k_pad];
        for (int32_t k = 0; k < t3; ++k) {
            double c, s;
            cs((int64_t)r * k, l1, &c, &s);
            const double w = (k == 0 || 2 * k == l1) ? 1.0 : 2.0;
            row[2 * k] = w * c;
            row[2 * k + 1] = -w * s;
        }
    }
}


}  // namespace

bool dctmm_host_plan(int32_t N, int32_t L, int32_t family, DctmmHostPlan* out)
{
    if (family != 0 && family != DCTMM_COOLEY_TUKEY && family != DCTMM_PRIME_FACTOR) return false;
    const int32_t first = family ? family : DCTMM_PRIME_FACTOR;
    bool ok = choose_factors(N, L, first, &out->plan, &out->rows2);
    if (!ok && family == 0) ok = choose_factors(N, L, DCTMM_COOLEY_TUKEY, &out->plan, &out->rows2);
    if (!ok) return false;
    out->table.clear();
    if (out->plan.family == DCTMM_PRIME_FACTOR)
        build_pf(out);
    else
        build_ct(out);
    return true;
}

namespace {

// prime-factor family: the same chain as the kernel's, with its matrices, table and index maps
void host_apply_pf(const DctmmHostPlan& hp, const double* x, int32_t C, double* y)
{
    const DctmmPlan& p = hp.plan;
    const int32_t N = p.n_in, L = p.n_keep;
    auto stage = [&](int s, const std::vector<double>& b, std::vector<double>* d) {
        const DctmmStage& st = p.st[s];
        d->assign((size_t)st.rows8 * st.outer * C, 0.0);
        for (int32_t r = 0; r < st.rows; ++r)
            for (int32_t k = 0; k < st.k; ++k) {
                const double f = hp.f[s][(size_t)r * st.k_pad + k];
                if (f == 0.0) continue;
                for (int32_t i = 0; i < st.outer * C; ++i) (*d)[(size_t)r * st.outer * C + i] += f * b[(size_t)k * st.outer * C + i];
            }
    };
    // rows (cos | sin, e) x outer o of stage s  ->  operand (k = part * outer + o, outer e) of stage s + 1
    auto transpose = [&](int s, const std::vector<double>& d, std::vector<double>* b) {
        const DctmmStage& st = p.st[s];
        const DctmmStage& nx = p.st[s + 1];
        const int32_t half = st.rows / 2;
        b->assign((size_t)nx.k * nx.outer * C, 0.0);
        for (int32_t r = 0; r < st.rows; ++r) {
            const int32_t part = r >= half, e = r - part * half;
            for (int32_t o = 0; o < st.outer; ++o)
                for (int32_t c = 0; c < C; ++c)
                    (*b)[((size_t)(part * st.outer + o) * nx.outer + e) * C + c] = d[((size_t)r * st.outer + o) * C + c];
        }
    };
    std::vector<double> b, d;
    b.assign((size_t)p.st[0].k * p.st[0].outer * C, 0.0);
    for (int32_t n = 0; n < N; ++n) {
        int32_t i1, bb;
        pf_row_map(n, p.n1, p.n2, &i1, &bb);
        for (int32_t c = 0; c < C; ++c) b[((size_t)bb * p.st[0].outer + i1) * C + c] = x[(size_t)n * C + c];
    }
    stage(0, b, &d);
    transpose(0, d, &b);
    stage(1, b, &d);
    // the table: entries number 16-byte pieces of stage 3's operand buffer
    {
        const DctmmStage& s2 = p.st[2];
        std::vector<double> pieces((size_t)s2.atoms * s2.k_pad * 8 * C, 0.0);
        const int32_t cols = p.st[1].atoms * 8;
        for (int32_t r = 0; r < p.rows2; ++r)
            for (int32_t o = 0; o < p.st[1].outer; ++o) {
                const uint16_t ent = hp.table[(size_t)r * cols + o];
                if (ent == 0xffffu) continue;
                const double scale = ((ent & 0x2000u) ? -1.0 : 1.0) * ((ent & 0x4000u) ? 0.5 : 1.0);
                for (int32_t c = 0; c < C; ++c) pieces[(size_t)(ent & 0x1fffu) * C + c] = scale * d[((size_t)r * p.st[1].outer + o) * C + c];
            }
        b.assign((size_t)s2.k * s2.outer * C, 0.0);
        for (int32_t k = 0; k < s2.k; ++k)
            for (int32_t o = 0; o < s2.outer; ++o)
                for (int32_t c = 0; c < C; ++c)
                    b[((size_t)k * s2.outer + o) * C + c] = pieces[(size_t)(b_piece((uint32_t)k, (uint32_t)o, (uint32_t)s2.k_pad) / 16) * C + c];
    }
    stage(2, b, &d);
    transpose(2, d, &b);
    stage(3, b, &d);
    int32_t out_a, out_w;
    pf_output_map(p, &out_a, &out_w);
    const int64_t L4 = 4 * (int64_t)L;
    for (int32_t r = 0; r < p.st[3].rows; ++r)
        for (int32_t o = 0; o < p.st[3].outer; ++o) {
            if ((r & 1) && o == 0) continue;
            const int64_t step = (r & 1) ? L4 - out_w : out_w;
            const int64_t m = ((int64_t)(2 * (r >> 1) + 1) * out_a + step * o) % L4;
            const int64_t j = (m < 2 * L ? m - 1 : L4 - m - 1) / 2;
            for (int32_t c = 0; c < C; ++c) y[(size_t)j * C + c] = d[((size_t)r * p.st[3].outer + o) * C + c];
        }
}

}  // namespace

void dctmm_host_apply(const DctmmHostPlan& hp, const double* x, int32_t C, double* y)
{
    if (hp.plan.family == DCTMM_PRIME_FACTOR) {
        host_apply_pf(hp, x, C, y);
        return;
    }
    const DctmmPlan& p = hp.plan;
    const int32_t N = p.n_in, L = p.n_keep, n1 = p.n1, n2 = p.n2, l1 = p.l1, l2 = p.l2, t1 = p.t1, t3 = p.t3;
    const double pi = 3.14159265358979323846;
    auto stage = [&](int s, const std::vector<double>& b, std::vector<double>* d) {
        // d[r][o][c] = sum_k F[r][k] b[k][o][c]
        const DctmmStage& st = p.st[s];
        d->assign((size_t)st.rows8 * st.outer * C, 0.0);
        for (int32_t r = 0; r < st.rows; ++r)
            for (int32_t k = 0; k < st.k; ++k) {
                const double f = hp.f[s][(size_t)r * st.k_pad + k];
                if (f == 0.0) continue;
                for (int32_t i = 0; i < st.outer * C; ++i) (*d)[(size_t)r * st.outer * C + i] += f * b[(size_t)k * st.outer * C + i];
            }
    };
    std::vector<double> b, d;
    // load: row n -> reordered position -> (k = n1 index, o = n2 index)
    b.assign((size_t)n1 * n2 * C, 0.0);
    for (int32_t n = 0; n < N; ++n) {
        const int32_t pos = (n & 1) ? N - 1 - (n >> 1) : (n >> 1);
        const int32_t k = pos / n2, o = pos % n2;
        for (int32_t c = 0; c < C; ++c) b[((size_t)k * n2 + o) * C + c] = x[(size_t)n * C + c];
    }
    stage(0, b, &d);
    // twiddle pass of stage 1 -> operand of stage 2: k = 2 n2 + part, o = t1
    b.assign((size_t)2 * n2 * t1 * C, 0.0);
    for (int32_t r = 0; r < p.st[0].rows; ++r) {
        const int32_t part = (r >> 4) & 1, t = (r >> 5) * 16 + (r & 15);
        if (t >= t1) continue;
        for (int32_t o = 0; o < n2; ++o) {
            const double ang = -pi * (double)(((int64_t)t * (4 * o + 1)) % (4 * (int64_t)N)) / (2.0 * N);
            const double wr = std::cos(ang), wi = std::sin(ang);
            for (int32_t c = 0; c < C; ++c) {
                const double v = d[((size_t)r * n2 + o) * C + c], other = d[((size_t)(r ^ 16) * n2 + o) * C + c];
                b[((size_t)(2 * o + part) * t1 + t) * C + c] = v * wr + other * (part ? wi : -wi);
            }
        }
    }
    stage(1, b, &d);
    // retained components -> operand of stage 3: k = (a | b) * L2 + t2', o = t1'
    b.assign((size_t)2 * l2 * t3 * C, 0.0);
    for (int32_t r = 0; r < p.rows2; ++r) {
        const DctmmRow2& m = hp.rows2[r];
        for (int32_t o = m.lo; o < m.hi; ++o) {
            const int32_t t = m.t_start + m.dir * o;
            for (int32_t c = 0; c < C; ++c) {
                const double v = d[((size_t)r * t1 + o) * C + c];
                if (t % l1 < t3) b[((size_t)(t / l1) * t3 + t % l1) * C + c] = v;
                if (t >= 1 && (L - t) % l1 < t3) b[((size_t)(l2 + (L - t) / l1) * t3 + (L - t) % l1) * C + c] = v;
            }
        }
    }
    stage(2, b, &d);
    // twiddle pass of stage 3 -> operand of stage 4: k = 2 t1' + part, o = j2
    b.assign((size_t)2 * t3 * l2 * C, 0.0);
    for (int32_t r = 0; r < p.st[2].rows; ++r) {
        const int32_t part = (r >> 4) & 1, j2 = (r >> 5) * 16 + (r & 15);
        if (j2 >= l2) continue;
        for (int32_t o = 0; o < t3; ++o) {
            const double ang = pi * (double)(((int64_t)(4 * j2 + 1) * o) % (4 * (int64_t)L)) / (2.0 * L);
            const double wr = std::cos(ang), wi = std::sin(ang);
            for (int32_t c = 0; c < C; ++c) {
                const double v = d[((size_t)r * t3 + o) * C + c], other = d[((size_t)(r ^ 16) * t3 + o) * C + c];
                b[((size_t)(2 * o + part) * l2 + j2) * C + c] = v * wr + other * (part ? wi : -wi);
            }
        }
    }
    stage(3, b, &d);
    const int32_t hL = (L + 1) / 2;
    for (int32_t r = 0; r < l1; ++r)
        for (int32_t o = 0; o < l2; ++o) {
            const int32_t j = l2 * r + o, m = j < hL ? 2 * j : 2 * (L - 1 - j) + 1;
            for (int32_t c = 0; c < C; ++c) y[(size_t)m * C + c] = d[((size_t)r * l2 + o) * C + c];
        }
}

bool dctmm_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep, int32_t family)
{
    if (dtype != FREQKV_BF16 || head_dim % 8 != 0 || n_in < 256) return false;
    DctmmPlan p;
    std::vector<DctmmRow2> rows2;
    if (family) return choose_factors(n_in, n_keep, family, &p, &rows2);
    return choose_factors(n_in, n_keep, DCTMM_PRIME_FACTOR, &p, &rows2) || choose_factors(n_in, n_keep, DCTMM_COOLEY_TUKEY, &p, &rows2);
}

cudaError_t dctmm_make_plan(int32_t n_in, int32_t n_keep, int32_t family, cudaStream_t stream, DctmmPlan* out)
{
    DctmmHostPlan hp;
    if (!dctmm_host_plan(n_in, n_keep, family, &hp)) return cudaErrorInvalidValue;
    DctmmPlan p = hp.plan;
    const size_t bytes = (size_t)p.f_bytes + p.tab_bytes + (size_t)round_up(n_in * 2, 16);
    std::vector<uint8_t> image(bytes, 0);
    // where row n of a slab goes in stage 1's operand (16-byte piece numbers; read from global memory
    // by the loading warps).  Cooley-Tukey: position p of the reordered sequence (v_p = x_2p,
    // v_{N-1-p} = x_{2p+1}) is piece (k = p / N2, o = p mod N2); prime-factor: piece (k = b, o = n1).
    for (int32_t n = 0; n < n_in; ++n) {
        int32_t k, o;
        if (p.family == DCTMM_PRIME_FACTOR) {
            pf_row_map(n, p.n1, p.n2, &o, &k);
        } else {
            const int32_t pos = (n & 1) ? n_in - 1 - (n >> 1) : (n >> 1);
            k = pos / p.n2;
            o = pos % p.n2;
        }
        const uint16_t piece = (uint16_t)(b_piece((uint32_t)k, (uint32_t)o, (uint32_t)p.st[0].k_pad) / 16);
        std::memcpy(&image[(size_t)p.f_bytes + p.tab_bytes + 2 * (size_t)n], &piece, 2);
    }
    for (int s = 0; s < 4; ++s) {
        const DctmmStage& st = p.st[s];
        for (int32_t m = 0; m < st.rows8; ++m)
            for (int32_t k = 0; k < st.k_pad; ++k) {
                const uint16_t v = to_bf16(hp.f[s][(size_t)m * st.k_pad + k]);
                // tile k / 64 starts at a_tile (a multiple of 1024 plus, for a shared narrow tile, its byte column)
                const int32_t column = (st.a_tile[k / 64] & 127) + (k % 64) * 2;
                const size_t off = (size_t)(st.a_tile[k / 64] & ~127) + (size_t)m * 128 + (size_t)((((column >> 4) ^ (m % 8)) << 4) + (column & 15));
                std::memcpy(&image[off], &v, 2);
            }
    }
    // where the value of row r, column o of stage 2 goes in the operand of stage 3 (16-byte piece
    // numbers): as a_{t2'} of column t mod L1 and / or as b_{t2'} of column (L - t) mod L1
    if (p.family == DCTMM_PRIME_FACTOR) {
        std::memcpy(&image[p.f_bytes], hp.table.data(), hp.table.size() * 2);
    } else {
        const int32_t cols = p.st[1].atoms * 8, k3_pad = p.st[2].k_pad;
        std::vector<uint32_t> tab((size_t)p.tab_bytes / 4, 0xffffffffu);
        for (int32_t r = 0; r < p.rows2; ++r) {
            const DctmmRow2& m = hp.rows2[r];
            for (int32_t o = m.lo; o < m.hi; ++o) {
                const int32_t t = m.t_start + m.dir * o;
                uint32_t da = 0xffffu, db = 0xffffu;
                if (t % p.l1 < p.t3) da = b_piece((uint32_t)(t / p.l1), (uint32_t)(t % p.l1), (uint32_t)k3_pad) / 16;
                if (t >= 1 && (p.n_keep - t) % p.l1 < p.t3)
                    db = b_piece((uint32_t)(p.l2 + (p.n_keep - t) / p.l1), (uint32_t)((p.n_keep - t) % p.l1), (uint32_t)k3_pad) / 16;
                tab[(size_t)r * cols + o] = da | (db << 16);
            }
        }
        std::memcpy(&image[p.f_bytes], tab.data(), (size_t)p.tab_bytes);
    }
    void* dev = nullptr;
    cudaError_t e = cudaMalloc(&dev, bytes);
    if (e != cudaSuccess) return e;
    // pageable source: the copy has left the host buffer when the call returns
    e = cudaMemcpyAsync(dev, image.data(), bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) {
        cudaFree(dev);
        return e;
    }
    p.image = dev;
    *out = p;
    return cudaSuccess;
}

void dctmm_free_plan(DctmmPlan* plan)
{
    if (plan->image) cudaFree(plan->image);
    plan->image = nullptr;
}

cudaError_t launch_dctmm(const CacheView& view, int32_t n_mat, const DctmmPlan& plan, int32_t sink, int32_t* status_dev,
                         unsigned long long wait_limit_ns, int sm_count, cudaStream_t stream)
{
    static PerDeviceOnce attrs;
    const cudaError_t attr_error = attrs.run([] {
        const cudaError_t e = cudaFuncSetAttribute(freqkv_dctmm_kernel<DCTMM_COOLEY_TUKEY>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT + 1024);
        if (e != cudaSuccess) return e;
        return cudaFuncSetAttribute(freqkv_dctmm_kernel<DCTMM_PRIME_FACTOR>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT + 1024);
    });
    if (attr_error != cudaSuccess) return attr_error;
    DctmmParams prm;
    prm.plan = plan;
    prm.out_a = prm.out_w = 0;
    if (plan.family == DCTMM_PRIME_FACTOR) pf_output_map(plan, &prm.out_a, &prm.out_w);
    prm.sink = sink;
    prm.slabs_per_matrix = view.head_dim / 8;
    const int64_t total = (int64_t)n_mat * prm.slabs_per_matrix;
    if (total > 0x7fffffff) return cudaErrorInvalidValue;
    prm.total_slabs = (int32_t)total;
    prm.status = status_dev;
    prm.wait_limit_ns = wait_limit_ns;
    const unsigned grid = (unsigned)std::min<int64_t>(total, sm_count);
    if (plan.family == DCTMM_PRIME_FACTOR)
        freqkv_dctmm_kernel<DCTMM_PRIME_FACTOR><<<grid, THREADS, plan.smem_bytes, stream>>>(view, prm);
    else
        freqkv_dctmm_kernel<DCTMM_COOLEY_TUKEY><<<grid, THREADS, plan.smem_bytes, stream>>>(view, prm);
    return cudaGetLastError();
}

}  // namespace freqkv
