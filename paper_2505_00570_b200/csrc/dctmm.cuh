// Fast transform on the tensor cores: the DCT-II -> truncate -> L-point IDCT chain of the
// compression (Section 3.3, Eq. 2-3; Appendix A: "can be computed using the FFT") factored into
// four small dense stages, each a tcgen05 matrix product.  Two families of factorisation:
// a prime-factor one (coprime factors, real arithmetic, no twiddles) and a Cooley-Tukey one
// (any factors, complex arithmetic, twiddles between the stages).  Declarations.
#pragma once
#include <vector>

#include "common.cuh"

namespace freqkv {

// One stage D = F * B: F is rows x k (K-major A operand, resident in shared memory), B holds the
// slab's data as k x (outer index, 8 channels) (MN-major operand).
struct DctmmStage {
    int32_t k;          // contraction length
    int32_t k_pad;      // ... rounded up to 16 (one instruction contracts 16)
    int32_t rows;       // rows of F that mean something (the instruction always computes 128)
    int32_t rows8;      // ... rounded up to 8: rows stored per 64-wide tile of F
    int32_t outer;      // values of the outer index (columns = outer * 8 channels)
    int32_t atoms;      // ceil(outer / 8): 64-column groups
    int32_t a_tile[8];  // byte offset in shared memory of each 64-wide tile of F (a last tile narrower than
                        // 64 may start 32, 64 or 96 bytes into rows it shares with another stage's)
    int32_t b_off;      // byte offset of this stage's B buffer in shared memory
};

constexpr int32_t DCTMM_COOLEY_TUKEY = 1, DCTMM_PRIME_FACTOR = 2;

// Row r of the second stage yields, at column t1, the retained spectrum value of index
// t = t_start + dir * t1 for lo <= t1 < hi (nothing elsewhere).
struct DctmmRow2 {
    int32_t t_start, dir, lo, hi;
};

struct DctmmPlan {
    int32_t family = 0;      // DCTMM_COOLEY_TUKEY or DCTMM_PRIME_FACTOR
    int32_t n_in = 0, n_keep = 0;
    int32_t n1 = 0, n2 = 0, l1 = 0, l2 = 0;  // n_in = n1 * n2, n_keep = l1 * l2
    int32_t t1 = 0, t3 = 0;                  // Cooley-Tukey: n1/2 + 1, l1/2 + 1, the independent outputs of a real-input stage
    DctmmStage st[4];
    int32_t rows2 = 0;
    int32_t f_bytes = 0;     // bytes of the four F images (start of shared memory)
    int32_t smem_bytes = 0;  // everything: F, two data buffers, table, barriers
    int32_t tab_off = 0, tab_bytes = 0;  // destination table of the pass after stage 2 (shared memory)
    int32_t n_zero = 0;      // prime-factor: pieces of stage 3's operand that no retained component fills
                             // (their numbers follow the table's row entries)
    int32_t bar_off = 0;
    void* image = nullptr;   // device: F images (f_bytes), that table, then where each row of a slab goes in
                             // stage 1's operand (n_in 16-bit piece numbers)
};

// Largest transform the kernel's shared memory can hold is found by trying: true when some
// factorisation of (n_in, n_keep) meets every limit (bf16 caches, head_dim a multiple of 8).
// family: 0 = either, else one of the two constants above.
bool dctmm_supported(int32_t dtype, int32_t head_dim, int32_t n_in, int32_t n_keep, int32_t family = 0);

// Host part of a plan: factor choice, stage shapes, the four matrices in fp64 (row-major,
// rows x k_pad, zero padded), the row table of stage 2 (Cooley-Tukey) or the destination table of
// the pass after it (prime-factor: see dctmm.cu).  Returns false when no factorisation fits.
// family 0 prefers the prime-factor form where it exists.
struct DctmmHostPlan {
    DctmmPlan plan;
    std::vector<double> f[4];
    std::vector<DctmmRow2> rows2;
    std::vector<uint16_t> table;  // prime-factor: rows2 x (8 atoms(stage 2)) entries, then n_zero piece numbers
};
bool dctmm_host_plan(int32_t n_in, int32_t n_keep, int32_t family, DctmmHostPlan* out);

// The factored chain applied on the host in fp64 to `channels` signals x[n * channels + c]
// (n < n_in) with the plan's own matrices and index maps; y[m * channels + c], m < n_keep.
// For checking a plan against the definition; not a compute path.
void dctmm_host_apply(const DctmmHostPlan& hp, const double* x, int32_t channels, double* y);

cudaError_t dctmm_make_plan(int32_t n_in, int32_t n_keep, int32_t family, cudaStream_t stream, DctmmPlan* out);
void dctmm_free_plan(DctmmPlan* plan);
cudaError_t launch_dctmm(const CacheView& view, int32_t n_mat, const DctmmPlan& plan, int32_t sink, int32_t* status_dev,
                         unsigned long long wait_limit_ns, int sm_count, cudaStream_t stream);

constexpr int32_t DCTMM_ERR_WAIT = 0x400;  // status-word bit: a barrier wait of the kernel ran out

}  // namespace freqkv
