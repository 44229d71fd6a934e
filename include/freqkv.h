/*
 * freqkv.h -- C ABI of the FreqKV iterative KV-cache compression library for NVIDIA B200
 * (sm_100a).
 *
 * The library keeps a bounded key/value cache usable for arbitrarily long contexts: new
 * tokens are appended until the cache is full, then the non-sink part of every
 * (batch, layer, kv_head) matrix of K and of V is compressed in the frequency domain along
 * the token axis and written back in place, shorter, so that appending can go on
 * (FreqKV, Sections 3.3 and 3.4).
 *
 * Conventions
 *  - All cache pointers are DEVICE pointers owned by the caller; the library never frees or
 *    reallocates them.  `lens`, `kept_len` arrays and layout structs are HOST memory.
 *  - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    Calls enqueue work on it and return without synchronising, unless stated otherwise.
 *  - Every function returns a freqkv_status.  Arguments are validated in full before anything
 *    is enqueued: on INVALID_ARG, UNSUPPORTED and CAPACITY nothing was enqueued and no caller
 *    memory was modified.  FREQKV_ERR_ALLOC / FREQKV_ERR_CUDA can also come from the middle of
 *    a call that works in several passes (large caches, ragged batches, host buffers): passes
 *    enqueued before the failure still run, so the rows a compression rewrites are then
 *    undefined (everything else keeps its bytes).  No C++ exception crosses the boundary.
 *  - A context belongs to one device and must not be used from two threads at once.  Its work
 *    areas are shared by its calls: a call enqueued on another stream than the previous one first
 *    waits (on the device) for that one, so calls on one context never overlap on the GPU; use
 *    one context per stream for concurrency.
 *  - There is no CPU fallback: without a CUDA device freqkv_create fails.
 */
#ifndef FREQKV_H_
#define FREQKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FREQKV_OK = 0,
    FREQKV_ERR_INVALID_ARG = 1, /* null pointer, negative or inconsistent size            */
    FREQKV_ERR_UNSUPPORTED = 2, /* dtype / head_dim / stride / variant not supported      */
    FREQKV_ERR_CAPACITY = 3,    /* append would exceed the cache capacity: compress first */
    FREQKV_ERR_ALLOC = 4,       /* device or host allocation failed                       */
    FREQKV_ERR_CUDA = 5,        /* a CUDA runtime or driver call failed                   */
    FREQKV_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up (see last_device_status) */
} freqkv_status;

typedef enum { FREQKV_BF16 = 0, FREQKV_F32 = 1 } freqkv_dtype;

/* Which kernel family executes the compression.
 *   GEMM  the DCT-II -> truncate -> IDCT -> rescale chain folded into one precomputed
 *         kept_len x n_in projection basis and run on the tcgen05 tensor cores (bf16 caches,
 *         head_dim 128 only); halved by the even/odd symmetry of the cosines after a fold pass
 *         over the cache (folded twice, to three eighths, where n_in is a multiple of 4 and
 *         kept_len even), or, for kept_len <= 256, straight from the cache without that pass;
 *   FDCT  fast transform, O(N log N) (Appendix A: the DCT "can be computed using the FFT"): for
 *         bf16 caches the transform pair is factored into four small dense stages that run on
 *         the tensor cores, in place with no scratch, for every n_in = N1 N2 and kept_len = L1 L2
 *         whose factors fit the kernel and its shared memory (n_in up to about 4400).  Two
 *         families of factorisation (see freqkv_set_fast_family): prime-factor, for coprime
 *         factors with N2 and L2 odd (N1 <= 63, N2 <= 127, L1 <= 63, L2 <= 127: the paper's
 *         4092 -> 2046 = 44 x 93 -> 22 x 93), real arithmetic and no twiddle factors; and
 *         Cooley-Tukey, for any factors (N1 <= 126, L2 <= 64, L1 <= 128, about 2 kept_len / N1
 *         <= 128: 4096 -> 2048), complex with twiddles.  fp32 caches: a radix-16 kernel for
 *         power-of-two lengths;
 *   SIMT  the same projection on the fp32 CUDA cores (any shape; the only path for fp32
 *         caches of non-power-of-two length);
 *   AUTO  picks per shape from a table filled from measurements. */
typedef enum { FREQKV_AUTO = 0, FREQKV_GEMM = 1, FREQKV_FDCT = 2, FREQKV_SIMT = 3 } freqkv_variant;

/* Layout of ONE cache tensor (K or V; both must share it):
 * element (b, l, h, t, c) lives at  base + b*stride_batch + l*stride_layer + h*stride_head
 *                                        + t*stride_token + c      (strides in ELEMENTS).
 * head_dim is the contiguous axis.  Requirements: head_dim a multiple of 8 and at most 256,
 * stride_token >= head_dim, every stride a multiple of 8 elements (so that rows are 16-byte
 * aligned when the base pointer is), and the strides must not make two matrices overlap. */
typedef struct {
    int32_t dtype; /* freqkv_dtype */
    int32_t batch, layers, kv_heads, capacity /* tokens */, head_dim;
    int64_t stride_batch, stride_layer, stride_head, stride_token;
} freqkv_layout;

typedef struct freqkv_ctx freqkv_ctx; /* opaque: projection bases, twiddles, scratch, status word */

/* Fill `out` with the dense row-major [batch, layers, kv_heads, capacity, head_dim] layout. */
freqkv_status freqkv_layout_contiguous(freqkv_layout* out, freqkv_dtype dtype, int32_t batch, int32_t layers,
                                       int32_t kv_heads, int32_t capacity, int32_t head_dim);

/* Create / destroy a context on CUDA device `device`.  Creation allocates a small status
 * word; plans and scratch are allocated lazily (cudaMalloc) by freqkv_plan or by the first
 * compression of a new shape, and freed by freqkv_destroy.  Destroy synchronises the device. */
freqkv_status freqkv_create(freqkv_ctx** out, int device);
freqkv_status freqkv_destroy(freqkv_ctx* ctx);

/* Force the variant used by later freqkv_compress* calls (default FREQKV_AUTO).  A forced
 * variant that cannot run a given shape makes that call return FREQKV_ERR_UNSUPPORTED. */
freqkv_status freqkv_set_variant(freqkv_ctx* ctx, freqkv_variant variant);

/* Which factorisation the bf16 fast transform (variant FDCT) uses in later calls: 0 (default) =
 * prime-factor where the lengths allow it, else Cooley-Tukey; FREQKV_FAST_COOLEY_TUKEY or
 * FREQKV_FAST_PRIME_FACTOR = that family only (a shape it cannot factor is then left to the
 * other kernels: the radix-16 fast transform for powers of two, else GEMM or SIMT).  INVALID_ARG
 * for any other value. */
#define FREQKV_FAST_COOLEY_TUKEY 1
#define FREQKV_FAST_PRIME_FACTOR 2
freqkv_status freqkv_set_fast_family(freqkv_ctx* ctx, int32_t family);

/* Which variant AUTO (or the forced setting) resolves to for this shape; FREQKV_AUTO is never
 * returned.  Returns FREQKV_ERR_UNSUPPORTED through *out_variant = -1 when none applies. */
freqkv_status freqkv_resolve_variant(freqkv_ctx* ctx, const freqkv_layout* layout, int32_t n_in, int32_t n_keep,
                                     int32_t* out_variant);

/* Optional warm-up: build and cache whatever tables the given variant needs to compress
 * n_in non-sink rows to n_keep rows (the projection basis of Eq. 2-3 folded with the
 * definitions of Appendix A, or the transform twiddles).  Work is enqueued on `cuda_stream`.
 * Calling freqkv_compress without it builds the plan on first use. */
freqkv_status freqkv_plan(freqkv_ctx* ctx, int32_t n_in, int32_t n_keep, freqkv_dtype dtype,
                          freqkv_variant variant, void* cuda_stream);

/* One compression of a uniform cache (Section 3.3, Eq. 2-3; sink tokens: Section 3.4).
 * For every (batch, layer, kv_head) and for K and V alike, with N = cache_len - sink and
 * L = kept_len, rows [sink, cache_len) are one signal per channel:
 *     z = DCT-II_N(x)  (orthonormal, Appendix A);  keep z[0:L];
 *     y = sqrt(L/N) * IDCT_L(z[0:L])               (L-point orthonormal inverse).
 * y is rounded once (nearest even) to the cache dtype and written to rows [sink, sink+L).
 * Nothing else is written: sink rows, rows >= sink+L and any stride padding keep their bytes.
 * The caller's new cache length is sink + kept_len.  Arithmetic: fp32 accumulation.
 * kept_len == cache_len - sink is the identity and enqueues nothing; kept_len == 0 or
 * cache_len == sink enqueue nothing.
 * Errors: INVALID_ARG (null pointers, sink < 0, sink > cache_len, cache_len > capacity,
 * kept_len < 0, kept_len > cache_len - sink, k == v), UNSUPPORTED (layout rules above, forced
 * variant not applicable), ALLOC, CUDA. */
freqkv_status freqkv_compress(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, int32_t cache_len,
                              int32_t kept_len, int32_t sink, void* cuda_stream);

/* The same compression with another band of components retained (the paper's ablation
 * "Retaining High/Low-Frequency Components"): components first_component .. first_component +
 * kept_len - 1 of the N-point DCT-II are kept instead of the lowest kept_len,
 *     y = sqrt(L/N) * IDCT_L(z[first_component : first_component + L]),
 * the retained components taking positions 0 .. L-1 of the L-point inverse (the paper does not say
 * where they go; this keeps the output length L).  first_component = 0 is freqkv_compress;
 * first_component = N - L retains the highest frequencies.  Same rows written, same errors, plus
 * INVALID_ARG when first_component < 0 or first_component + kept_len > N.  The fast-transform
 * variant does not take first_component != 0 (UNSUPPORTED when forced; AUTO uses another variant). */
freqkv_status freqkv_compress_band(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, int32_t cache_len,
                                   int32_t kept_len, int32_t sink, int32_t first_component, void* cuda_stream);

/* Average power spectrum of the cached states along the token axis (Section 3.1, the analysis
 * behind the paper's power-spectrum figures): every channel of rows [sink, cache_len) of every
 * matrix is transformed with the orthonormal N-point DCT-II of Appendix A (N = cache_len - sink)
 * and the squared components are averaged over the batch and over head_dim.
 *   spectrum_k, spectrum_v  DEVICE pointers to fp32 arrays [layers, kv_heads, N], overwritten;
 *                           either may be NULL (not both).
 * The cache is only read.  bf16 caches with head_dim 128 (the tensor-core path; components are
 * computed with bf16 operands and fp32 accumulation); anything else: UNSUPPORTED.  The DCT
 * matrix of a new N is built on first use and kept by the context (N^2 bytes). */
freqkv_status freqkv_power_spectrum(freqkv_ctx* ctx, const freqkv_layout* layout, const void* k, const void* v,
                                    int32_t cache_len, int32_t sink, float* spectrum_k, float* spectrum_v,
                                    void* cuda_stream);

/* Ragged form: sequence b holds lens[b] rows and is compressed to sink + kept_len[b] rows,
 * each sequence with the transform of its own length (same definition as above with
 * N = lens[b] - sink, L = kept_len[b]).  `lens` and `kept_len` are host arrays of
 * layout->batch entries; on success lens[b] is updated to sink + kept_len[b].  All arguments
 * are validated for every sequence before anything is enqueued.  When every sequence that needs
 * work takes the folded tensor-core form (bf16, head_dim 128, more than 256 kept rows) the whole
 * batch is ONE fold launch and ONE tensor-core launch over a host-built work list (longest
 * sequences first), all plans built and all memory allocated before the first of them; the folded
 * inputs of the whole batch then live in the context's scratch (as many bytes as the non-sink
 * rows; beyond 64 GiB, or with other variants in the batch, the call goes run by run). */
freqkv_status freqkv_compress_ragged(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, int32_t* lens,
                                     const int32_t* kept_len, int32_t sink, void* cuda_stream);

/* Append n_new incoming tokens to every sequence (Section 3.4: incoming tokens are appended
 * to the compressed cache).  new_k / new_v are device pointers to dense
 * [batch, layers, kv_heads, n_new, head_dim] tensors of the cache dtype; rows
 * [lens[b], lens[b] + n_new) of sequence b are overwritten and lens[b] (host) grows by n_new.
 * If any lens[b] + n_new exceeds the capacity nothing is enqueued and FREQKV_ERR_CAPACITY is
 * returned: the caller compresses and retries -- this is the lazy trigger that reproduces the
 * compression counts of the paper's tables (a 4K-token input causes no compression). */
freqkv_status freqkv_append(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, const void* new_k,
                            const void* new_v, int32_t n_new, int32_t* lens, void* cuda_stream);

/* One decode step as a replayable CUDA graph, with the cache lengths on the DEVICE: no host
 * round trip decides when to compress (Section 3.4: the incoming token is appended; when the
 * cache is full it is compressed first).  For uniform batches: every sequence has the same length.
 *   lens_device   DEVICE array of `batch` int32 lengths, read and updated by the graph;
 *   new_k, new_v  DEVICE staging rows, dense [batch, layers, kv_heads, 1, head_dim]; the caller
 *                 refills them (on the launching stream) before each launch.
 * Each launch runs: a one-thread trigger kernel; if every sequence holds `capacity` rows, the
 * compression of rows [sink, capacity) to kept_len rows (tensor-core variant) and lens := sink +
 * kept_len -- skipped otherwise by a conditional graph node; then the append of the staged row at
 * lens[b] and lens[b] += 1.  If some but not all sequences are full, nothing is compressed, the
 * full ones are skipped and freqkv_last_device_status reports FREQKV_ERR_CAPACITY.
 * create allocates and builds everything the step needs (plan, scratch, graph) and may
 * synchronise the device; launch only enqueues the graph on `cuda_stream`.  The pointers are
 * baked into the graph.  Requirements: bf16, head_dim 128, 1 <= kept_len < capacity - sink.
 * destroy synchronises the device.  A graph must be destroyed before its context. */
typedef struct freqkv_decode_graph freqkv_decode_graph;
freqkv_status freqkv_decode_graph_create(freqkv_ctx* ctx, const freqkv_layout* layout, void* k, void* v, const void* new_k,
                                         const void* new_v, int32_t* lens_device, int32_t kept_len, int32_t sink,
                                         freqkv_decode_graph** out);
freqkv_status freqkv_decode_graph_launch(freqkv_decode_graph* graph, void* cuda_stream);
freqkv_status freqkv_decode_graph_destroy(freqkv_decode_graph* graph);

/* Host-buffer form of freqkv_compress for callers whose cache lives in host memory (pinned
 * memory gives full copy bandwidth; pageable memory works).  k_host / v_host use `layout` in
 * host memory.  Rows [sink, cache_len) of every matrix are copied to a device staging cache the
 * context owns (allocated on first use, same layout), compressed there exactly as
 * freqkv_compress does, and rows [sink, sink+kept_len) are copied back over the host rows.
 * The work is pipelined over groups of layers on three streams the context owns (copy in,
 * compress, copy out overlap; both directions of the bus are used at once); it starts after
 * everything enqueued on `cuda_stream` so far, and work enqueued on `cuda_stream` afterwards starts
 * after it.  The host buffers must stay valid and untouched until that stream has been
 * synchronised.  h2d_bytes / d2h_bytes (optional, may be NULL) receive the bytes moved each way. */
freqkv_status freqkv_compress_host(freqkv_ctx* ctx, const freqkv_layout* layout, void* k_host, void* v_host,
                                   int32_t cache_len, int32_t kept_len, int32_t sink, void* cuda_stream,
                                   int64_t* h2d_bytes, int64_t* d2h_bytes);

/* Attention of one newly incoming token per sequence over the bounded cache of one layer
 * (Section 3.4: the new token attends to the sink tokens, the compressed tokens and the recent
 * tokens, i.e. to cache rows [0, lens[b]) of its KV head; its own key and value are the last of
 * those rows, appended before this call).
 * Position encoding (Section 3.4, last paragraph): keys are cached BEFORE RoPE.  Here cached key
 * row j is rotated to position j -- its index inside the cache, not inside the original sequence
 * -- and the query to position lens[b] - 1.  RoPE pairs channel c with channel c + head_dim/2 (the
 * LLaMA layout) and turns pair c by  position * rope_base^(-2c/head_dim);  rope_base <= 0 switches
 * it off (plain softmax attention).
 *   q, out  DEVICE pointers, dense [batch, kv_heads * q_heads_per_kv, head_dim] in the cache dtype;
 *           query head i uses KV head i / q_heads_per_kv (grouped-query attention); q is given
 *           before RoPE; out = softmax(scale * q_rot . K_rot^T) V, fp32 arithmetic, rounded once.
 *           bf16 caches with q_heads_per_kv >= 2 take both products on the tensor cores (fp32
 *           accumulation): rotated keys and scaled queries are rounded to fp16 for the scores,
 *           the softmax weights to bf16 for the second product; keys and  scale * log2(e) * q
 *           must then stay below 65504 in magnitude (larger values give infinities).
 *   scale   score scale; <= 0 selects 1/sqrt(head_dim).
 *   lens    HOST array of `batch` cache lengths, each in [1, capacity].
 * Nothing in the cache is written.  Errors: INVALID_ARG (null pointers, q == out, layer out of
 * range, a length outside [1, capacity], NaN scale or base), UNSUPPORTED (head_dim != 128,
 * q_heads_per_kv not 1, 2, 4 or 8, misaligned pointers, layout rules), ALLOC, CUDA.  The first call
 * with a new rope_base builds a cos/sin table (capacity x head_dim/2 entries) the context keeps. */
freqkv_status freqkv_attend_decode(freqkv_ctx* ctx, const freqkv_layout* layout, const void* k, const void* v,
                                   int32_t layer, const void* q, void* out, int32_t q_heads_per_kv, const int32_t* lens,
                                   float rope_base, float scale, void* cuda_stream);

/* Attention of a chunk of n_new incoming tokens per sequence over the bounded cache of one layer
 * (Section 3.3: during training and prefilling the sequence is processed chunk-wise, attention
 * interleaved with compression; first attention equation).  The chunk's keys and values have been
 * appended already: they are cache rows [lens[b] - n_new, lens[b]).  Token i of the chunk attends
 * to the sink tokens, the compressed tokens, the chunk's earlier tokens and itself, i.e. to rows
 * [0, lens[b] - n_new + i]; keys and queries get the RoPE of Section 3.4 at those row indices
 * (key row j at j, query i at lens[b] - n_new + i; same pairing and rope_base rule as above).
 *   q, out  DEVICE pointers, dense [batch, kv_heads * q_heads_per_kv, n_new, head_dim], bf16;
 *           out = softmax(mask(scale * q_rot . K_rot^T)) V.  Both products run on the tensor
 *           cores with fp32 accumulation: rotated keys and scaled queries are rounded to fp16,
 *           the softmax weights to bf16; keys and  scale * log2(e) * q  must stay below 65504.
 *   lens    HOST array of `batch` cache lengths (chunk included), each in [n_new, capacity].
 * Nothing in the cache is written.  Errors: INVALID_ARG (null pointers, q == out, layer out of
 * range, n_new < 1, a length outside [n_new, capacity], NaN scale or base), UNSUPPORTED (fp32
 * caches, head_dim != 128, misaligned pointers, layout rules), ALLOC, CUDA.  The context keeps
 * two scratch buffers (rotated keys of one layer, rotated queries of one chunk) and the cos/sin
 * table; they are allocated, or grown after a device synchronisation, by the first call that
 * needs them (so make that call before any stream capture).  A barrier wait inside the kernel that runs out (2 s) ends the kernel and shows up in
 * freqkv_last_device_status as TIMEOUT. */
freqkv_status freqkv_attend_prefill(freqkv_ctx* ctx, const freqkv_layout* layout, const void* k, const void* v,
                                    int32_t layer, const void* q, void* out, int32_t q_heads_per_kv, int32_t n_new,
                                    const int32_t* lens, float rope_base, float scale, void* cuda_stream);

/* Instrumentation for benchmarks.  With timing enabled every compression records a CUDA event
 * pair on the caller's stream around its transform kernel (the projection / fast-transform
 * launch, not the copy-back or table builders).  freqkv_get_timing waits for the recorded
 * events, returns the number of timed transform launches and their summed device time in
 * milliseconds since the last call, plus the number of kernels of any kind this context has
 * launched since creation, and resets the timing sums.  Any output pointer may be NULL. */
freqkv_status freqkv_set_timing(freqkv_ctx* ctx, int32_t enabled);
freqkv_status freqkv_get_timing(freqkv_ctx* ctx, int64_t* transform_launches, double* transform_ms,
                                int64_t* kernels_launched);

/* Compression for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a packaging variant of freqkv_compress, same definition, same result.)
 *
 * Who needs it: code that runs where cudaMalloc is not allowed or not safe -- under a lock that
 * an allocation's implicit device synchronisation could deadlock against, in a serving loop
 * whose device-memory budget is frozen, or inside a host framework that owns all device memory.
 * freqkv_compress does not fit there: its context, its plan and its staging buffer all come
 * from cudaMalloc.
 *
 * What it does: the CUDA-core (SIMT) projection of freqkv_compress with its two work areas --
 * the fp32 projection basis and the staging area for compressed rows -- placed in fixed arrays
 * inside the library image instead of allocated memory.  No context is needed; `k` and `v` are
 * device pointers exactly as for freqkv_compress and the arrays of the device that owns them are
 * used: both must be plain device allocations of ONE device (INVALID_ARG for host or managed
 * memory, or when k and v live on different devices).  The call itself performs no cudaMalloc,
 * cudaFree or other allocating call, so free device memory is the same before and after it.
 * If a launch fails (FREQKV_ERR_CUDA) the groups of matrices enqueued before it still run.
 *
 * Limits (FREQKV_ERR_UNSUPPORTED beyond them, nothing enqueued): with n_in = cache_len - sink,
 *   roundup(n_in, 64) * roundup(kept_len, 64) <= FREQKV_NOALLOC_MAX_BASIS_ELEMS   (1 Mi entries),
 *   kept_len * head_dim * sizeof(element)     <= FREQKV_NOALLOC_STAGING_BYTES      (4 MiB);
 * any number of matrices is accepted (they are processed in groups that fit the staging area).
 * Cost: every GPU that loads the library holds the 8 MiB of arrays until the process exits.
 *
 * First call on a device: it looks up the device addresses of the arrays (once per device), so
 * make the first call on each device before starting any stream capture.
 * Sharing: all calls on a device share the arrays.  Calls on one stream are ordered and safe;
 * calls whose kernels may overlap on the GPU (different streams, different threads) race on them
 * and must be serialised by the caller.  Stale contents of earlier calls are never read: the
 * part of the basis a call uses is rewritten by that call. */
#define FREQKV_NOALLOC_MAX_BASIS_ELEMS (1u << 20)
#define FREQKV_NOALLOC_STAGING_BYTES (4u << 20)
freqkv_status freqkv_compress_noalloc(const freqkv_layout* layout, void* k, void* v, int32_t cache_len,
                                      int32_t kept_len, int32_t sink, void* cuda_stream);

/* Every wait of a tensor-core kernel on one of its barriers is bounded; this sets the bound for
 * later launches of this context (default 2 s; at least 1000 ns).  A wait that runs out ends the
 * kernel and is reported by freqkv_last_device_status as FREQKV_ERR_TIMEOUT. */
freqkv_status freqkv_set_wait_limit(freqkv_ctx* ctx, int64_t nanoseconds);

/* Self-test of that give-up path: enqueues a one-thread kernel that waits, with the kernels' own
 * bounded wait, on a barrier nothing ever arrives on.  After `nanoseconds` (1000 .. 1e9) it gives
 * up, sets its bit in the status word and returns -- the next freqkv_last_device_status reports
 * FREQKV_ERR_TIMEOUT, the one after that FREQKV_OK, and the context stays usable. */
freqkv_status freqkv_selftest_bounded_wait(freqkv_ctx* ctx, int64_t nanoseconds, void* cuda_stream);

/* Synchronise `cuda_stream`, then read and clear the device status word.  FREQKV_OK unless a
 * kernel's bounded wait (mbarrier / flag) ran out, in which case the affected output rows are
 * undefined and FREQKV_ERR_TIMEOUT is returned; the context stays usable. */
freqkv_status freqkv_last_device_status(freqkv_ctx* ctx, void* cuda_stream);

/* Host-only argument checks, exactly the ones freqkv_compress / freqkv_append apply before
 * they enqueue anything (they touch no device and need no context; freqkv_check_attend and
 * freqkv_check_attend_prefill likewise for the two attention calls): the status those calls
 * would return for these arguments, FREQKV_OK if they would go ahead. */
freqkv_status freqkv_check_compress(const freqkv_layout* layout, const void* k, const void* v, int32_t cache_len,
                                    int32_t kept_len, int32_t sink);
freqkv_status freqkv_check_append(const freqkv_layout* layout, const void* k, const void* v, const void* new_k,
                                  const void* new_v, int32_t n_new, const int32_t* lens);
freqkv_status freqkv_check_attend(const freqkv_layout* layout, const void* k, const void* v, int32_t layer, const void* q,
                                  const void* out, int32_t q_heads_per_kv, const int32_t* lens);
freqkv_status freqkv_check_attend_prefill(const freqkv_layout* layout, const void* k, const void* v, int32_t layer,
                                          const void* q, const void* out, int32_t q_heads_per_kv, int32_t n_new,
                                          const int32_t* lens);

/* Host-only diagnostic of the fast transform's plan (no device, no context): applies the
 * factored chain the FDCT variant would run for (n_in, n_keep) -- same factor choice, same
 * matrices before rounding, same index maps -- in fp64 on the host to `channels` signals
 * x[n * channels + c], n < n_in, and writes y[m * channels + c], m < n_keep.  It exists so that a
 * plan can be checked against the definition (Section 3.3, Eq. 2-3; Appendix A) without a GPU; it
 * is not a compute path.  family as in freqkv_set_fast_family.  factors (optional, 5 values)
 * receives N1, N2, L1, L2 and the family used.  UNSUPPORTED when no factorisation of these lengths
 * fits the kernel. */
freqkv_status freqkv_fast_plan_apply_host(int32_t n_in, int32_t n_keep, int32_t family, const double* x, int32_t channels,
                                          double* y, int32_t* factors);

/* Host-only: how many levels of the even/odd symmetry fold (Appendix A's cosines are even or odd
 * under n -> N-1-n) variant GEMM applies to a compression of n_in rows to kept_len components
 * starting at first_component: 0 = none (kept_len <= 256: straight from the cache), 1, or 2 (n_in a
 * multiple of 4, kept_len even, first_component 0, and fewer 64-row slices that way).  The executed
 * multiply-adds per matrix are 2 * ceil(L/2) * ceil(N/2) * head_dim with one level and
 * 3 * ceil(L/4) * (N/2) * head_dim with two.  -1 for invalid lengths.  Ragged batches and the power
 * spectrum always use one level. */
int32_t freqkv_gemm_fold_levels(int32_t n_in, int32_t kept_len, int32_t first_component);

/* Text of the most recent CUDA failure or device-status report seen by this context (owned by
 * the context, valid until its next call); "" if none. */
const char* freqkv_last_error(freqkv_ctx* ctx);

/* Static, human-readable name of a status code. */
const char* freqkv_status_string(freqkv_status status);

/* Library version as major*10000 + minor*100 + patch. */
int32_t freqkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FREQKV_H_ */
