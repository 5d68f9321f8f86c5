/*
 * btc.h -- C ABI of the B200 (sm_100a) codebook-binary linear layer.
 *
 * The layer (BTC-LLM inference path) stores a weight matrix as indices into a
 * binary codebook plus a row-wise scale:
 *
 *     W^[n, j*v:(j+1)*v] = alpha_n * C[idx[n, j]] (+ mu_n),   C in {+1,-1}^{Kc x v}
 *     y[m, n]            = sum_k x[m, k] * W^[n, k]
 *
 * (storage rule and block-dot sum: paper appendix "Binary codebook LUT-GEMM";
 * row-wise alpha / mu: Eq. 1-2 and the "Dequantize" step of Algorithm "Binary
 * Transformation and Compression").  Rows of W^ are output features, blocks of
 * length v run along the input dimension K, and v must divide K.
 *
 * Conventions for every entry point
 *   - All array arguments are DEVICE pointers owned by the caller unless a
 *     parameter is explicitly called "host".  The library allocates no device
 *     memory, never synchronises, and enqueues its work on `stream` (a
 *     cudaStream_t passed as void*, NULL = the legacy default stream).
 *   - Returns a btc_status; never aborts, traps or prints.  Argument errors are
 *     detected on the host before anything is launched.
 *   - idx values must be < Kc; this is the caller's contract (kernels do not
 *     check it).  btc_validate_indices checks it on the device.  With the
 *     environment variable BTC_DEBUG_CHECK_INDICES=1 every btc_linear_* call first
 *     enqueues that check on the same stream; a violation raises the device-side
 *     status word (btc_device_status then reports BTC_ERR_INDEX), nothing traps.
 *   - Programmatic dependent launch: the decode kernels let the next kernel on the
 *     stream start early and themselves start before their predecessor has
 *     finished.  They read x only after the predecessor has completed, but they
 *     prefetch idx, C_packed, alpha and mu right away.  So idx, C_packed, alpha and
 *     mu must be complete in memory before the call is enqueued: they must not be
 *     written by a preceding kernel that itself triggers its dependents early (the
 *     library's own kernels that write them -- btc_codebook_pack,
 *     btc_codebook_kmeans -- do not).  The same holds for the arrays of a
 *     btc_transform (sigma_bits, P1, P2): the transform kernel stages them before
 *     its predecessor has finished.  x and y carry no such restriction.
 *   - Ranges: 1 <= v <= 32, K % v == 0, 1 <= Kc <= 65536 (Kc need not be a power
 *     of two), N >= 1, M >= 1.
 *   - Alignment: x, idx, y and C_packed 16-byte aligned; alpha / mu 2-byte.
 */
#ifndef BTC_H_
#define BTC_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BTC_API __attribute__((visibility("default")))
#else
#define BTC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BTC_OK = 0,
    BTC_ERR_NULL = 1,        /* a required pointer is NULL                              */
    BTC_ERR_SHAPE = 2,       /* v, Kc, M, N, K out of range, or v does not divide K     */
    BTC_ERR_ALIGN = 3,       /* a pointer misses its alignment                          */
    BTC_ERR_UNSUPPORTED = 4, /* dtype / option not implemented by this entry point      */
    BTC_ERR_WORKSPACE = 5,   /* workspace missing or smaller than ..._workspace_bytes() */
    BTC_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed                     */
    BTC_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out (status word)        */
    BTC_ERR_INDEX = 8        /* debug check: an index >= Kc was seen (status word)      */
} btc_status;

typedef enum { BTC_F16 = 0, BTC_BF16 = 1, BTC_F32 = 2 } btc_dtype;

/* Optional online activation transform x' = x * D * (P1 (x) P2), D = diag(sigma) with
 * sigma in {+1,-1} (paper Section 4.2 "Transformation Pair", applied at inference as
 * X <- X T).  With x viewed row-major as a k1 x k2 matrix X:  X' = P1^T (X o sigma) P2.
 * sigma_bits: device uint32[ceil(K/32)], bit k set = -1 (flip channel k).
 * P1 [k1*k1], P2 [k2*k2]: device fp32, row-major.  k1 * k2 == K. */
typedef struct {
    const uint32_t *sigma_bits;
    const float *P1;
    const float *P2;
    int k1;
    int k2;
} btc_transform;

/* Library version (major*10000 + minor*100 + patch) and a static description of a status. */
BTC_API int btc_version(void);
BTC_API const char *btc_status_string(int status);

/* Last CUDA error code (cudaError_t as int) recorded by a call that returned BTC_ERR_CUDA
 * on this host thread; 0 if none. */
BTC_API int btc_last_cuda_error(void);

/* ---- codebook packing (offline, once per layer) --------------------------------------------
 * Bit map b = (c + 1) / 2 (Algorithm "Efficient Binary Vector Packing and Unpacking"): bit t
 * (LSB first) of C_packed[k] is 1 where C_pm1[k][t] >= 0 (sign(0) = +1, Section 4.1 M-step),
 * bits >= v are 0.  C_pm1: int8 [Kc][v] row-major.
 * C_packed is a buffer of btc_codebook_packed_bytes(Kc, v) bytes, 16-byte aligned: the first Kc
 * uint32 words are the public form just described (the interchange format); the rest is a
 * kernel-private re-arrangement of the same bits that the linear kernels read, so the whole
 * buffer must be passed to them unchanged.  btc_codebook_packed_bytes returns 0 for an invalid
 * shape. */
BTC_API size_t btc_codebook_packed_bytes(int Kc, int v);
BTC_API int btc_codebook_pack(const int8_t *C_pm1, int Kc, int v, uint32_t *C_packed, void *stream);
/* Same mapping with both pointers in HOST memory; runs on the calling thread, no GPU work. */
BTC_API int btc_codebook_pack_host(const int8_t *C_pm1_host, int Kc, int v, uint32_t *C_packed_host);

/* ---- codebook construction (offline; the step before the layer) -----------------------------
 * Section 4.1 "Flash and Accurate Binary Codebook", steps (1)-(3), with the loop of the appendix
 * Algorithm "Binary Codebook Optimization": the c most frequent distinct vectors are the initial
 * centroids; E-step z_i = argmin_k d_H(b_i, c_k) (POPCNT of the XOR; ||b - c||^2 = 4 d_H); M-step
 * c_k = element-wise majority of its vectors (ties -> +1; a cluster without vectors keeps its
 * centroid); stop when an E-step changes no assignment, or after max_iter E-steps.
 * Choices the paper leaves open: equally frequent vectors are ordered by their packed word,
 * ascending; among equally near centroids the smallest index wins.
 *   vecs      device, n uint32 words, bit t (LSB first) = (b_t + 1) / 2, bits >= v ignored
 *   C_words   device, Kc uint32 words out: the centroids in the public packed form (what
 *             btc_codebook_pack calls the first section); slots >= info[1] are 0
 *   z         device, n uint16 out: the assignment of the last E-step that ran
 *   info      device, 4 ints out: E-steps run; min(Kc, number of distinct vectors); number of
 *             distinct vectors; 1 if the loop ended because nothing changed
 *   workspace device, btc_codebook_kmeans_workspace_bytes(v, Kc) bytes, 256-byte aligned
 * Integer arithmetic only: the result is unique.  Work is enqueued on `stream`, nothing is
 * allocated, nothing synchronises (the loop is max_iter rounds of launches; rounds after the
 * last one return at once).  v <= 20 (the steps keep tables of 2^v entries); 20 < v <= 32 returns
 * BTC_ERR_UNSUPPORTED.  1 <= Kc <= 65536, 1 <= n < 2^31, 1 <= max_iter <= 4096. */
BTC_API size_t btc_codebook_kmeans_workspace_bytes(int v, int Kc);
BTC_API int btc_codebook_kmeans(const uint32_t *vecs, size_t n, int v, int Kc, int max_iter, uint32_t *C_words,
                                uint16_t *z, int *info, void *workspace, size_t workspace_bytes, void *stream);

/* ---- the layer ---------------------------------------------------------------------------
 * y[m, n] = alpha_n * sum_j <x[m, j*v:(j+1)*v], C[idx[n, j]]>  (+ mu_n * sum_k x[m, k])
 *
 *   x        [M, K] row-major, x_dtype = BTC_F16 or BTC_BF16
 *   idx      uint16 [N, K/v] row-major
 *   C_packed the buffer written by btc_codebook_pack (btc_codebook_packed_bytes(Kc, v) bytes)
 *   alpha    fp16 [N]; mu fp16 [N] or NULL (NULL = no mean term)
 *   T        NULL, or an activation transform applied to x first (see btc_transform)
 *   y        [M, N] row-major, y_dtype = BTC_F32 (also BTC_F16 / BTC_BF16, rounded to nearest)
 *   workspace / workspace_bytes: scratch of at least btc_linear_workspace_bytes(...) bytes,
 *            256-byte aligned; may be NULL when that function returns 0.  Contents are
 *            undefined afterwards; concurrent calls need distinct workspaces.  For a layer with
 *            few 128-row tiles and a long K (v = 16) the size includes room for the partial sums
 *            of a K split over the idle SMs, added in a fixed order by a second small kernel.
 *
 * btc_linear_gemv: the decode path, 1 <= M <= 8, built on the identity <x, c> = 2 * sum_{bit=1} x - sum x.
 *   M <= 2: x is quantised per K-slice to a block-fixed-point integer (2^-20 of the slice's largest magnitude
 *   for v = 16), the sums over set bits are exact integer sums on the warp-level int8 MMA, recombined and added
 *   over the slices in fp32.  M = 3..8: masked codeword bits act as fp16 numbers on the warp-level fp16 MMA with
 *   fp32 accumulation (one layer per call runs on an older kernel of the same arithmetic, a CTA per row tile; the
 *   fused multi-layer launch of btc_linear_gemv_batch on a newer one).  With v = 16, at most 74 tiles of 128 rows and a workspace of the size
 *   btc_linear_workspace_bytes asks for, M = 5..8 at K >= 8192 and M = 6..8 at K >= 4096 go to the tensor-core launch
 *   of btc_linear_gemm with K split over the SMs instead (it is the faster one there).  All stay well inside a
 *   relative error of 2e-3 against the exact product.  Shapes outside what these kernels cover (v not a multiple
 *   of 4 or above 20, K/v not a multiple of 8) run on slower general kernels with the same result.
 * btc_linear_gemm: any M >= 1, built for M >= 128: index tiles are decoded to +-1 bf16 (fp16 for fp16 x) tiles
 *   and multiplied on the tcgen05 tensor cores with fp32 accumulation in tensor memory; alpha (and mu) are
 *   applied in fp32 in the epilogue.  M <= 8 is forwarded to the decode path.
 * Errors: NULL / SHAPE / ALIGN / UNSUPPORTED / WORKSPACE as above; BTC_ERR_CUDA if a launch
 * fails.  Both are asynchronous: a device-side failure shows up at the caller's next sync.
 */
BTC_API size_t btc_linear_workspace_bytes(int M, int N, int K, int v, int Kc);
/* The same plus, when has_transform != 0, the room for the transformed activations (a call with T != NULL needs this
 * much): M*K fp32 values for the decode path (M <= 8, which then reads fp32 activations: no 16-bit rounding of x'),
 * M*K values in the dtype of x otherwise. */
BTC_API size_t btc_linear_workspace_bytes_ex(int M, int N, int K, int v, int Kc, int has_transform);

BTC_API int btc_linear_gemv(const void *x, int x_dtype, const uint16_t *idx, const uint32_t *C_packed,
                    const void *alpha, const void *mu, const btc_transform *T, void *y, int y_dtype,
                    int M, int N, int K, int v, int Kc, void *workspace, size_t workspace_bytes,
                    void *stream);

BTC_API int btc_linear_gemm(const void *x, int x_dtype, const uint16_t *idx, const uint32_t *C_packed,
                    const void *alpha, const void *mu, const btc_transform *T, void *y, int y_dtype,
                    int M, int N, int K, int v, int Kc, void *workspace, size_t workspace_bytes,
                    void *stream);

/* ---- several independent layers in one launch (decode path) ---------------------------------
 * A decode step is a handful of small layers (the q/k/v projections share one x; gate/up likewise),
 * each only a few MB of indices: launched one by one, launch latency and pipeline ramp-up cost more
 * than the index stream itself.  btc_linear_gemv_batch runs `count` independent layers
 *     y_i[m, n] = alpha_i[n] * sum_j <x_i[m, j*v:(j+1)*v], C_i[idx_i[n, j]]>  (+ mu_i[n] * sum_k x_i[m, k])
 * (same definition as btc_linear_gemv: paper appendix "Binary codebook LUT-GEMM", second display,
 * with the row-wise dequantisation of Eq. 1-2) as one persistent kernel over the concatenated
 * work, up to BTC_BATCH_MAX layers per launch; longer lists and layers the fused kernel does not
 * cover are run by further launches on the same stream, so the call never fails for that reason.
 *   problems  HOST array of `count` descriptors; it is read before the call returns.  Every pointer
 *             inside a descriptor is a DEVICE pointer with the layout, alignment and ranges stated
 *             for btc_linear_gemv; 1 <= M <= 8 for every layer.  No transform argument: transform the shared
 *             input once with btc_activation_transform.  x_dtype may also be BTC_F32 (what that call hands over)
 *             for layers with v a multiple of 4 up to 20 and K/v a multiple of 8 (BTC_ERR_UNSUPPORTED otherwise).
 *   The layers must be independent: no y_i may alias an x_j, idx_j or another y_j of the same call.
 * Errors: as btc_linear_gemv; the first failing layer's status is returned and later layers of the
 * list may not have been enqueued.
 */
#define BTC_BATCH_MAX 8
typedef struct {
    const void *x;
    const void *idx;       /* uint16 [N, K/v]; or, with idx_bits set, the rows written by btc_index_pack */
    const uint32_t *C_packed;
    const void *alpha;
    const void *mu;        /* NULL = no mean term */
    void *y;
    int x_dtype, y_dtype;
    int M, N, K, v, Kc;
    int idx_bits;          /* 0 or 16: uint16 containers; else btc_index_bits(Kc): dense-packed rows (see below) */
    int x_stride;          /* elements from one row of x to the next; 0 = K.  A multiple of 8 (see btc_linear_gemv_sum) */
    int idx_stride;        /* elements from one row of idx to the next; 0 = K/v.  A multiple of 8; uint16 containers only */
} btc_linear_problem;
BTC_API int btc_linear_gemv_batch(const btc_linear_problem *problems, int count, void *stream);

/* ---- the activation transform on its own ------------------------------------------------------------
 * xt = x * D * (P1 (x) P2) for M rows (see btc_transform; Section 4.2, X <- X T), for layers that share their
 * input: in a decode block q/k/v read one transformed activation vector and gate/up another, so the transform runs
 * once per distinct input and the layers follow as ONE btc_linear_gemv_batch call on xt.  xt_dtype is BTC_F32 (no
 * 16-bit rounding of x'; btc_linear_gemv_batch accepts such activations, see there) or the dtype of x.  x and xt are
 * [M, K] row-major, 16-byte aligned, and must not overlap.  Asynchronous on `stream`; no workspace.
 * Errors: NULL / SHAPE (k1 * k2 != K) / ALIGN / UNSUPPORTED (x not fp16 / bf16; xt neither fp32 nor the dtype of x; or
 * factors that do not fit shared memory: K above about 40000 for the few-row form). */
BTC_API int btc_activation_transform(const void *x, int x_dtype, const btc_transform *T, void *xt, int xt_dtype, int M, int K,
                                     void *stream);

/* ---- a layer whose weight is a SUM of codebook-binary terms (decode path, M <= 8) -----------------
 *     y[m, n] = sum_t ( alpha_t[n] * sum_j <x[m, k0_t + j*v : k0_t + (j+1)*v], C_t[idx_t[n, j]]>  +  mu_t[n] * sum_k x[m, k0_t + k] )
 * Two things the binariser of Section 3 emits have this form.  (1) Several scale groups per row: the non-salient
 * columns are split by split points into groups with their own (alpha, mu) (Eq. 1-2 per group; the split-point
 * ablation of Section 5) -- with the columns ordered by group, each group is a term over a column range.  (2) The
 * residual binarisation of salient columns, W ~ alpha_1 B_1 + alpha_2 B_2: two terms over the same range.  The paper
 * does not say how group membership is stored at inference; taken here: contiguous column ranges (a fixed column
 * order is free: it folds into the activation transform).
 * Each term is a btc_linear_problem whose x points at column k0_t of the activations (x_stride = the full K, in
 * elements, when M > 1) and whose idx is either its own [N, K_t/v] matrix or a column range of a wider one
 * (idx_stride).  k0_t, x_stride and idx_stride are multiples of 8 (16-byte alignment).  Every term names the same y,
 * M and N; with more than one term y is fp32.  The terms run as `count` launches in order on `stream`: the first
 * writes y, the others add to it (deterministic).  No transform argument.
 * Errors: as btc_linear_gemv_batch; BTC_ERR_UNSUPPORTED when a term is outside what the decode kernel covers
 * (v a multiple of 4 up to 20, K_t/v a multiple of 8). */
BTC_API int btc_linear_gemv_sum(const btc_linear_problem *terms, int count, void *stream);

/* ---- the paper's own kernel scheme (alternative to btc_linear_gemv) ---------------------------------
 * Same layer, same arguments (1 <= M <= 8, no transform), computed by the two-stage lookup of the appendix "Binary
 * codebook LUT-GEMM": Stage I builds, per block of x, the signed sums LUT_{j,p}[s] of its P = v/mu segments (mu = 8
 * when 8 divides v, else 4) over all 2^mu sign patterns; Stage II builds CBLUT_j[k] = sum_p LUT_{j,p}[key[k,p]] for
 * every codeword (keys = bit fields of the packed codeword); the product is then one lookup and one add per
 * (row, block).  Tables sit in shared memory, CBLUT entries in fp16 as the paper packs them (so an output carries an
 * fp16 rounding per block: about 2^-12 of the block dots' magnitude), row sums in fp32.  K is cut into slices of 8
 * blocks whose partial sums meet in `workspace` (btc_linear_gemv_lut_workspace_bytes(...) bytes, 16-byte aligned)
 * and are added in slice order by a second kernel.  Needs v a multiple of 4, K/v a multiple of 8 and 16*Kc bytes of
 * tables to fit shared memory (Kc up to about 13000); otherwise BTC_ERR_UNSUPPORTED.  Building CBLUT costs Kc*K/v*P
 * lookups per CTA row chunk whatever N is, so this route pays only when N is much larger than Kc; it is kept for
 * comparison (see the benchmark) and is not what btc_linear_gemv dispatches to. */
BTC_API size_t btc_linear_gemv_lut_workspace_bytes(int M, int N, int K, int v, int Kc);
BTC_API int btc_linear_gemv_lut(const void *x, int x_dtype, const uint16_t *idx, const uint32_t *C_packed,
                    const void *alpha, const void *mu, void *y, int y_dtype, int M, int N, int K, int v, int Kc,
                    void *workspace, size_t workspace_bytes, void *stream);

/* ---- dense-packed indices ------------------------------------------------------------------
 * The paper's storage count gives an index ceil(log2 c) bits ("v*c + ceil(log2 c) * mn/v", Section 4.3): 12 bits for
 * 4096 centroids, 13 for 8192 (Table 3a pairs v = 16 with codebooks of that size), which is what makes v = 16 a
 * sub-1-bit format; in uint16 containers the same layer occupies 16/v = 1 bit per weight.  btc_index_pack rewrites
 * uint16 [N, Kb] indices as N rows of btc_index_packed_row_bytes(Kb, Kc) bytes (the bit string rounded up to 16
 * bytes; padding is zero): row n is the little-endian bit string of its Kb indices, btc_index_bits(Kc) bits each --
 * bit q of index j is bit j*bits + q of the row, bit p of the row is bit p % 8 of byte p / 8.  btc_index_unpack is
 * the inverse.  idx values must be < 2^bits (higher bits are dropped).  Both are device-to-device, asynchronous on
 * `stream`; `packed` 16-byte aligned.
 * btc_linear_gemv_packed is btc_linear_gemv (no transform, no workspace) reading such rows; the same layers ride in
 * btc_linear_gemv_batch with idx_bits set.  The decode kernel unpacks widths of 12 and 13 bits (v a multiple of 4 up
 * to 16, codeword table in shared memory); other widths return BTC_ERR_UNSUPPORTED -- keep those layers in uint16
 * containers.  All layers of one batch call must use the same index format. */
BTC_API int btc_index_bits(int Kc);                            /* ceil(log2 Kc), at least 1; 0 for an invalid Kc */
BTC_API size_t btc_index_packed_row_bytes(int Kb, int Kc);
BTC_API int btc_index_pack(const uint16_t *idx, int N, int Kb, int Kc, void *packed, void *stream);
BTC_API int btc_index_unpack(const void *packed, int N, int Kb, int Kc, uint16_t *idx, void *stream);
BTC_API int btc_linear_gemv_packed(const void *x, int x_dtype, const void *idx_packed, const uint32_t *C_packed,
                    const void *alpha, const void *mu, void *y, int y_dtype, int M, int N, int K, int v, int Kc,
                    void *stream);

/* ---- btc_linear_gemm for callers that cannot allocate device memory ---------------------------
 * (No counterpart in the paper: this is a packaging variant of btc_linear_gemm, same arithmetic.)
 *
 * Some callers have no way to hand over a workspace: code that runs where cudaMalloc is forbidden
 * (inside a region that must not touch the allocator, a plugin whose host gives it only its input
 * and output buffers, a process whose memory was carved up in advance).  For them the scratch that
 * btc_linear_gemm needs for the mean term (the fp32 row sums of x, 4*M bytes) lives in a fixed
 * array inside the library's device image, BTC_STATIC_SCRATCH_BYTES long.  Every GPU that loads
 * the library holds that array until the process exits.
 *
 * Arguments are those of btc_linear_gemm without workspace / workspace_bytes.  Differences:
 *   - Needs 4*M <= BTC_STATIC_SCRATCH_BYTES, i.e. M <= BTC_STATIC_SCRATCH_BYTES / 4 rows of x;
 *     larger M returns BTC_ERR_WORKSPACE and nothing is launched.  K is never split here: only the
 *     bytes of the row sums are handed to the kernels, so no partial sums of y ever sit in the
 *     array.  T must be NULL (the transform needs M*K*2 bytes more): BTC_ERR_UNSUPPORTED.
 *   - The first call on each device looks up the array's device address (no allocation, no
 *     launch) and caches it; make that first call outside any stream capture.  The device that is
 *     current at the call is the one used, as for every other entry point.
 *   - All calls on one device share the one array.  Two calls whose kernels may overlap on the
 *     GPU (different streams, no ordering between them) race on it and may corrupt each other's
 *     mean term; order them on one stream or with events.  The array keeps the previous call's
 *     contents; each call overwrites the part it reads, so nothing has to be cleared.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine, on any call.
 */
#define BTC_STATIC_SCRATCH_BYTES 65536
BTC_API int btc_linear_gemm_static_scratch(const void *x, int x_dtype, const uint16_t *idx,
                    const uint32_t *C_packed, const void *alpha, const void *mu, const btc_transform *T,
                    void *y, int y_dtype, int M, int N, int K, int v, int Kc, void *stream);

/* ---- helpers (not on the hot path) --------------------------------------------------------- */

/* B^[n, j*v + t] = +1 / -1 as int8 [N, K]: the decoded sign matrix, for bit-exact checks. */
BTC_API int btc_decode_pm1(const uint16_t *idx, const uint32_t *C_packed, int N, int K, int v, int Kc,
                   int8_t *B_out, void *stream);

/* Counts entries of idx[0..count) that are >= Kc into *bad_count (device int32, zeroed by the
 * call before counting). */
BTC_API int btc_validate_indices(const uint16_t *idx, size_t count, int Kc, int *bad_count, void *stream);

/* Reads the library's device-side status word into *status_host (host pointer): BTC_OK, or
 * BTC_ERR_TIMEOUT if a bounded wait inside a tensor-core kernel ran out since the library was
 * loaded (the output of that launch is undefined).  This helper SYNCHRONISES the device. */
BTC_API int btc_device_status(int *status_host);
/* Clears the status word (SYNCHRONISES the device).  Host bookkeeping, no counterpart in the paper. */
BTC_API int btc_device_status_reset(void);
/* Failure-detection self-test (no counterpart in the paper): launches one warp that waits, with a limit of about a
 * millisecond, on a barrier nothing will ever arrive on.  The wait must give up, raise the status word
 * (btc_device_status then reports BTC_ERR_TIMEOUT) and let the kernel return, leaving the context usable: the same
 * path every bounded wait of the linear kernels takes when its partner is lost.  Asynchronous like the other calls. */
BTC_API int btc_selftest_bounded_wait(void *stream);

/* Bits per weight.  mode 0: log2(Kc)/v; 1: ceil(log2 Kc)/v (the paper's accounting, Section 4.3);
 * 2: 16/v (uint16 containers as stored here).  Adds scale_bits_per_row/K, and v*Kc/(N*K) for the
 * codebook when with_codebook != 0.  Host arithmetic only; returns -1 for an invalid shape. */
BTC_API double btc_bits_per_weight(int N, int K, int v, int Kc, int scale_bits_per_row, int mode,
                           int with_codebook);

#ifdef __cplusplus
}
#endif
#endif /* BTC_H_ */
