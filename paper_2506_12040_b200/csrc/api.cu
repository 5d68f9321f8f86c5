// Host side of the C ABI: argument validation, variant selection, launch.
#include <cmath>
#include "btc_internal.cuh"

namespace btc {

static thread_local int g_last_cuda_error = 0;

int cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return BTC_ERR_CUDA;
}

static bool aligned(const void *p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; }

static int validate(const void *x, int x_dt, const uint16_t *idx, const uint32_t *Cp, const void *alpha,
                    void *y, int y_dt, int M, int N, int K, int v, int Kc)
{
    if (!x || !idx || !Cp || !alpha || !y) return BTC_ERR_NULL;
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || M < 1 || N < 1 || K < 1 || K % v) return BTC_ERR_SHAPE;
    if (x_dt != BTC_F16 && x_dt != BTC_BF16) return BTC_ERR_UNSUPPORTED;
    if (y_dt != BTC_F32 && y_dt != BTC_F16 && y_dt != BTC_BF16) return BTC_ERR_UNSUPPORTED;
    if (!aligned(x, 16) || !aligned(idx, 16) || !aligned(y, 16) || !aligned(Cp, 16) || !aligned(alpha, 2))
        return BTC_ERR_ALIGN;
    return BTC_OK;
}

enum Path { PATH_GEMV, PATH_GEMM };

// Room for the transformed activations at the front of the workspace (fp32 for the decode path, see run_linear).
static size_t transform_bytes(int M, int K, int v)
{
    const bool f32 = M <= 8 && v % 4 == 0 && v <= 20 && (K / v) % 8 == 0 && K % 8 == 0;
    return (((size_t)M * K * (f32 ? 4 : 2) + 255) / 256) * 256;
}

static int run_linear(Path path, const void *x, int x_dt, const uint16_t *idx, const uint32_t *Cp,
                      const void *alpha, const void *mu, const btc_transform *T, void *y, int y_dt, int M,
                      int N, int K, int v, int Kc, void *ws, size_t ws_bytes, void *stream)
{
    int rc = validate(x, x_dt, idx, Cp, alpha, y, y_dt, M, N, K, v, Kc);
    if (rc != BTC_OK) return rc;
    if (mu && !aligned(mu, 2)) return BTC_ERR_ALIGN;
    if (path == PATH_GEMV && M > 8) return BTC_ERR_SHAPE;
    // (btc_linear_workspace_bytes may ask for more: room for a K split, which the kernels do without when it is missing)
    size_t need = (M <= 8) ? gemv_decode_workspace_bytes(M, N, K, v, Kc) : 0;
    if (gemm_tcgen05_workspace_min(M) > need) need = gemm_tcgen05_workspace_min(M);
    need = (need + 255) / 256 * 256;
    // the transformed activations go to the front of the workspace: as fp32 where the decode kernel will read them (it
    // quantises or rounds the activations itself), else in the dtype of x
    const bool xt_f32 = T && M <= 8 && v % 4 == 0 && v <= 20 && (K / v) % 8 == 0 && K % 8 == 0;
    const size_t xt_bytes = T ? transform_bytes(M, K, v) : 0;
    if (need + xt_bytes > 0) {
        if (!ws || ws_bytes < need + xt_bytes) return BTC_ERR_WORKSPACE;
        if (!aligned(ws, 256)) return BTC_ERR_ALIGN;
    }
    cudaStream_t s = (cudaStream_t)stream;
    if (debug_check_indices_enabled()) {
        rc = launch_index_check(idx, (size_t)N * (K / v), Kc, s);
        if (rc != BTC_OK) return rc;
    }

    LinearArgs a;
    a.x = x; a.idx = idx; a.Cp = Cp;
    a.alpha = reinterpret_cast<const __half *>(alpha);
    a.mu = reinterpret_cast<const __half *>(mu);
    a.y = y; a.workspace = ws; a.workspace_bytes = ws_bytes;
    a.x_dt = x_dt; a.y_dt = y_dt;
    a.M = M; a.N = N; a.K = K; a.v = v; a.Kc = Kc; a.Kb = K / v;

    if (T) {
        // The transformed activations live at the front of the workspace; the kernels' own
        // scratch follows.
        if (!T->sigma_bits || !T->P1 || !T->P2) return BTC_ERR_NULL;
        if (T->k1 < 1 || T->k2 < 1 || (long long)T->k1 * T->k2 != K) return BTC_ERR_SHAPE;
        rc = launch_transform(x, x_dt, *T, ws, xt_f32 ? BTC_F32 : x_dt, M, K, s);
        if (rc != BTC_OK) return rc;
        a.x = ws;
        if (xt_f32) a.x_dt = BTC_F32;
        a.workspace = static_cast<char *>(ws) + xt_bytes;
        a.workspace_bytes = ws_bytes - xt_bytes;
    }

    rc = BTC_ERR_UNSUPPORTED;
    if (path == PATH_GEMV || M <= 8) {
        // the decode kernel (integer form up to two rows of x, fp16 form above; the older fp16 kernel where the table
        // does not fit shared memory); for M = 5..8 with few row tiles and a
        // very long K the tensor-core launch with K split over the SMs, when the workspace has room for its partial
        // sums; the older fp16 kernel and the any-shape kernel take what the first does not cover
        if (M > 2 && a.x_dt != BTC_F32 && gemm_tcgen05_small_m_pays(M, N, K, v)) rc = launch_gemm_tcgen05(a, s, true);
        // M = 3..8, one layer per call: the older fp16 kernel (a CTA per row tile over the whole K) is the faster one --
        // 8.5 against 10.1 us for 4096 x 4096 at M = 3, 15.8 against 24.6 us for 4096 x 11008, 13.8 against 19.6 us for
        // 5120 x 5120 with 65536 centroids at M = 4; the newer fp16 form earns its keep in the fused multi-layer launch
        if (rc == BTC_ERR_UNSUPPORTED && M > 2 && a.x_dt != BTC_F32) rc = launch_gemv_decode(a, s);
        if (rc == BTC_ERR_UNSUPPORTED && M <= 2) rc = launch_gemv_imma_wide(&a, 1, s);     // (plain launches at M <= 2: the faster geometry)
        if (rc == BTC_ERR_UNSUPPORTED) rc = launch_gemv_imma(&a, 1, s);
        if (rc == BTC_ERR_UNSUPPORTED) rc = launch_gemv_decode(a, s);
    }
    else rc = launch_gemm_tcgen05(a, s);
    if (rc == BTC_ERR_UNSUPPORTED) {
        if (path == PATH_GEMM && M <= 8) rc = launch_gemv_decode(a, s);
        if (rc == BTC_ERR_UNSUPPORTED) rc = launch_linear_generic(a, s);
    }
    return rc;
}

}  // namespace btc

using namespace btc;

extern "C" int btc_version(void) { return 100; }

extern "C" const char *btc_status_string(int st)
{
    switch (st) {
    case BTC_OK: return "ok";
    case BTC_ERR_NULL: return "a required pointer is NULL";
    case BTC_ERR_SHAPE: return "shape out of range (1<=v<=32, v divides K, 1<=Kc<=65536, M,N,K>=1; gemv needs M<=8)";
    case BTC_ERR_ALIGN: return "pointer alignment (x, idx, y, C_packed: 16 bytes; workspace: 256 bytes)";
    case BTC_ERR_UNSUPPORTED: return "dtype or option not supported";
    case BTC_ERR_WORKSPACE: return "workspace missing or too small";
    case BTC_ERR_CUDA: return "CUDA call failed (see btc_last_cuda_error)";
    case BTC_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case BTC_ERR_INDEX: return "an index >= Kc was seen (debug check, BTC_DEBUG_CHECK_INDICES=1)";
    default: return "unknown status";
    }
}

extern "C" int btc_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" size_t btc_codebook_packed_bytes(int Kc, int v)
{
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536) return 0;
    // three sections of (Kc rounded up to 4) 32-bit words and one of (Kc rounded up to 8) 16-bit halves
    return (size_t)((Kc + 3) / 4 * 4) * 12 + (size_t)((Kc + 7) / 8 * 8) * 2;
}

extern "C" size_t btc_linear_workspace_bytes(int M, int N, int K, int v, int Kc)
{
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || M < 1 || N < 1 || K < 1 || K % v) return 0;
    size_t a = (M <= 8) ? gemv_decode_workspace_bytes(M, N, K, v, Kc) : 0;
    size_t b = gemm_tcgen05_workspace_bytes(M, N, K, v, Kc);
    size_t w = a > b ? a : b;
    return (w + 255) / 256 * 256;
}

extern "C" size_t btc_linear_workspace_bytes_ex(int M, int N, int K, int v, int Kc, int has_transform)
{
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || M < 1 || N < 1 || K < 1 || K % v) return 0;
    return btc_linear_workspace_bytes(M, N, K, v, Kc) + (has_transform ? transform_bytes(M, K, v) : 0);
}

extern "C" int btc_linear_gemv(const void *x, int x_dtype, const uint16_t *idx, const uint32_t *C_packed,
                               const void *alpha, const void *mu, const btc_transform *T, void *y, int y_dtype,
                               int M, int N, int K, int v, int Kc, void *workspace, size_t workspace_bytes,
                               void *stream)
{
    return run_linear(PATH_GEMV, x, x_dtype, idx, C_packed, alpha, mu, T, y, y_dtype, M, N, K, v, Kc,
                      workspace, workspace_bytes, stream);
}

extern "C" int btc_linear_gemm(const void *x, int x_dtype, const uint16_t *idx, const uint32_t *C_packed,
                               const void *alpha, const void *mu, const btc_transform *T, void *y, int y_dtype,
                               int M, int N, int K, int v, int Kc, void *workspace, size_t workspace_bytes,
                               void *stream)
{
    return run_linear(PATH_GEMM, x, x_dtype, idx, C_packed, alpha, mu, T, y, y_dtype, M, N, K, v, Kc,
                      workspace, workspace_bytes, stream);
}

namespace btc {
static int run_batch(const btc_linear_problem *problems, int count, void *stream, int accumulate_from, int max_group);
}

extern "C" int btc_linear_gemv_batch(const btc_linear_problem *problems, int count, void *stream)
{
    return btc::run_batch(problems, count, stream, 0, IM_MAXP);
}

extern "C" int btc_linear_gemv_sum(const btc_linear_problem *terms, int count, void *stream)
{
    if (!terms) return BTC_ERR_NULL;
    if (count < 1) return BTC_ERR_SHAPE;
    for (int i = 1; i < count; ++i)
        if (terms[i].y != terms[0].y || terms[i].M != terms[0].M || terms[i].N != terms[0].N || terms[i].y_dtype != terms[0].y_dtype)
            return BTC_ERR_SHAPE;
    if (count > 1 && terms[0].y_dtype != BTC_F32) return BTC_ERR_UNSUPPORTED;
    // one launch per term, in order on the stream: the first writes y, every later one adds to it
    return btc::run_batch(terms, count, stream, 1, 1);
}

// accumulate_from > 0: problems with index >= accumulate_from add to y; max_group: layers per launch
static int btc::run_batch(const btc_linear_problem *problems, int count, void *stream, int accumulate_from, int max_group)
{
    if (!problems) return BTC_ERR_NULL;
    if (count < 1) return BTC_ERR_SHAPE;
    cudaStream_t s = (cudaStream_t)stream;
    LinearArgs group[IM_MAXP];
    int i = 0;
    while (i < count) {
        // longest run of layers (at most IM_MAXP) starting at i
        int n = 0;
        for (; n < max_group && i + n < count; ++n) {
            const btc_linear_problem &p = problems[i + n];
            // fp32 activations (what btc_activation_transform hands over) are the decode kernel's alone: they are
            // accepted where that kernel covers the layer
            const bool x_f32 = p.x_dtype == BTC_F32;
            if (x_f32 && !(p.v >= 4 && p.v % 4 == 0 && p.v <= 20 && p.K % p.v == 0 && (p.K / p.v) % 8 == 0 && p.K % 8 == 0 && p.M <= 8))
                return BTC_ERR_UNSUPPORTED;
            int rc = validate(p.x, x_f32 ? (int)BTC_F16 : p.x_dtype, static_cast<const uint16_t *>(p.idx), p.C_packed, p.alpha, p.y, p.y_dtype, p.M, p.N, p.K, p.v, p.Kc);
            if (rc != BTC_OK) return rc;
            if (p.mu && !aligned(p.mu, 2)) return BTC_ERR_ALIGN;
            if (p.M > 8) return BTC_ERR_SHAPE;
            if (debug_check_indices_enabled() && (p.idx_bits == 0 || p.idx_bits == 16) && p.idx_stride == 0) {
                rc = launch_index_check(static_cast<const uint16_t *>(p.idx), (size_t)p.N * (p.K / p.v), p.Kc, s);
                if (rc != BTC_OK) return rc;
            }
            LinearArgs &a = group[n];
            a = LinearArgs();
            if (p.idx_bits != 0 && p.idx_bits != 16) {
                // dense-packed rows: the width must be the codebook's index width
                if (p.idx_bits != btc_index_bits(p.Kc)) return BTC_ERR_SHAPE;
                a.idx_bits = p.idx_bits;
                a.idx_packed = p.idx;
                a.idx_pitch = btc_index_packed_row_bytes(p.K / p.v, p.Kc);
            }
            a.x = p.x; a.idx = static_cast<const uint16_t *>(p.idx); a.Cp = p.C_packed;
            a.x_stride = p.x_stride; a.idx_stride = p.idx_stride; a.accumulate = accumulate_from > 0 && (i + n) >= accumulate_from ? 1 : 0;
            a.alpha = reinterpret_cast<const __half *>(p.alpha);
            a.mu = reinterpret_cast<const __half *>(p.mu);
            a.y = p.y; a.workspace = nullptr; a.workspace_bytes = 0;
            a.x_dt = p.x_dtype; a.y_dt = p.y_dtype;
            a.M = p.M; a.N = p.N; a.K = p.K; a.v = p.v; a.Kc = p.Kc; a.Kb = p.K / p.v;
        }
        // plain launches at M <= 2 take the one-CTA-per-SM geometry (it declines anything else); a sum of terms never does,
        // so that all its terms share one arithmetic
        int rc = accumulate_from > 0 ? BTC_ERR_UNSUPPORTED : launch_gemv_imma_wide(group, n, s);
        // a run of one plain layer at M = 3..8: the older fp16 kernel, as in btc_linear_gemv
        if (rc == BTC_ERR_UNSUPPORTED && n == 1 && accumulate_from == 0 && group[0].M > 2 && group[0].x_dt != BTC_F32 &&
            !group[0].idx_bits && !group[0].x_stride && !group[0].idx_stride)
            rc = launch_gemv_decode(group[0], s);
        if (rc == BTC_ERR_UNSUPPORTED) rc = launch_gemv_imma(group, n, s);
        if (rc == BTC_ERR_UNSUPPORTED) {
            // some layer of the run is outside the fused kernel: one launch per layer instead
            for (int k = 0; k < n; ++k) {
                rc = accumulate_from > 0 ? BTC_ERR_UNSUPPORTED : launch_gemv_imma_wide(&group[k], 1, s);
                if (rc == BTC_ERR_UNSUPPORTED) rc = launch_gemv_imma(&group[k], 1, s);
                // only the decode kernel reads dense indices, fp32 activations, column ranges of wider matrices, or adds to y
                if (rc == BTC_ERR_UNSUPPORTED && (group[k].idx_bits || group[k].x_stride || group[k].idx_stride || group[k].accumulate ||
                                                  group[k].x_dt == BTC_F32)) return rc;
                if (rc == BTC_ERR_UNSUPPORTED) rc = launch_gemv_decode(group[k], s);
                if (rc == BTC_ERR_UNSUPPORTED) rc = launch_linear_generic(group[k], s);
                if (rc != BTC_OK) return rc;
            }
        } else if (rc != BTC_OK) {
            return rc;
        }
        i += n;
    }
    return BTC_OK;
}

extern "C" int btc_activation_transform(const void *x, int x_dtype, const btc_transform *T, void *xt, int xt_dtype, int M, int K,
                                       void *stream)
{
    if (!x || !T || !xt || !T->sigma_bits || !T->P1 || !T->P2) return BTC_ERR_NULL;
    if (M < 1 || K < 1 || T->k1 < 1 || T->k2 < 1 || (long long)T->k1 * T->k2 != K) return BTC_ERR_SHAPE;
    if (x_dtype != BTC_F16 && x_dtype != BTC_BF16) return BTC_ERR_UNSUPPORTED;
    if (xt_dtype != BTC_F32 && xt_dtype != x_dtype) return BTC_ERR_UNSUPPORTED;
    if (!aligned(x, 16) || !aligned(xt, 16)) return BTC_ERR_ALIGN;
    return launch_transform(x, x_dtype, *T, xt, xt_dtype, M, K, (cudaStream_t)stream);
}

extern "C" double btc_bits_per_weight(int N, int K, int v, int Kc, int scale_bits_per_row, int mode,
                                      int with_codebook)
{
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || N < 1 || K < 1 || mode < 0 || mode > 2) return -1.0;
    double ib;
    if (mode == 0) ib = std::log2((double)Kc);
    else if (mode == 1) { int b = 0; while ((1 << b) < Kc) ++b; ib = b; }
    else ib = 16.0;
    double r = ib / v + (double)scale_bits_per_row / K;
    if (with_codebook) r += (double)v * Kc / ((double)N * K);
    return r;
}

extern "C" int btc_linear_gemv_packed(const void *x, int x_dtype, const void *idx_packed, const uint32_t *C_packed,
                                      const void *alpha, const void *mu, void *y, int y_dtype, int M, int N, int K,
                                      int v, int Kc, void *stream)
{
    btc_linear_problem p = {};
    p.x = x; p.idx = idx_packed; p.C_packed = C_packed; p.alpha = alpha; p.mu = mu; p.y = y;
    p.x_dtype = x_dtype; p.y_dtype = y_dtype; p.M = M; p.N = N; p.K = K; p.v = v; p.Kc = Kc;
    p.idx_bits = btc_index_bits(Kc);
    if (p.idx_bits == 16) p.idx_bits = 0;                    // 16-bit fields ARE the uint16 container
    return btc_linear_gemv_batch(&p, 1, stream);
}
