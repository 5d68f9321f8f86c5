// Internal declarations shared by the translation units of the library (not installed).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "btc.h"

namespace btc {

struct LinearArgs {
    const void *x;
    const uint16_t *idx;
    const uint32_t *Cp;
    const __half *alpha;
    const __half *mu;      // may be nullptr
    void *y;
    void *workspace;
    size_t workspace_bytes;
    int x_dt, y_dt;
    int M, N, K, v, Kc, Kb;   // Kb = K / v
    // dense-packed indices (idx_bits > 0): idx is unused, idx_packed holds rows of idx_pitch bytes, idx_bits bits per index
    const void *idx_packed = nullptr;
    size_t idx_pitch = 0;
    int idx_bits = 0;
    // a term of a sum of layers: x / idx may be column ranges of wider matrices (row strides in elements, 0 = dense),
    // and the result may be added to y (fp32) instead of overwriting it
    int x_stride = 0;
    int idx_stride = 0;
    int accumulate = 0;
};

// Records a CUDA error for btc_last_cuda_error() and maps it to BTC_ERR_CUDA.
int cuda_fail(cudaError_t e);
inline int cuda_check_launch() {
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? BTC_OK : cuda_fail(e);
}

// gemv_generic.cu: any v / Kc / M (M is tiled by 8 over grid.y), plain CUDA cores.
int launch_linear_generic(const LinearArgs &a, cudaStream_t s);

// gemv_decode.cu: the tuned decode path (M <= 8).  Returns BTC_ERR_UNSUPPORTED when the shape
// is outside what it covers, in which case the caller falls back to the generic kernel.
int launch_gemv_decode(const LinearArgs &a, cudaStream_t s);
size_t gemv_decode_workspace_bytes(int M, int N, int K, int v, int Kc);

// gemm_tcgen05.cu: tensor-core path.  Same UNSUPPORTED convention.
int launch_gemm_tcgen05(const LinearArgs &a, cudaStream_t s, bool small_m = false);   // small_m: also 5 <= M <= 8 where it pays
bool gemm_tcgen05_small_m_pays(int M, int N, int K, int v);
size_t gemm_tcgen05_workspace_bytes(int M, int N, int K, int v, int Kc);   // with room for a K split where one pays
size_t gemm_tcgen05_workspace_min(int M);                                 // what the kernels cannot do without

// gemv_imma.cu: integer-MMA decode path; runs up to IM_MAXP independent layers (M <= 8 each) in one launch.
// Returns BTC_ERR_UNSUPPORTED when a shape is outside what it covers (nothing is launched then).
constexpr int IM_MAXP = 8;
int launch_gemv_imma(const LinearArgs *problems, int count, cudaStream_t s);
int imma_status_read(int *out);
int imma_status_reset();
int imma_selftest_wait(cudaStream_t s);

// pack.cu: debug check of the index range (BTC_DEBUG_CHECK_INDICES=1) and its status word.
bool debug_check_indices_enabled();
int launch_index_check(const uint16_t *idx, size_t count, int Kc, cudaStream_t s);
int index_status_read(int *out);
int index_status_reset();

// gemv_lut.cu: the paper's two-stage lookup scheme (alternative route, own entry point).
int launch_gemv_lut(const LinearArgs &a, cudaStream_t s);
size_t gemv_lut_workspace_bytes(int M, int N, int K, int v);

// gemv_imma_wide.cu: the integer form for M <= 2 in its one-CTA-per-SM geometry (plain launches only; UNSUPPORTED otherwise).
int launch_gemv_imma_wide(const LinearArgs *problems, int count, cudaStream_t s);
int wide_status_read(int *out);
int wide_status_reset();

// transform.cu: x' = x * D * (P1 (x) P2) into xt (same shape as x, dtype out_dt).
int launch_transform(const void *x, int x_dt, const btc_transform &T, void *xt, int out_dt, int M, int K,
                     cudaStream_t s);

// ---- small device helpers ------------------------------------------------------------------
__device__ __forceinline__ float load_as_float(const void *p, int dt, size_t i) {
    if (dt == BTC_F16) return __half2float(reinterpret_cast<const __half *>(p)[i]);
    if (dt == BTC_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p)[i]);
    return reinterpret_cast<const float *>(p)[i];
}
__device__ __forceinline__ void store_from_float(void *p, int dt, size_t i, float f) {
    if (dt == BTC_F32) reinterpret_cast<float *>(p)[i] = f;
    else if (dt == BTC_F16) reinterpret_cast<__half *>(p)[i] = __float2half_rn(f);
    else reinterpret_cast<__nv_bfloat16 *>(p)[i] = __float2bfloat16_rn(f);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace btc
