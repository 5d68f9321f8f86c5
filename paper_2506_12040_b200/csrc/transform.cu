// Online activation transform  x' = x * D * (P1 (x) P2),  D = diag(sigma), sigma in {+1,-1}
// (paper Section 4.2 "Transformation Pair": learnable sign flips and a Kronecker-factored matrix, applied
// at inference as X <- X T).  With a row of x viewed row-major as a k1 x k2 matrix X (k1 * k2 = K):
//     X' = P1^T (X o sigma) P2,     X'[c][d] = sum_a sum_b P1[a][c] * sigma[a k2 + b] * X[a][b] * P2[b][d]
// computed as two small products with fp32 accumulation: Y = (X o sigma) P2, then X' = P1^T Y.
// A CTA owns one row of x and a tile of TR_DT output columns d: it needs all of X (K values), the k2 x TR_DT slab of
// P2 and all of P1, and produces X'[:, d-tile]; a decode step with one row of x therefore spreads over k2 / TR_DT SMs
// instead of one.  The result is written as fp32 for the decode path (which quantises or rounds the activations
// itself, so no intermediate 16-bit rounding is added) and in the dtype of x for the tensor-core path.
#include "btc_internal.cuh"

namespace btc {

constexpr int TR_THREADS = 256;
constexpr int TR_DT = 8;            // output columns d per CTA

__global__ void __launch_bounds__(TR_THREADS)
transform_kernel(const void *__restrict__ x, int x_dt, const uint32_t *__restrict__ sigma_bits,
                 const float *__restrict__ P1, const float *__restrict__ P2, int k1, int k2, void *__restrict__ xt, int out_dt)
{
    extern __shared__ float tr_smem[];
    const int K = k1 * k2;
    const int d0 = blockIdx.x * TR_DT, nd = min(TR_DT, k2 - d0);
    float *X = tr_smem;                    // [k1][k2]   (sign-flipped activations)
    float *Pd = X + K;                     // [k2][TR_DT] slab of P2
    float *Y = Pd + k2 * TR_DT;            // [k1][TR_DT]
    const size_t row = (size_t)blockIdx.y * K;
    for (int i = threadIdx.x; i < K; i += TR_THREADS) {
        float v = load_as_float(x, x_dt, row + i);
        if ((sigma_bits[i >> 5] >> (i & 31)) & 1u) v = -v;
        X[i] = v;
    }
    for (int i = threadIdx.x; i < k2 * TR_DT; i += TR_THREADS) {
        const int b = i / TR_DT, d = i - b * TR_DT;
        Pd[i] = d < nd ? __ldg(P2 + (size_t)b * k2 + d0 + d) : 0.f;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < k1 * TR_DT; o += TR_THREADS) {       // Y[a][d] = sum_b X[a][b] * P2[b][d0 + d]
        const int a = o / TR_DT, d = o - a * TR_DT;
        float s = 0.f;
        for (int b = 0; b < k2; ++b) s = fmaf(X[a * k2 + b], Pd[b * TR_DT + d], s);
        Y[o] = s;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < k1 * TR_DT; o += TR_THREADS) {       // X'[c][d0 + d] = sum_a P1[a][c] * Y[a][d]
        const int c = o / TR_DT, d = o - c * TR_DT;
        if (d >= nd) continue;
        float s = 0.f;
        for (int a = 0; a < k1; ++a) s = fmaf(__ldg(P1 + (size_t)a * k1 + c), Y[a * TR_DT + d], s);
        store_from_float(xt, out_dt, row + (size_t)c * k2 + d0 + d, s);
    }
}

int launch_transform(const void *x, int x_dt, const btc_transform &T, void *xt, int out_dt, int M, int K, cudaStream_t s)
{
    if ((long long)T.k1 * T.k2 != K) return BTC_ERR_SHAPE;
    const size_t smem = ((size_t)K + (size_t)T.k2 * TR_DT + (size_t)T.k1 * TR_DT) * sizeof(float);
    if (smem > 200 * 1024 || M > 65535) return BTC_ERR_UNSUPPORTED;       // K up to about 50000
    cudaError_t e = cudaFuncSetAttribute(transform_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    transform_kernel<<<dim3((unsigned)((T.k2 + TR_DT - 1) / TR_DT), (unsigned)M), TR_THREADS, smem, s>>>(
        x, x_dt, T.sigma_bits, T.P1, T.P2, T.k1, T.k2, xt, out_dt);
    return cuda_check_launch();
}

}  // namespace btc
