// Online activation transform  x' = x * D * (P1 (x) P2),  D = diag(sigma), sigma in {+1,-1}
// (paper Section 4.2 "Transformation Pair": learnable sign flips and a Kronecker-factored matrix, applied
// at inference as X <- X T).  With a row of x viewed row-major as a k1 x k2 matrix X (k1 * k2 = K):
//     X' = P1^T (X o sigma) P2,     X'[c][d] = sum_a sum_b P1[a][c] * sigma[a k2 + b] * X[a][b] * P2[b][d]
// computed as two small products with fp32 accumulation: Y = (X o sigma) P2, then X' = P1^T Y.
// One CTA per row of x; X and Y live in shared memory.  The result is rounded to the dtype of x, because
// the linear kernels take fp16 / bf16 activations.
#include "btc_internal.cuh"

namespace btc {

constexpr int TR_THREADS = 512;

__global__ void __launch_bounds__(TR_THREADS)
transform_kernel(const void *__restrict__ x, int x_dt, const uint32_t *__restrict__ sigma_bits,
                 const float *__restrict__ P1, const float *__restrict__ P2, int k1, int k2, void *__restrict__ xt)
{
    extern __shared__ float tr_smem[];
    const int K = k1 * k2;
    float *X = tr_smem, *Y = tr_smem + K;
    const size_t row = (size_t)blockIdx.x * K;
    for (int i = threadIdx.x; i < K; i += TR_THREADS) {
        float v = load_as_float(x, x_dt, row + i);
        if ((sigma_bits[i >> 5] >> (i & 31)) & 1u) v = -v;
        X[i] = v;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < K; o += TR_THREADS) {          // Y[a][d] = sum_b X[a][b] * P2[b][d]
        const int a = o / k2, d = o - a * k2;
        float s = 0.f;
        for (int b = 0; b < k2; ++b) s = fmaf(X[a * k2 + b], __ldg(P2 + (size_t)b * k2 + d), s);
        Y[o] = s;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < K; o += TR_THREADS) {          // X'[c][d] = sum_a P1[a][c] * Y[a][d]
        const int c = o / k2, d = o - c * k2;
        float s = 0.f;
        for (int a = 0; a < k1; ++a) s = fmaf(__ldg(P1 + (size_t)a * k1 + c), Y[a * k2 + d], s);
        store_from_float(xt, x_dt, row + o, s);
    }
}

int launch_transform(const void *x, int x_dt, const btc_transform &T, void *xt, int M, int K, cudaStream_t s)
{
    if ((long long)T.k1 * T.k2 != K) return BTC_ERR_SHAPE;
    const size_t smem = (size_t)2 * K * sizeof(float);
    if (smem > 200 * 1024) return BTC_ERR_UNSUPPORTED;           // K up to 25600
    cudaError_t e = cudaFuncSetAttribute(transform_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    transform_kernel<<<M, TR_THREADS, smem, s>>>(x, x_dt, T.sigma_bits, T.P1, T.P2, T.k1, T.k2, xt);
    return cuda_check_launch();
}

}  // namespace btc
