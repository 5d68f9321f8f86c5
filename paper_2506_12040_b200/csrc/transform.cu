// Online activation transform  x' = x * D * (P1 (x) P2),  D = diag(sigma), sigma in {+1,-1}
// (paper Section 4.2 "Transformation Pair": learnable sign flips and a Kronecker-factored matrix, applied
// at inference as X <- X T).  With a row of x viewed row-major as a k1 x k2 matrix X (k1 * k2 = K):
//     X' = P1^T (X o sigma) P2,     X'[c][d] = sum_a sum_b P1[a][c] * sigma[a k2 + b] * X[a][b] * P2[b][d]
// computed as two small products with fp32 accumulation: Y = (X o sigma) P2, then X' = P1^T Y.
// A CTA owns a tile of TR_DT output columns d and a group of rows of x: it stages the k2 x TR_DT slab of P2 and all
// of P1 in shared memory once, then for each of its rows loads X (K values) and produces X'[:, d-tile]; a decode step
// with one row of x therefore spreads over k2 / TR_DT SMs instead of one, and a prefill batch shares the staged factors.  The result is written as fp32 for the decode path (which quantises or rounds the activations
// itself, so no intermediate 16-bit rounding is added) and in the dtype of x for the tensor-core path.
#include "btc_internal.cuh"

namespace btc {

constexpr int TR_THREADS = 256;
constexpr int TR_DT = 8;            // output columns d per CTA

__global__ void __launch_bounds__(TR_THREADS)
transform_kernel(const void *__restrict__ x, int x_dt, const uint32_t *__restrict__ sigma_bits,
                 const float *__restrict__ P1, const float *__restrict__ P2, int k1, int k2, void *__restrict__ xt, int out_dt,
                 int M, int rows_per_cta)
{
    extern __shared__ float tr_smem[];
    // (the layer kernel that follows may start right away and prefetch its indices; it reads x' only after this grid
    // has completed)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int K = k1 * k2;
    const int d0 = blockIdx.x * TR_DT, nd = min(TR_DT, k2 - d0);
    const int xp = k2 + 4;                 // X row pitch: four words of padding put the 8 rows x 4 lanes of a warp on 32 banks
    const int kp = k1 + 8;                 // P1 row pitch, for the same reason
    float *X = tr_smem;                    // [k1][xp]   (sign-flipped activations of the current row)
    float *Pd = X + ((k1 * xp + 3) & ~3);                     // [k2][TR_DT] slab of P2
    float *Y = Pd + k2 * TR_DT;            // [k1][TR_DT]
    float *Q1 = Y + k1 * TR_DT;            // [k1][kp]   P1, staged once per CTA
    for (int i = threadIdx.x; i < k2 * TR_DT; i += TR_THREADS) {
        const int b = i / TR_DT, d = i - b * TR_DT;
        Pd[i] = d < nd ? __ldg(P2 + (size_t)b * k2 + d0 + d) : 0.f;
    }
    for (int i = threadIdx.x; i < k1 * k1; i += TR_THREADS) Q1[(i / k1) * kp + (i % k1)] = __ldg(P1 + i);
    const int m0 = blockIdx.y * rows_per_cta, m1 = min(M, m0 + rows_per_cta);
    for (int m = m0; m < m1; ++m) {
        const size_t row = (size_t)m * K;
        __syncthreads();                   // (previous row's X and Y are no longer read; P slabs are in place)
        if (x_dt != BTC_F32 && (k2 & 7) == 0) {
            // 16-bit activations, eight per 16-byte load (rows are 16-byte aligned when 8 divides K)
            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(x) + row);
            for (int i = threadIdx.x; i < K / 8; i += TR_THREADS) {
                const uint4 q = __ldg(src + i);
                const uint32_t sg = __ldg(sigma_bits + (i >> 2)) >> ((i & 3) * 8);
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
                const int rr = 4 * ((8 * i) / k2);     // the eight elements share a row of X (8 divides k2 here)
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    float lo, hi;
                    if (x_dt == BTC_F16) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[h]));
                        lo = f.x; hi = f.y;
                    } else {
                        lo = __uint_as_float(w[h] << 16); hi = __uint_as_float(w[h] & 0xffff0000u);
                    }
                    const int e0 = 8 * i + 2 * h;                                    // element e of row r sits at e + 4 r
                    X[e0 + rr] = ((sg >> (2 * h)) & 1u) ? -lo : lo;
                    X[e0 + 1 + rr] = ((sg >> (2 * h + 1)) & 1u) ? -hi : hi;
                }
            }
        } else {
            for (int i = threadIdx.x; i < K; i += TR_THREADS) {
                float v = load_as_float(x, x_dt, row + i);
                if ((__ldg(sigma_bits + (i >> 5)) >> (i & 31)) & 1u) v = -v;
                X[i + 4 * (i / k2)] = v;
            }
        }
        __syncthreads();
        // Y[a][d] = sum_b X[a][b] * P2[b][d0 + d]: four lanes share a row a, each sums a quarter of b for all TR_DT columns
        // (one X value and one slab row per 8 FMAs), then the quad adds up
        for (int w0 = 0; w0 < k1 * 4; w0 += TR_THREADS) {
            const int w = w0 + threadIdx.x, a = w >> 2, q = w & 3;
            float acc[TR_DT];
#pragma unroll
            for (int d = 0; d < TR_DT; ++d) acc[d] = 0.f;
            if (a < k1) {
                const float *xa = X + (size_t)a * xp;
                for (int b = q; b < k2; b += 4) {                      // (interleaved quarters: the quad reads four neighbouring slab rows)
                    const float xv = xa[b];
                    const float4 p0 = *reinterpret_cast<const float4 *>(Pd + b * TR_DT), p1 = *reinterpret_cast<const float4 *>(Pd + b * TR_DT + 4);
                    acc[0] = fmaf(xv, p0.x, acc[0]); acc[1] = fmaf(xv, p0.y, acc[1]); acc[2] = fmaf(xv, p0.z, acc[2]); acc[3] = fmaf(xv, p0.w, acc[3]);
                    acc[4] = fmaf(xv, p1.x, acc[4]); acc[5] = fmaf(xv, p1.y, acc[5]); acc[6] = fmaf(xv, p1.z, acc[6]); acc[7] = fmaf(xv, p1.w, acc[7]);
                }
            }
#pragma unroll
            for (int d = 0; d < TR_DT; ++d) {
                acc[d] += __shfl_xor_sync(0xffffffffu, acc[d], 1);
                acc[d] += __shfl_xor_sync(0xffffffffu, acc[d], 2);
            }
            if (a < k1 && q == 0) {
                *reinterpret_cast<float4 *>(Y + a * TR_DT) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                *reinterpret_cast<float4 *>(Y + a * TR_DT + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
            }
        }
        __syncthreads();
        // X'[c][d0 + d] = sum_a P1[a][c] * Y[a][d]: the same split, quarters of a
        for (int w0 = 0; w0 < k1 * 4; w0 += TR_THREADS) {
            const int w = w0 + threadIdx.x, c = w >> 2, q = w & 3;
            float acc[TR_DT];
#pragma unroll
            for (int d = 0; d < TR_DT; ++d) acc[d] = 0.f;
            if (c < k1) {
                for (int a = q; a < k1; a += 4) {
                    const float pv = Q1[a * kp + c];
                    const float4 y0 = *reinterpret_cast<const float4 *>(Y + a * TR_DT), y1 = *reinterpret_cast<const float4 *>(Y + a * TR_DT + 4);
                    acc[0] = fmaf(pv, y0.x, acc[0]); acc[1] = fmaf(pv, y0.y, acc[1]); acc[2] = fmaf(pv, y0.z, acc[2]); acc[3] = fmaf(pv, y0.w, acc[3]);
                    acc[4] = fmaf(pv, y1.x, acc[4]); acc[5] = fmaf(pv, y1.y, acc[5]); acc[6] = fmaf(pv, y1.z, acc[6]); acc[7] = fmaf(pv, y1.w, acc[7]);
                }
            }
#pragma unroll
            for (int d = 0; d < TR_DT; ++d) {
                acc[d] += __shfl_xor_sync(0xffffffffu, acc[d], 1);
                acc[d] += __shfl_xor_sync(0xffffffffu, acc[d], 2);
            }
            if (c < k1 && q == 0) {
#pragma unroll
                for (int d = 0; d < TR_DT; ++d)
                    if (d < nd) store_from_float(xt, out_dt, row + (size_t)c * k2 + d0 + d, acc[d]);
            }
        }
    }
}

int launch_transform(const void *x, int x_dt, const btc_transform &T, void *xt, int out_dt, int M, int K, cudaStream_t s)
{
    if ((long long)T.k1 * T.k2 != K) return BTC_ERR_SHAPE;
    const size_t smem = ((size_t)K + 4 * T.k1 + 4 + (size_t)T.k2 * TR_DT + (size_t)T.k1 * TR_DT + (size_t)T.k1 * (T.k1 + 8)) * sizeof(float);
    if (smem > 200 * 1024) return BTC_ERR_UNSUPPORTED;
    cudaError_t e = cudaFuncSetAttribute(transform_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    // rows per CTA: about two CTAs per SM in all (the P slabs are staged once per CTA and serve all its rows)
    const int tiles = (T.k2 + TR_DT - 1) / TR_DT;
    int groups = (2 * 148 + tiles - 1) / tiles;
    if (groups > M) groups = M;
    const int rows = (M + groups - 1) / groups;
    groups = (M + rows - 1) / rows;
    if (groups > 65535) return BTC_ERR_UNSUPPORTED;
    transform_kernel<<<dim3((unsigned)tiles, (unsigned)groups), TR_THREADS, smem, s>>>(
        x, x_dt, T.sigma_bits, T.P1, T.P2, T.k1, T.k2, xt, out_dt, M, rows);
    return cuda_check_launch();
}

}  // namespace btc
