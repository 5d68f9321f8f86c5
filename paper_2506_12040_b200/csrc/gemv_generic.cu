// Generic codebook-binary linear kernel: any v in [1,32], any Kc, any M.
// One warp per output row; lanes stride over the K/v blocks of that row, look the centroid word
// up in global memory (L1/L2 cached) and accumulate the signed sum  sum_t s_t * x_t  in fp32
// (block dot of the paper's appendix, second display).  Used for shapes the tuned kernels do
// not cover; correctness first, no tiling tricks.
#include "btc_internal.cuh"

namespace btc {

constexpr int GEN_WARPS = 8;
constexpr int GEN_MT = 8;   // rows of x per CTA

__global__ void __launch_bounds__(GEN_WARPS * 32)
linear_generic_kernel(LinearArgs a)
{
    __shared__ float s_sumx[GEN_MT];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int m0 = blockIdx.y * GEN_MT;
    const int mt = min(GEN_MT, a.M - m0);

    if (a.mu != nullptr) {
        // sum_k x[m,k] for the mean term, one warp per row of x
        for (int m = warp; m < mt; m += GEN_WARPS) {
            float s = 0.f;
            for (int k = lane; k < a.K; k += 32) s += load_as_float(a.x, a.x_dt, (size_t)(m0 + m) * a.K + k);
            s = warp_sum(s);
            if (lane == 0) s_sumx[m] = s;
        }
        __syncthreads();
    }

    const int n = blockIdx.x * GEN_WARPS + warp;
    if (n >= a.N) return;

    float acc[GEN_MT];
#pragma unroll
    for (int m = 0; m < GEN_MT; ++m) acc[m] = 0.f;

    const uint16_t *row = a.idx + (size_t)n * a.Kb;
    for (int j = lane; j < a.Kb; j += 32) {
        const uint32_t w = __ldg(a.Cp + row[j]);
        const size_t k0 = (size_t)j * a.v;
        for (int t = 0; t < a.v; ++t) {
            const bool plus = (w >> t) & 1u;
#pragma unroll
            for (int m = 0; m < GEN_MT; ++m) {
                if (m < mt) {
                    const float xv = load_as_float(a.x, a.x_dt, (size_t)(m0 + m) * a.K + k0 + t);
                    acc[m] += plus ? xv : -xv;
                }
            }
        }
    }
    const float al = __half2float(a.alpha[n]);
    const float mu = a.mu ? __half2float(a.mu[n]) : 0.f;
#pragma unroll
    for (int m = 0; m < GEN_MT; ++m) {
        if (m < mt) {
            float s = warp_sum(acc[m]);
            if (lane == 0) {
                float r = al * s;
                if (a.mu) r += mu * s_sumx[m];
                store_from_float(a.y, a.y_dt, (size_t)(m0 + m) * a.N + n, r);
            }
        }
    }
}

int launch_linear_generic(const LinearArgs &a, cudaStream_t s)
{
    const long long gy = (a.M + GEN_MT - 1) / GEN_MT;
    if (gy > 65535) return BTC_ERR_SHAPE;
    dim3 grid((a.N + GEN_WARPS - 1) / GEN_WARPS, (unsigned)gy);
    linear_generic_kernel<<<grid, GEN_WARPS * 32, 0, s>>>(a);
    return cuda_check_launch();
}

}  // namespace btc
