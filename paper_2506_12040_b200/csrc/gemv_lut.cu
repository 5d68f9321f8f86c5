// The paper's own kernel scheme for the layer, kept as an alternative to the MMA decode path: the two-stage lookup of
// the appendix "Binary codebook LUT-GEMM".
//   Stage I  (activation LUT):  every block x_j is cut into P = v / mu segments of mu activations (mu = 8 when 8 divides
//            v, else 4); LUT_{j,p}[s] = sum_t sigma_t(s) * x_{j,p}[t] over the 2^mu sign patterns s (bit t of s set <=> +1).
//   Stage II (codebook LUT):    CBLUT_j[k] = sum_p LUT_{j,p}[key[k, p]],  key[k, p] = bits p*mu .. p*mu+mu-1 of the packed
//            codeword k (the "keys precomputed offline" are the public packed words themselves).
//   Gather:                     y_r = alpha_r * sum_j CBLUT_j[I_{r,j}]  (+ mu_r * sum_k x_k): one lookup and one add per
//            (row, block).
// Placement follows the appendix: both tables in shared memory, CBLUT entries in fp16 (the paper packs half2 entries),
// the row sums in fp32.  A CTA owns LB consecutive blocks of K (its tables) and a chunk of rows; since a CBLUT has Kc
// entries per block whatever the number of rows, every CTA of a K-slice rebuilds it: the build costs Kc * K/v * P
// lookups per layer against N * K/v gathers, which is why this scheme only pays when N is much larger than Kc.
// K-slices meet through a workspace of partial sums, added in slice order by a second kernel (deterministic).
#include "btc_internal.cuh"

namespace btc {

constexpr int LUT_LB = 8;            // blocks of K per CTA (16 bytes of a row of idx)
constexpr int LUT_THREADS = 512;

struct LutParams {
    const void *x;
    const uint16_t *idx;
    const uint32_t *Cp;      // public packed codewords: bit t = (c_t + 1) / 2
    float *part;             // [slices][M][N] partial sums, then [M] sums of x
    int M, N, K, v, Kc, Kb;
    int x_dt;
    int mu, P;               // segment length and segments per block
    int rows_per_cta, slices;
};

__global__ void __launch_bounds__(LUT_THREADS, 1)
lut_gemv_kernel(const LutParams p)
{
    extern __shared__ __align__(16) unsigned char lut_smem[];
    const int tid = threadIdx.x;
    const int slice = blockIdx.x, j0 = slice * LUT_LB;
    const int nb = min(LUT_LB, p.Kb - j0);                       // blocks of this slice
    const int r0 = blockIdx.y * p.rows_per_cta, r1 = min(p.N, r0 + p.rows_per_cta);
    const int nseg = 1 << p.mu;
    float *s_lut = reinterpret_cast<float *>(lut_smem);          // [LB][P][2^mu]
    float *s_x = s_lut + (size_t)LUT_LB * p.P * nseg;            // [LB][v] activations of the slice
    __half *s_cb = reinterpret_cast<__half *>(s_x + LUT_LB * 32);   // [LB][Kc]
    const uint32_t kmask = (uint32_t)nseg - 1u;

    for (int m = 0; m < p.M; ++m) {
        // ---- Stage I: signed sums of every segment for every sign pattern (the slice's activations first go to shared
        //      memory; entry s is built from entry s with its lowest set bit cleared: one add per entry)
        for (int e = tid; e < nb * p.v; e += LUT_THREADS) s_x[e] = load_as_float(p.x, p.x_dt, (size_t)m * p.K + (size_t)j0 * p.v + e);
        __syncthreads();
        for (int jp = tid; jp < nb * p.P; jp += LUT_THREADS) {
            const float *xs = s_x + (size_t)jp * p.mu;               // (block j, segment seg) = jp: mu consecutive activations
            float *lut = s_lut + ((size_t)jp << p.mu);
            float neg = 0.f;
            for (int t = 0; t < p.mu; ++t) neg -= xs[t];
            lut[0] = neg;                                            // all signs -1
            for (int sp = 1; sp < nseg; ++sp) {
                const int low = __ffs(sp) - 1;                       // lowest set bit: flipping it from -1 to +1 adds 2 x
                lut[sp] = lut[sp & (sp - 1)] + 2.0f * xs[low];
            }
        }
        __syncthreads();
        // ---- Stage II: one entry per (block, codeword), P lookups each, rounded to fp16 as the paper stores it
        for (int k = tid; k < p.Kc; k += LUT_THREADS) {
            const uint32_t w = __ldg(p.Cp + k);
            for (int j = 0; j < nb; ++j) {
                float acc = 0.f;
                for (int seg = 0; seg < p.P; ++seg)
                    acc += s_lut[((j * p.P + seg) << p.mu) + ((w >> (seg * p.mu)) & kmask)];
                s_cb[(size_t)j * p.Kc + k] = __float2half_rn(acc);
            }
        }
        __syncthreads();
        // ---- gather: a thread per row, one lookup and one add per block
        for (int n = r0 + tid; n < r1; n += LUT_THREADS) {
            const uint16_t *row = p.idx + (size_t)n * p.Kb + j0;
            float acc = 0.f;
            if (nb == LUT_LB) {
                const uint4 q = __ldg(reinterpret_cast<const uint4 *>(row));     // K/v is a multiple of 8: 16-byte aligned
                const uint32_t wd[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int j = 0; j < LUT_LB; ++j) {
                    const uint32_t i = (j & 1) ? (wd[j >> 1] >> 16) : (wd[j >> 1] & 0xffffu);
                    acc += __half2float(s_cb[(size_t)j * p.Kc + i]);
                }
            } else {
                for (int j = 0; j < nb; ++j) acc += __half2float(s_cb[(size_t)j * p.Kc + row[j]]);
            }
            p.part[((size_t)slice * p.M + m) * p.N + n] = acc;
        }
        __syncthreads();
    }
}

// Adds the K-slices' partial sums in slice order, applies alpha (and mu * sum_k x, summed by the block in a fixed order).
__global__ void __launch_bounds__(256)
lut_reduce_kernel(const float *__restrict__ part, int slices, int M, int N, int K, const void *x, int x_dt,
                  const __half *__restrict__ alpha, const __half *__restrict__ mu, void *y, int y_dt)
{
    __shared__ float s_red[256];
    const int m = blockIdx.y;
    float sx = 0.f;
    if (mu) {
        float a = 0.f;
        for (int k = threadIdx.x; k < K; k += 256) a += load_as_float(x, x_dt, (size_t)m * K + k);
        s_red[threadIdx.x] = a;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if ((int)threadIdx.x < o) s_red[threadIdx.x] += s_red[threadIdx.x + o];
            __syncthreads();
        }
        sx = s_red[0];
    }
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= N) return;
    float acc = 0.f;
    for (int s = 0; s < slices; ++s) acc += part[((size_t)s * M + m) * N + n];
    float yv = __half2float(alpha[n]) * acc;
    if (mu) yv += __half2float(mu[n]) * sx;
    store_from_float(y, y_dt, (size_t)m * N + n, yv);
}

size_t gemv_lut_workspace_bytes(int M, int N, int K, int v)
{
    const int Kb = K / v;
    const size_t slices = (size_t)(Kb + LUT_LB - 1) / LUT_LB;
    return slices * (size_t)M * N * sizeof(float);
}

int launch_gemv_lut(const LinearArgs &a, cudaStream_t s)
{
    // covered: v a multiple of 4 up to 32 (segments of 8 when 8 divides v, else 4), K/v a multiple of 8, and a codebook
    // whose LB tables of Kc fp16 entries fit shared memory beside the activation tables
    if (a.M < 1 || a.M > 8 || a.v % 4 != 0 || a.Kb % 8 != 0) return BTC_ERR_UNSUPPORTED;
    LutParams p;
    p.mu = (a.v % 8 == 0) ? 8 : 4;
    p.P = a.v / p.mu;
    const size_t smem = ((size_t)LUT_LB * p.P * (1u << p.mu) + LUT_LB * 32) * sizeof(float) + (size_t)LUT_LB * a.Kc * sizeof(__half);
    if (smem > 227u * 1024u) return BTC_ERR_UNSUPPORTED;
    const size_t need = gemv_lut_workspace_bytes(a.M, a.N, a.K, a.v);
    if (!a.workspace || a.workspace_bytes < need) return BTC_ERR_WORKSPACE;
    p.x = a.x; p.idx = a.idx; p.Cp = a.Cp; p.part = reinterpret_cast<float *>(a.workspace);
    p.M = a.M; p.N = a.N; p.K = a.K; p.v = a.v; p.Kc = a.Kc; p.Kb = a.Kb; p.x_dt = a.x_dt;
    p.slices = (a.Kb + LUT_LB - 1) / LUT_LB;
    // row chunks: enough CTAs to fill the SMs once, no more (every CTA of a K-slice rebuilds that slice's tables)
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int chunks = (sms + p.slices - 1) / p.slices;
    if (chunks < 1) chunks = 1;
    p.rows_per_cta = (a.N + chunks - 1) / chunks;
    chunks = (a.N + p.rows_per_cta - 1) / p.rows_per_cta;
    cudaError_t e = cudaFuncSetAttribute(lut_gemv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    lut_gemv_kernel<<<dim3((unsigned)p.slices, (unsigned)chunks), LUT_THREADS, smem, s>>>(p);
    int rc = cuda_check_launch();
    if (rc != BTC_OK) return rc;
    lut_reduce_kernel<<<dim3((unsigned)((a.N + 255) / 256), (unsigned)a.M), 256, 0, s>>>(p.part, p.slices, a.M, a.N, a.K, a.x, a.x_dt,
                                                                                      a.alpha, a.mu, a.y, a.y_dt);
    return cuda_check_launch();
}

}  // namespace btc

using namespace btc;

extern "C" size_t btc_linear_gemv_lut_workspace_bytes(int M, int N, int K, int v, int Kc)
{
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || M < 1 || N < 1 || K < 1 || K % v) return 0;
    return (gemv_lut_workspace_bytes(M, N, K, v) + 255) / 256 * 256;
}

extern "C" int btc_linear_gemv_lut(const void *x, int x_dtype, const uint16_t *idx, const uint32_t *C_packed, const void *alpha,
                                   const void *mu, void *y, int y_dtype, int M, int N, int K, int v, int Kc, void *workspace,
                                   size_t workspace_bytes, void *stream)
{
    if (!x || !idx || !C_packed || !alpha || !y) return BTC_ERR_NULL;
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || M < 1 || M > 8 || N < 1 || K < 1 || K % v) return BTC_ERR_SHAPE;
    if (x_dtype != BTC_F16 && x_dtype != BTC_BF16) return BTC_ERR_UNSUPPORTED;
    if (y_dtype != BTC_F32 && y_dtype != BTC_F16 && y_dtype != BTC_BF16) return BTC_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(idx) % 16 || reinterpret_cast<uintptr_t>(workspace) % 16) return BTC_ERR_ALIGN;
    LinearArgs a;
    a.x = x; a.idx = idx; a.Cp = C_packed;
    a.alpha = reinterpret_cast<const __half *>(alpha);
    a.mu = reinterpret_cast<const __half *>(mu);
    a.y = y; a.workspace = workspace; a.workspace_bytes = workspace_bytes;
    a.x_dt = x_dtype; a.y_dt = y_dtype;
    a.M = M; a.N = N; a.K = K; a.v = v; a.Kc = Kc; a.Kb = K / v;
    return launch_gemv_lut(a, (cudaStream_t)stream);
}
