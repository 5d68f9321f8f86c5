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

// TMU / TP: segment length and segments per block as compile-time constants (0: taken from the parameters), so that
// the table-build loops unroll with immediate offsets.
template <int TMU, int TP>
__global__ void __launch_bounds__(LUT_THREADS, 1)
lut_gemv_kernel(const LutParams p)
{
    const int mu = TMU ? TMU : p.mu, P = TP ? TP : p.P;
    extern __shared__ __align__(16) unsigned char lut_smem[];
    const int tid = threadIdx.x;
    const int slice = blockIdx.x, j0 = slice * LUT_LB;
    const int nb = min(LUT_LB, p.Kb - j0);                       // blocks of this slice
    const int r0 = blockIdx.y * p.rows_per_cta, r1 = min(p.N, r0 + p.rows_per_cta);
    const int nseg = 1 << mu;
    float *s_lut = reinterpret_cast<float *>(lut_smem);          // [LB][P][2^mu]
    float *s_x = s_lut + (size_t)LUT_LB * P * nseg;            // [LB][v] activations of the slice
    __half *s_cb = reinterpret_cast<__half *>(s_x + LUT_LB * 32);   // [LB][Kc]
    const uint32_t kmask = (uint32_t)nseg - 1u;

    for (int m = 0; m < p.M; ++m) {
        // ---- Stage I: signed sums of every segment for every sign pattern (the slice's activations first go to shared
        //      memory; one thread per table entry)
        for (int e = tid; e < nb * p.v; e += LUT_THREADS) s_x[e] = load_as_float(p.x, p.x_dt, (size_t)m * p.K + (size_t)j0 * p.v + e);
        __syncthreads();
        for (int e = tid; e < (nb * P) << mu; e += LUT_THREADS) {
            // entry sp of the table of (block j, segment seg) = jp: the signed sum of its mu activations (bit t of sp set <=> +)
            const int jp = e >> mu, sp = e & (nseg - 1);
            const float *xs = s_x + (size_t)jp * mu;
            float acc = 0.f;
            for (int t = 0; t < mu; ++t) acc += ((sp >> t) & 1) ? xs[t] : -xs[t];
            s_lut[e] = acc;
        }
        __syncthreads();
        // ---- Stage II: one entry per (block, codeword), P lookups each, rounded to fp16 as the paper stores it.  The
        //      codeword words go out eight loads at a time before any is used.
        for (int k0 = tid; k0 < p.Kc; k0 += 8 * LUT_THREADS) {
            uint32_t wv[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int k = k0 + u * LUT_THREADS;
                wv[u] = k < p.Kc ? __ldg(p.Cp + k) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int k = k0 + u * LUT_THREADS;
                if (k < p.Kc) {
                    if (TMU && nb == LUT_LB) {
#pragma unroll
                        for (int j = 0; j < LUT_LB; ++j) {
                            float acc = 0.f;
#pragma unroll
                            for (int seg = 0; seg < (TP ? TP : 1); ++seg)
                                acc += s_lut[((j * P + seg) << mu) + ((wv[u] >> (seg * mu)) & kmask)];
                            s_cb[(size_t)j * p.Kc + k] = __float2half_rn(acc);
                        }
                    } else {
                        for (int j = 0; j < nb; ++j) {
                            float acc = 0.f;
                            for (int seg = 0; seg < P; ++seg)
                                acc += s_lut[((j * P + seg) << mu) + ((wv[u] >> (seg * mu)) & kmask)];
                            s_cb[(size_t)j * p.Kc + k] = __float2half_rn(acc);
                        }
                    }
                }
            }
        }
        __syncthreads();
        // ---- gather: a thread per row, one lookup and one add per block
        if (nb == LUT_LB) {
            // whole slices: 16 bytes of indices per row (K/v is a multiple of 8: aligned), four rows' loads in flight
            for (int n0 = r0 + tid; n0 < r1; n0 += 4 * LUT_THREADS) {
                uint4 q[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int n = n0 + u * LUT_THREADS;
                    q[u] = n < r1 ? __ldg(reinterpret_cast<const uint4 *>(p.idx + (size_t)n * p.Kb + j0)) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int n = n0 + u * LUT_THREADS;
                    if (n < r1) {
                        const uint32_t wd[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
                        float acc = 0.f;
#pragma unroll
                        for (int j = 0; j < LUT_LB; ++j) {
                            const uint32_t i = (j & 1) ? (wd[j >> 1] >> 16) : (wd[j >> 1] & 0xffffu);
                            acc += __half2float(s_cb[(size_t)j * p.Kc + i]);
                        }
                        p.part[((size_t)slice * p.M + m) * p.N + n] = acc;
                    }
                }
            }
        } else {
            for (int n = r0 + tid; n < r1; n += LUT_THREADS) {
                const uint16_t *row = p.idx + (size_t)n * p.Kb + j0;
                float acc = 0.f;
                for (int j = 0; j < nb; ++j) acc += __half2float(s_cb[(size_t)j * p.Kc + row[j]]);
                p.part[((size_t)slice * p.M + m) * p.N + n] = acc;
            }
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
    // row chunks: as many CTAs as fit the SMs in one round, no more (every CTA of a K-slice rebuilds that slice's tables)
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int chunks = sms / p.slices;                 // (rounded down: a second round of CTAs would cost a whole table build)
    if (chunks < 1) chunks = 1;
    p.rows_per_cta = (a.N + chunks - 1) / chunks;
    chunks = (a.N + p.rows_per_cta - 1) / p.rows_per_cta;
    void (*kern)(const LutParams) = lut_gemv_kernel<0, 0>;
    if (p.mu == 8 && p.P == 2) kern = lut_gemv_kernel<8, 2>;          // v = 16
    else if (p.mu == 8 && p.P == 1) kern = lut_gemv_kernel<8, 1>;     // v = 8
    else if (p.mu == 4 && p.P == 5) kern = lut_gemv_kernel<4, 5>;     // v = 20
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    kern<<<dim3((unsigned)p.slices, (unsigned)chunks), LUT_THREADS, smem, s>>>(p);
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
