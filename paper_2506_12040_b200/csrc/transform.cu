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
    // the factors are parameters of the layer, complete before the call was enqueued: they were staged while the kernel
    // before this one may still be running; x is read only once that kernel has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
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

// ---- many rows of x (the tensor-core path's prologue): the two products on the warp-level tensor cores ----------------
// For M >= 64 the two products are dense contractions: (M k1) x k2 x k2 and, per row, k1 x k1 x k2 -- 1.2 G multiply-adds
// for 512 rows of K = 11008 = 86 x 128.  Here a CTA keeps both factors in shared memory as tf32 and takes whole rows of
// x: Y = (X o sigma) P2 and X' = P1^T Y as mma.sync.m16n8k8 (tf32 operands, fp32 accumulation).  16-bit activations are
// exact in tf32; the factors and Y carry a 2^-11 rounding, below the 2^-9 of the 16-bit result this path writes.
// Shared-memory pitches are 4 or 8 words past a multiple of 32, so the fragment reads of a warp fall on 32 banks.
constexpr int TM_THREADS = 256;
constexpr int TM_WARPS = TM_THREADS / 32;

__device__ __forceinline__ uint32_t tm_tf32(float f) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(f));
    return r;
}
__device__ __forceinline__ void tm_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct TmLayout { int k1m, k1k, xp, yp, p1p, p2p; size_t x_off, y_off, p1_off, p2_off, words; };
__host__ __device__ inline TmLayout tm_layout(int k1, int k2)
{
    TmLayout L;
    L.k1m = (k1 + 15) / 16 * 16;            // k1 as an M dimension (16-row tiles)
    L.k1k = (k1 + 7) / 8 * 8;               // k1 as a K dimension (8-wide steps)
    L.xp = k2 + 4;                          // X [k1m][xp]: A operand of the first product (rows a, columns b)
    L.yp = k2 + 8;                          // Y [k1k][yp]: B operand of the second (rows a, columns d)
    L.p1p = L.k1m + 8;                      // P1 [k1k][p1p]: A operand of the second, read transposed (rows a, columns c)
    L.p2p = k2 + 8;                         // P2 [k2][p2p]: B operand of the first (rows b, columns d)
    L.x_off = 0;
    L.y_off = L.x_off + (size_t)L.k1m * L.xp;
    L.p1_off = L.y_off + (size_t)L.k1k * L.yp;
    L.p2_off = L.p1_off + (size_t)L.k1k * L.p1p;
    L.words = L.p2_off + (size_t)k2 * L.p2p;
    return L;
}

// MT: 16-row tiles of k1.  TK1 / TK2: the factor sizes as compile-time constants (0: taken from the arguments), so
// that the pitches and loop bounds of the common shapes fold into immediates.
template <int MT, int TK1, int TK2>
__global__ void __launch_bounds__(TM_THREADS, 1)
transform_mma_kernel(const void *__restrict__ x, int x_dt, const uint32_t *__restrict__ sigma_bits, const float *__restrict__ P1,
                     const float *__restrict__ P2, int k1_arg, int k2_arg, void *__restrict__ xt, int out_dt, int M)
{
    extern __shared__ __align__(16) uint32_t tm_smem[];
    const int k1 = TK1 ? TK1 : k1_arg, k2 = TK2 ? TK2 : k2_arg;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const TmLayout L = tm_layout(k1, k2);
    uint32_t *Xs = tm_smem + L.x_off, *Ys = tm_smem + L.y_off, *P1s = tm_smem + L.p1_off, *P2s = tm_smem + L.p2_off;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int K = k1 * k2;
    // the factors, once per CTA, zero-padded to whole tiles; so are the pad rows of X and Y.  Loads go out in batches
    // of eight or sixteen before any of them is used (a loop of load-convert-store would wait for each trip to L2 in turn)
    {
        const int n1 = L.k1k * L.p1p, n2 = k2 * L.p2p;
        for (int i0 = tid; i0 < n1; i0 += 16 * TM_THREADS) {
            float f[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int i = i0 + u * TM_THREADS, a = i / L.p1p, c = i - a * L.p1p;
                f[u] = (i < n1 && a < k1 && c < k1) ? __ldg(P1 + (size_t)a * k1 + c) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int i = i0 + u * TM_THREADS;
                if (i < n1) P1s[i] = tm_tf32(f[u]);
            }
        }
        if ((reinterpret_cast<uintptr_t>(P2) & 15u) == 0) {
            // rows of P2 are k2 floats, k2 a multiple of 16: four per load, eight loads in flight
            const int q2 = k2 / 4, nq = k2 * q2;
            for (int i0 = tid; i0 < nq; i0 += 8 * TM_THREADS) {
                float4 f[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = i0 + u * TM_THREADS;
                    f[u] = i < nq ? __ldg(reinterpret_cast<const float4 *>(P2) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = i0 + u * TM_THREADS;
                    if (i < nq) {
                        const int b = i / q2, d = 4 * (i - b * q2);
                        *reinterpret_cast<uint4 *>(P2s + (size_t)b * L.p2p + d) = make_uint4(tm_tf32(f[u].x), tm_tf32(f[u].y), tm_tf32(f[u].z), tm_tf32(f[u].w));
                    }
                }
            }
            for (int i = tid; i < k2 * 8; i += TM_THREADS) P2s[(size_t)(i >> 3) * L.p2p + k2 + (i & 7)] = 0u;   // pad columns
        } else {
            for (int i0 = tid; i0 < n2; i0 += 8 * TM_THREADS) {
                float f[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = i0 + u * TM_THREADS, b = i / L.p2p, d = i - b * L.p2p;
                    f[u] = (i < n2 && d < k2) ? __ldg(P2 + (size_t)b * k2 + d) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = i0 + u * TM_THREADS;
                    if (i < n2) P2s[i] = tm_tf32(f[u]);
                }
            }
        }
    }
    for (int i = tid; i < L.k1m * L.xp; i += TM_THREADS) Xs[i] = 0u;
    for (int i = tid; i < L.k1k * L.yp; i += TM_THREADS) Ys[i] = 0u;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int npairs = k2 / 16;             // pairs of 8-column tiles of d
    constexpr int MG = (MT + 1) / 2;        // a warp's work item: half of the a (or c) tiles x one pair of d tiles
    // a row of x: eight 16-bit activations per load (k2 is a multiple of 16: they share a row a of X); the loads of the
    // next row are in flight while this row's products run
    constexpr int NQ = 8;                   // loads per thread: K <= 8 * NQ * TM_THREADS
    const int nvec = K / 8;
    uint4 q[NQ];
    auto load_row = [&](int m) {
        const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(x) + (size_t)m * K);
#pragma unroll
        for (int u = 0; u < NQ; ++u) {
            const int i = tid + u * TM_THREADS;
            q[u] = i < nvec ? __ldg(src + i) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    if ((int)blockIdx.x < M) load_row(blockIdx.x);
    for (int m = blockIdx.x; m < M; m += gridDim.x) {
        const size_t row = (size_t)m * K;
        __syncthreads();                    // (the previous row's X and Y are no longer read; pads and factors are in place)
#pragma unroll
        for (int u = 0; u < NQ; ++u) {
            const int i = tid + u * TM_THREADS;
            if (i < nvec) {
                const int k = 8 * i, a = k / k2, bcol = k - a * k2;
                const uint32_t sg = __ldg(sigma_bits + (k >> 5)) >> (k & 31);
                const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
                uint32_t o[8];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    float lo, hi;
                    if (x_dt == BTC_F16) { const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[h])); lo = f.x; hi = f.y; }
                    else { lo = __uint_as_float(w[h] << 16); hi = __uint_as_float(w[h] & 0xffff0000u); }
                    if ((sg >> (2 * h)) & 1u) lo = -lo;
                    if ((sg >> (2 * h + 1)) & 1u) hi = -hi;
                    o[2 * h] = tm_tf32(lo); o[2 * h + 1] = tm_tf32(hi);
                }
                uint4 *dst = reinterpret_cast<uint4 *>(Xs + (size_t)a * L.xp + bcol);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
        if (m + (int)gridDim.x < M) load_row(m + gridDim.x);
        __syncthreads();
        // ---- Y[a][d] = sum_b X[a][b] P2[b][d]
        for (int item = warp; item < 2 * npairs; item += TM_WARPS) {
            const int pr = item >> 1, mt0 = (item & 1) * MG;
            float acc[MG][2][4];
#pragma unroll
            for (int mt = 0; mt < MG; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[mt][h][i] = 0.f;
            const int d0 = pr * 16;
            for (int kk = 0; kk < k2; kk += 8) {
                uint32_t b0[2], b1[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    b0[h] = P2s[(size_t)(kk + t) * L.p2p + d0 + 8 * h + g];
                    b1[h] = P2s[(size_t)(kk + t + 4) * L.p2p + d0 + 8 * h + g];
                }
#pragma unroll
                for (int mt = 0; mt < MG; ++mt) {
                    if (mt0 + mt < MT) {
                        const uint32_t *xa = Xs + (size_t)((mt0 + mt) * 16 + g) * L.xp + kk + t;
                        const uint32_t a0 = xa[0], a1 = xa[8 * L.xp], a2 = xa[4], a3 = xa[8 * L.xp + 4];
#pragma unroll
                        for (int h = 0; h < 2; ++h) tm_mma(acc[mt][h], a0, a1, a2, a3, b0[h], b1[h]);
                    }
                }
            }
#pragma unroll
            for (int mt = 0; mt < MG; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int a = (mt0 + mt) * 16 + g, d = d0 + 8 * h + 2 * t;
                    if (a < L.k1k) *reinterpret_cast<uint2 *>(Ys + (size_t)a * L.yp + d) = make_uint2(tm_tf32(acc[mt][h][0]), tm_tf32(acc[mt][h][1]));
                    if (a + 8 < L.k1k) *reinterpret_cast<uint2 *>(Ys + (size_t)(a + 8) * L.yp + d) = make_uint2(tm_tf32(acc[mt][h][2]), tm_tf32(acc[mt][h][3]));
                }
        }
        __syncthreads();
        // ---- X'[c][d] = sum_a P1[a][c] Y[a][d]
        for (int item = warp; item < 2 * npairs; item += TM_WARPS) {
            const int pr = item >> 1, mt0 = (item & 1) * MG;
            float acc[MG][2][4];
#pragma unroll
            for (int mt = 0; mt < MG; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[mt][h][i] = 0.f;
            const int d0 = pr * 16;
            for (int kk = 0; kk < L.k1k; kk += 8) {
                uint32_t b0[2], b1[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    b0[h] = Ys[(size_t)(kk + t) * L.yp + d0 + 8 * h + g];
                    b1[h] = Ys[(size_t)(kk + t + 4) * L.yp + d0 + 8 * h + g];
                }
#pragma unroll
                for (int mt = 0; mt < MG; ++mt) {
                    if (mt0 + mt < MT) {
                        // A[c][a] = P1[a][c]: element (row c = 16 mt + g (+8), column a = kk + t (+4))
                        const uint32_t *pa = P1s + (size_t)(kk + t) * L.p1p + (mt0 + mt) * 16 + g;
                        const uint32_t a0 = pa[0], a1 = pa[8], a2 = pa[4 * L.p1p], a3 = pa[4 * L.p1p + 8];
#pragma unroll
                        for (int h = 0; h < 2; ++h) tm_mma(acc[mt][h], a0, a1, a2, a3, b0[h], b1[h]);
                    }
                }
            }
#pragma unroll
            for (int mt = 0; mt < MG; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int c = (mt0 + mt) * 16 + g, d = d0 + 8 * h + 2 * t;
                    if (c < k1) {
                        store_from_float(xt, out_dt, row + (size_t)c * k2 + d, acc[mt][h][0]);
                        store_from_float(xt, out_dt, row + (size_t)c * k2 + d + 1, acc[mt][h][1]);
                    }
                    if (c + 8 < k1) {
                        store_from_float(xt, out_dt, row + (size_t)(c + 8) * k2 + d, acc[mt][h][2]);
                        store_from_float(xt, out_dt, row + (size_t)(c + 8) * k2 + d + 1, acc[mt][h][3]);
                    }
                }
        }
    }
}

template <int MT, int TK1 = 0, int TK2 = 0>
static int launch_transform_mma(const void *x, int x_dt, const btc_transform &T, void *xt, int out_dt, int M, size_t smem, cudaStream_t s)
{
    auto kern = transform_mma_kernel<MT, TK1, TK2>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(M < sms ? M : sms));
    cfg.blockDim = dim3(TM_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, x, x_dt, T.sigma_bits, T.P1, T.P2, T.k1, T.k2, xt, out_dt, M);
    return e == cudaSuccess ? BTC_OK : cuda_fail(e);
}

int launch_transform(const void *x, int x_dt, const btc_transform &T, void *xt, int out_dt, int M, int K, cudaStream_t s)
{
    if ((long long)T.k1 * T.k2 != K) return BTC_ERR_SHAPE;
    // many rows: the tensor-core form, when the factors fit shared memory beside one row (k2 a multiple of 16)
    if (M >= 64 && x_dt != BTC_F32 && T.k2 % 16 == 0 && T.k1 <= 128 && K <= 8 * 8 * TM_THREADS) {
        const size_t bytes = tm_layout(T.k1, T.k2).words * sizeof(uint32_t);
        if (bytes <= 227u * 1024u) {
            const int mt = (T.k1 + 15) / 16;
            // the factor shapes of the LLaMA-2-7B widths (4096 = 64 x 64, 11008 = 86 x 128) have instantiations of their own
            if (T.k1 == 64 && T.k2 == 64) return launch_transform_mma<4, 64, 64>(x, x_dt, T, xt, out_dt, M, bytes, s);
            if (T.k1 == 86 && T.k2 == 128) return launch_transform_mma<6, 86, 128>(x, x_dt, T, xt, out_dt, M, bytes, s);
            switch (mt) {
            case 1: return launch_transform_mma<1>(x, x_dt, T, xt, out_dt, M, bytes, s);
            case 2: return launch_transform_mma<2>(x, x_dt, T, xt, out_dt, M, bytes, s);
            case 3: return launch_transform_mma<3>(x, x_dt, T, xt, out_dt, M, bytes, s);
            case 4: return launch_transform_mma<4>(x, x_dt, T, xt, out_dt, M, bytes, s);
            case 5: return launch_transform_mma<5>(x, x_dt, T, xt, out_dt, M, bytes, s);
            case 6: return launch_transform_mma<6>(x, x_dt, T, xt, out_dt, M, bytes, s);
            case 7: return launch_transform_mma<7>(x, x_dt, T, xt, out_dt, M, bytes, s);
            default: return launch_transform_mma<8>(x, x_dt, T, xt, out_dt, M, bytes, s);
            }
        }
    }
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
    // programmatic launch: the kernel may start (and stage the factors) before its predecessor on the stream has finished
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)tiles, (unsigned)groups);
    cfg.blockDim = dim3(TR_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, transform_kernel, x, x_dt, T.sigma_bits, T.P1, T.P2, T.k1, T.k2, xt, out_dt, M, rows);
    return e == cudaSuccess ? BTC_OK : cuda_fail(e);
}

}  // namespace btc
