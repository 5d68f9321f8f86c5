// Decode path for small M (1..8): streams the index matrices of up to IM_MAXP independent layers
// once and evaluates every block dot
//     <x_j, C[idx]> = 2 * sum_{bit=1} x  -  sum x            (identity for +-1 codewords)
// (block-dot sum of the paper's appendix "Binary codebook LUT-GEMM") with EXACT integer accumulation.
//
// Why integers.  One output needs K sign applications.  At the HBM rate an SM receives 180 weights per
// clock (v = 16), while its plain ALUs issue 64 integer lane-operations per clock and the warp-level
// fp16 MMA retires one m16n8k16 per 2.2 clocks; measured, the fp16 bit trick tops out at 76 weights
// per clock per SM, the int8 form below at 121.  So the sum over set bits is taken by
// mma.sync.m16n8k32 (u8 x s8 -> s32):
//   A (16 rows x 32 k, u8) = masked codeword bits: the codeword table stores weight t at bit (t >> 2)
//       of byte (t & 3), so `word & (0x01010101 << c)` IS the four bytes {0 or 2^c} of weights
//       4c .. 4c+3: one LOP3 expands four weights.
//   B (32 k x 8 cols, s8)  = the activations as balanced base-256 digits of a block-fixed-point
//       integer: X = rint(x * 2^s) with s chosen per row of x from its largest magnitude, pre-shifted
//       by (cmax - c) so that every product is bit * X * 2^cmax; digit d of row m sits in column
//       m * D + d.
//   D (16 x 8, s32)        = exact partial sums; the digits are recombined once per output.
// The result is the exact +-1 dot product of the quantised activations; the only roundings are the
// quantisation of x (relative to the row maximum: 2^-20 for v = 16 with three digits, 2^-28 with
// four) and one rounding per output when alpha is applied.
//
// Work split: persistent CTAs.  The unit of work is an "iteration": up to two 16-row tiles over the
// full K of one layer.  A CTA owns a contiguous range of iterations of the launch (over all layers).
//   warps 0..15  compute: each owns a K-slice; lane (g = lane / 4, t = lane % 4) supplies rows g and
//                g + 8 of the tile and the blocks 16 q + 4 t + e of its slice; its activations stay
//                in registers as MMA B fragments.
//   warp 16      producer: cp.async.bulk of index tiles (contiguous in memory) into a shared ring,
//                and of the codeword table.
//   warp 17      epilogue: adds the 16 partial tiles in a fixed order, recombines digits, applies
//                alpha (and mu), stores y.
// Every mbarrier wait is bounded; when one runs out the CTA raises a status word and drains.
#include "btc_internal.cuh"

namespace btc {

constexpr int IM_CWARPS = 16;
constexpr int IM_THREADS = (IM_CWARPS + 2) * 32;
constexpr int IM_STAGES = 4;
constexpr int IM_STAGE_BYTES = 24 * 1024;       // one iteration's indices (<= 2 tiles)
constexpr int IM_TR = 2;                        // max 16-row tiles per iteration

__device__ int g_imma_status = 0;

struct ImProblem {
    const void *x;
    const uint16_t *idx;
    const uint32_t *tab;      // byte-lane codeword words [Kc]
    const __half *alpha;
    const __half *mu;         // may be nullptr
    void *y;
    int M, N, K, v, Kc, Kb;
    int x_dt, y_dt;
    int nq;                   // 8-byte index chunks per lane per row: ceil(Kb / 256)
    int tr;                   // tiles per iteration (1 or 2)
    int tiles;                // ceil(N / 16)
    int iter_begin;           // first iteration of this layer in the launch's numbering
    int iters;                // ceil(tiles / tr)
    int ncls;                 // ceil(v / 4)
};

struct ImBatch {
    ImProblem p[IM_MAXP];
    int count;
    int total_iters;
    int tab_smem_bytes;       // bytes reserved for the codeword table (0: gather from global memory)
};

// ------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t im_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void im_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void im_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void im_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool im_mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false (and the CTA-wide abort flag latched) once ~1 s has passed.
__device__ __forceinline__ bool im_mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (im_mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (!im_mbar_try(bar, parity)) {
        if ((++spins & 255) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > 2000000000LL) {
                *abort_flag = 1;
                atomicExch(&g_imma_status, (int)BTC_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void im_bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void im_mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void im_named_bar(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Shared-memory layout (dynamic), offsets computed identically on host and device.
struct ImSmem {
    uint32_t bars;        // mbarriers: full[S], empty[S], part_full[2], part_empty[2], tab_full, tab_free
    uint32_t misc;        // abort flag, per-segment scale slots, reduction scratch
    uint32_t tab;         // codeword table
    uint32_t ring;        // index stages
    uint32_t part;        // partial sums [2][16 warps][part_ints]
    uint32_t total;
};
constexpr int IM_NBARS = 2 * IM_STAGES + 6;
constexpr int IM_SLOTS = 3;                      // per-segment scale slots
constexpr int IM_MISC_BYTES = 16 + IM_SLOTS * 16 * 8 + IM_CWARPS * 8 * 4 + IM_CWARPS * 8 * 8;

__host__ __device__ inline ImSmem im_smem_layout(int tab_bytes, int part_ints)
{
    ImSmem L;
    uint32_t o = 0;
    L.bars = o; o += IM_NBARS * 8;
    o = (o + 15u) & ~15u;
    L.misc = o; o += IM_MISC_BYTES;
    o = (o + 127u) & ~127u;
    L.tab = o; o += (uint32_t)tab_bytes;
    o = (o + 127u) & ~127u;
    L.ring = o; o += IM_STAGES * IM_STAGE_BYTES;
    L.part = o; o += 2u * IM_CWARPS * (uint32_t)part_ints * 4u;
    L.total = o;
    return L;
}

// Two packed fp16 (dt = BTC_F16) or bf16 numbers -> two floats.
__device__ __forceinline__ void im_unpack2(uint32_t w, int dt, float &lo, float &hi)
{
    if (dt == BTC_F16) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w));
        lo = f.x; hi = f.y;
    } else {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xffff0000u);
    }
}

template <int NCLS, int NQ, int NM>
__global__ void __launch_bounds__(IM_THREADS, 1)
gemv_imma_kernel(const __grid_constant__ ImBatch batch)
{
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int TRK = (NM == 1) ? IM_TR : 1;           // tiles per iteration this instantiation supports
    constexpr int PART_INTS = TRK * 16 * 8 * NM;
    const ImSmem L = im_smem_layout(batch.tab_smem_bytes, PART_INTS);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + L.misc);
    double *s_slot = reinterpret_cast<double *>(smem + L.misc + 16);              // [IM_SLOTS][16]: inv_scale[8], sumX[8]
    float *s_redf = reinterpret_cast<float *>(smem + L.misc + 16 + IM_SLOTS * 128);   // [16][8]
    double *s_redd = reinterpret_cast<double *>(smem + L.misc + 16 + IM_SLOTS * 128 + IM_CWARPS * 32);   // [16][8]
    uint32_t *s_tab = reinterpret_cast<uint32_t *>(smem + L.tab);
    unsigned char *s_ring = smem + L.ring;
    int *s_part = reinterpret_cast<int *>(smem + L.part);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto bar_full = [&](int s) { return im_smem_u32(bars + s); };
    auto bar_empty = [&](int s) { return im_smem_u32(bars + IM_STAGES + s); };
    auto bar_pfull = [&](int b) { return im_smem_u32(bars + 2 * IM_STAGES + b); };
    auto bar_pempty = [&](int b) { return im_smem_u32(bars + 2 * IM_STAGES + 2 + b); };
    const uint32_t bar_tabfull = im_smem_u32(bars + 2 * IM_STAGES + 4);
    const uint32_t bar_tabfree = im_smem_u32(bars + 2 * IM_STAGES + 5);

    if (tid == 0) {
        for (int s = 0; s < IM_STAGES; ++s) { im_mbar_init(bar_full(s), 1); im_mbar_init(bar_empty(s), IM_CWARPS); }
        for (int b = 0; b < 2; ++b) { im_mbar_init(bar_pfull(b), IM_CWARPS); im_mbar_init(bar_pempty(b), 1); }
        im_mbar_init(bar_tabfull, 1);
        im_mbar_init(bar_tabfree, IM_CWARPS);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- this CTA's range of iterations, and the layers (segments) it touches
    const int total = batch.total_iters;
    const int per = total / gridDim.x, rem = total % gridDim.x;
    const int it_begin = blockIdx.x * per + min((int)blockIdx.x, rem);
    const int it_end = it_begin + per + ((int)blockIdx.x < rem ? 1 : 0);
    const bool tab_smem = batch.tab_smem_bytes > 0;
    constexpr int D = (NM == 1) ? 4 : 3;                 // digits per activation
    constexpr int MAXM = (NM == 1) ? 2 : (NM == 2 ? 5 : 8);
    auto problem_of = [&](int it) {
        int pi = 0;
        while (pi + 1 < batch.count && it >= batch.p[pi + 1].iter_begin) ++pi;
        return pi;
    };

    if (warp == IM_CWARPS) {
        // ============================================================ producer
        int li = 0, seg = 0;
        for (int it = it_begin; it < it_end; ++seg) {
            const ImProblem &P = batch.p[problem_of(it)];
            const int seg_end = min(it_end, P.iter_begin + P.iters);
            if (tab_smem) {
                if (seg > 0 && !im_mbar_wait(bar_tabfree, (seg - 1) & 1, s_abort)) break;
                if (lane == 0) {
                    const uint32_t bytes = (uint32_t)((P.Kc + 3) / 4 * 16);
                    im_mbar_expect_tx(bar_tabfull, bytes);
                    im_bulk_g2s(im_smem_u32(s_tab), P.tab, bytes, bar_tabfull);
                }
            }
            bool ok = true;
            for (; it < seg_end; ++it, ++li) {
                const int s = li % IM_STAGES;
                if (li >= IM_STAGES && !im_mbar_wait(bar_empty(s), ((li / IM_STAGES) & 1) ^ 1, s_abort)) { ok = false; break; }
                const int tile0 = (it - P.iter_begin) * P.tr;
                const int ntile = min(P.tr, P.tiles - tile0);
                const int row0 = tile0 * 16;
                const int rows = min(ntile * 16, P.N - row0);
                const uint32_t bytes = (uint32_t)rows * (uint32_t)P.Kb * 2u;
                const uint32_t bulk = bytes & ~15u;
                const uint32_t tile_bytes = (uint32_t)ntile * 16u * (uint32_t)P.Kb * 2u;
                unsigned char *stage = s_ring + (size_t)s * IM_STAGE_BYTES;
                const unsigned char *src = reinterpret_cast<const unsigned char *>(P.idx + (size_t)row0 * P.Kb);
                if (bulk != tile_bytes) {
                    // ragged tail: the last bytes by hand, rows past N zero-filled (index 0 is always valid)
                    for (uint32_t o = bulk + 2u * lane; o < tile_bytes; o += 64u)
                        *reinterpret_cast<uint16_t *>(stage + o) =
                            (o < bytes) ? *reinterpret_cast<const uint16_t *>(src + o) : (uint16_t)0;
                    __syncwarp();
                }
                if (lane == 0) {
                    if (bulk) {
                        im_mbar_expect_tx(bar_full(s), bulk);
                        im_bulk_g2s(im_smem_u32(stage), src, bulk, bar_full(s));
                    } else {
                        im_mbar_arrive(bar_full(s));
                    }
                }
            }
            if (!ok) break;
        }
    } else if (warp == IM_CWARPS + 1) {
        // ============================================================ epilogue
        asm volatile("griddepcontrol.wait;" ::: "memory");
        int li = 0, seg = 0;
        for (int it = it_begin; it < it_end; ++seg) {
            const ImProblem &P = batch.p[problem_of(it)];
            const int seg_end = min(it_end, P.iter_begin + P.iters);
            const double *slot = s_slot + (seg % IM_SLOTS) * 16;
            const double unshift = 1.0 / (double)(1 << (P.ncls - 1));
            bool ok = true;
            for (; it < seg_end; ++it, ++li) {
                const int buf = li & 1;
                const int tile0 = (it - P.iter_begin) * P.tr;
                const int ntile = min(P.tr, P.tiles - tile0);
                const int n = tile0 * 16 + lane;
                const bool live = (lane < ntile * 16) && (n < P.N);
                float al = 0.f, mu = 0.f;
                if (live) {
                    al = __half2float(P.alpha[n]);
                    if (P.mu) mu = __half2float(P.mu[n]);
                }
                if (!im_mbar_wait(bar_pfull(buf), (li >> 1) & 1, s_abort)) { ok = false; break; }
                int sum[NM * 8];
#pragma unroll
                for (int c = 0; c < NM * 8; ++c) sum[c] = 0;
                const int *base = s_part + (size_t)buf * IM_CWARPS * PART_INTS + (size_t)lane * NM * 8;
#pragma unroll 4
                for (int w = 0; w < IM_CWARPS; ++w) {
                    if (lane >= TRK * 16) break;                 // a warp's partial tile has TRK * 16 rows
                    const int4 *pw = reinterpret_cast<const int4 *>(base + (size_t)w * PART_INTS);
#pragma unroll
                    for (int c4 = 0; c4 < NM * 2; ++c4) {
                        const int4 v4 = pw[c4];
                        sum[c4 * 4 + 0] += v4.x; sum[c4 * 4 + 1] += v4.y; sum[c4 * 4 + 2] += v4.z; sum[c4 * 4 + 3] += v4.w;
                    }
                }
                double inv[MAXM], sx[MAXM];
#pragma unroll
                for (int m = 0; m < MAXM; ++m) { inv[m] = slot[m < 8 ? m : 0]; sx[m] = slot[8 + (m < 8 ? m : 0)]; }
                __syncwarp();
                if (lane == 0) im_mbar_arrive(bar_pempty(buf));
                if (live) {
#pragma unroll
                    for (int m = 0; m < MAXM; ++m) {
                        if (m < P.M) {
                            double T = 0.0;
#pragma unroll
                            for (int d = D - 1; d >= 0; --d) T = T * 256.0 + (double)sum[m * D + d];
                            const double sumx = sx[m] * inv[m];
                            const double dot = (2.0 * T * unshift - sx[m]) * inv[m];
                            const float yv = (float)((double)al * dot + (double)mu * sumx);
                            store_from_float(P.y, P.y_dt, (size_t)m * P.N + n, yv);
                        }
                    }
                }
            }
            if (!ok) break;
        }
    } else {
        // ============================================================ compute warps
        const int g = lane >> 2, t = lane & 3;
        const int ctid = tid;                                  // 0 .. 511
        constexpr int CT = IM_CWARPS * 32;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        int li = 0, seg = 0;
        for (int it = it_begin; it < it_end; ++seg) {
            const ImProblem &P = batch.p[problem_of(it)];
            const int seg_end = min(it_end, P.iter_begin + P.iters);
            double *slot = s_slot + (seg % IM_SLOTS) * 16;
            const int M = P.M, K = P.K, Kb = P.Kb, v = P.v, nq = P.nq;
            const int cmax = P.ncls - 1;
            const int PBITS = 8 * D - 2 - cmax;                // |X| <= 2^PBITS

            // ---- quantisation of x, step 1: per-row scale from the largest magnitude (16-byte loads)
            {
                const int nvec = K >> 3;                        // K % 16 == 0 (checked on the host)
                for (int m = 0; m < M; ++m) {
                    float a = 0.f;
                    const uint4 *xr = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(P.x) + (size_t)m * K);
                    for (int i = ctid; i < nvec; i += CT) {
                        const uint4 q4 = __ldg(xr + i);
                        const uint32_t wds[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float lo, hi;
                            im_unpack2(wds[j], P.x_dt, lo, hi);
                            a = fmaxf(a, fmaxf(fabsf(lo), fabsf(hi)));
                        }
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
                    if (lane == 0) s_redf[warp * 8 + m] = a;
                }
            }
            im_named_bar(1, CT);
            if (ctid < M) {
                float a = 0.f;
                for (int w = 0; w < IM_CWARPS; ++w) a = fmaxf(a, s_redf[w * 8 + ctid]);
                int e = 0;
                if (a > 0.f) (void)frexpf(a, &e);              // a = f * 2^e, f in [0.5, 1)
                slot[ctid] = (a > 0.f) ? ldexp(1.0, e - PBITS) : 1.0;
            }
            im_named_bar(1, CT);

            // ---- step 2: B fragments of this lane (blocks wbase + 16 q + 4 t + e, classes c, column
            //      g + 8 nm = m * D + d) and the integer row sums, from 8-byte loads of x
            const int wbase = warp * 16 * nq;
            uint32_t breg[NQ][4][NCLS][NM];
            long long xsum[NM];
#pragma unroll
            for (int nm = 0; nm < NM; ++nm) {
                xsum[nm] = 0;
                const int col = g + 8 * nm;
                const int m = col / D, d = col - m * D;
                const bool colvalid = m < M;
                const float sc = colvalid ? (float)(1.0 / slot[colvalid ? m : 0]) : 0.f;
                const uint16_t *xrow = reinterpret_cast<const uint16_t *>(P.x) + (size_t)(colvalid ? m : 0) * K;
                const uint32_t sel = (uint32_t)d | ((uint32_t)(4 + d) << 4);
                const uint32_t flip = (d < D - 1) ? 0x80808080u : 0u;
                constexpr int BIAS = (D == 4) ? 0x00808080 : 0x00008080;
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    uint2 raw[4][NCLS];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int jb = wbase + 16 * q + 4 * t + e;
                        const bool bvalid = colvalid && (q < nq) && (jb < Kb);
#pragma unroll
                        for (int c = 0; c < NCLS; ++c) {
                            raw[e][c] = make_uint2(0u, 0u);
                            if (bvalid && c <= cmax)
                                raw[e][c] = __ldg(reinterpret_cast<const uint2 *>(xrow + (size_t)jb * v + 4 * c));
                        }
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e)
#pragma unroll
                        for (int c = 0; c < NCLS; ++c) {
                            float f0, f1, f2, f3;
                            im_unpack2(raw[e][c].x, P.x_dt, f0, f1);
                            im_unpack2(raw[e][c].y, P.x_dt, f2, f3);
                            const int X0 = __float2int_rn(f0 * sc), X1 = __float2int_rn(f1 * sc);
                            const int X2 = __float2int_rn(f2 * sc), X3 = __float2int_rn(f3 * sc);
                            if (d == 0) xsum[nm] += (long long)(X0 + X1) + (long long)(X2 + X3);
                            const int sh = 1 << ((c <= cmax) ? (cmax - c) : 0);
                            // balanced digit d of Y: byte d of (Y + BIAS), with 0x80 flipped back below the top digit
                            const uint32_t y01 = __byte_perm((uint32_t)(X0 * sh + BIAS), (uint32_t)(X1 * sh + BIAS), sel);
                            const uint32_t y23 = __byte_perm((uint32_t)(X2 * sh + BIAS), (uint32_t)(X3 * sh + BIAS), sel);
                            const bool on = colvalid && (c <= cmax);
                            breg[q][e][c][nm] = on ? (__byte_perm(y01, y23, 0x5410) ^ flip) : 0u;
                        }
                }
            }
            // integer row sums: the four lanes (t) of column m * D hold disjoint blocks of row m
#pragma unroll
            for (int nm = 0; nm < NM; ++nm) {
                const int col = g + 8 * nm;
                const int m = col / D, d = col - m * D;
                long long sacc = xsum[nm];
                sacc += __shfl_xor_sync(0xffffffffu, sacc, 1);
                sacc += __shfl_xor_sync(0xffffffffu, sacc, 2);
                if (t == 0 && d == 0 && m < M) s_redd[warp * 8 + m] = (double)sacc;
            }
            im_named_bar(1, CT);
            if (ctid < M) {
                double sacc = 0.0;
                for (int w = 0; w < IM_CWARPS; ++w) sacc += s_redd[w * 8 + ctid];
                slot[8 + ctid] = sacc;
            }
            // (the epilogue warp reads the slot only after a partial-sum barrier that follows this point)

            if (tab_smem && !im_mbar_wait(bar_tabfull, seg & 1, s_abort)) break;
            const uint32_t *tab = tab_smem ? s_tab : P.tab;

            bool ok = true;
            for (; it < seg_end; ++it, ++li) {
                const int s = li % IM_STAGES;
                const int tile0 = (it - P.iter_begin) * P.tr;
                const int ntile = min(P.tr, P.tiles - tile0);
                if (!im_mbar_wait(bar_full(s), (li / IM_STAGES) & 1, s_abort)) { ok = false; break; }
                const unsigned char *stage = s_ring + (size_t)s * IM_STAGE_BYTES;
                uint2 ia[TRK][NQ], ib[TRK][NQ];
#pragma unroll
                for (int r = 0; r < TRK; ++r) {
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        const int jb0 = wbase + 16 * q + 4 * t;
                        ia[r][q] = make_uint2(0u, 0u);
                        ib[r][q] = make_uint2(0u, 0u);
                        if (r < ntile && q < nq && jb0 < Kb) {
                            ia[r][q] = *reinterpret_cast<const uint2 *>(stage + ((size_t)(r * 16 + g) * Kb + jb0) * 2);
                            ib[r][q] = *reinterpret_cast<const uint2 *>(stage + ((size_t)(r * 16 + g + 8) * Kb + jb0) * 2);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) im_mbar_arrive(bar_empty(s));

                int acc[TRK][NM][4];
#pragma unroll
                for (int r = 0; r < TRK; ++r)
#pragma unroll
                    for (int nm = 0; nm < NM; ++nm)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[r][nm][i] = 0;
#pragma unroll
                for (int r = 0; r < TRK; ++r) {
                    if (r < ntile) {
#pragma unroll
                        for (int q = 0; q < NQ; ++q) {
                            if (q < nq) {
                                uint32_t w0[4], w1[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const uint32_t pa = (e < 2) ? ia[r][q].x : ia[r][q].y;
                                    const uint32_t pb = (e < 2) ? ib[r][q].x : ib[r][q].y;
                                    const uint32_t i0 = (e & 1) ? (pa >> 16) : (pa & 0xffffu);
                                    const uint32_t i1 = (e & 1) ? (pb >> 16) : (pb & 0xffffu);
                                    w0[e] = tab_smem ? tab[i0] : __ldg(tab + i0);
                                    w1[e] = tab_smem ? tab[i1] : __ldg(tab + i1);
                                }
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
#pragma unroll
                                    for (int cp = 0; cp < NCLS / 2; ++cp) {
                                        const uint32_t ma = 0x01010101u << (2 * cp), mb = 0x01010101u << (2 * cp + 1);
#pragma unroll
                                        for (int nm = 0; nm < NM; ++nm)
                                            im_mma_u8s8(acc[r][nm], w0[e] & ma, w1[e] & ma, w0[e] & mb, w1[e] & mb,
                                                        breg[q][e][2 * cp][nm], breg[q][e][2 * cp + 1][nm]);
                                    }
                                }
                                if (NCLS & 1) {
                                    const uint32_t ml = 0x01010101u << (NCLS - 1);
#pragma unroll
                                    for (int ep = 0; ep < 2; ++ep)
#pragma unroll
                                        for (int nm = 0; nm < NM; ++nm)
                                            im_mma_u8s8(acc[r][nm], w0[2 * ep] & ml, w1[2 * ep] & ml, w0[2 * ep + 1] & ml,
                                                        w1[2 * ep + 1] & ml, breg[q][2 * ep][NCLS - 1][nm],
                                                        breg[q][2 * ep + 1][NCLS - 1][nm]);
                                }
                            }
                        }
                    }
                }
                const int buf = li & 1;
                if (li >= 2 && !im_mbar_wait(bar_pempty(buf), ((li >> 1) & 1) ^ 1, s_abort)) { ok = false; break; }
                int *mine = s_part + ((size_t)buf * IM_CWARPS + warp) * PART_INTS;
#pragma unroll
                for (int r = 0; r < TRK; ++r)
#pragma unroll
                    for (int nm = 0; nm < NM; ++nm) {
                        *reinterpret_cast<int2 *>(mine + ((r * 16 + g) * NM + nm) * 8 + 2 * t) = make_int2(acc[r][nm][0], acc[r][nm][1]);
                        *reinterpret_cast<int2 *>(mine + ((r * 16 + g + 8) * NM + nm) * 8 + 2 * t) = make_int2(acc[r][nm][2], acc[r][nm][3]);
                    }
                __syncwarp();
                if (lane == 0) im_mbar_arrive(bar_pfull(buf));
            }
            if (!ok) break;
            if (tab_smem) {
                __syncwarp();
                if (lane == 0) im_mbar_arrive(bar_tabfree);
            }
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------ host side
static int im_sm_count()
{
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

template <int NCLS, int NQ, int NM>
static int im_launch(const ImBatch &b, cudaStream_t s)
{
    constexpr int TRK = (NM == 1) ? IM_TR : 1;
    const ImSmem L = im_smem_layout(b.tab_smem_bytes, TRK * 16 * 8 * NM);
    auto kern = gemv_imma_kernel<NCLS, NQ, NM>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total);
    if (e != cudaSuccess) return cuda_fail(e);
    cudaLaunchConfig_t cfg = {};
    const int sms = im_sm_count();
    cfg.gridDim = dim3((unsigned)(b.total_iters < sms ? b.total_iters : sms));
    cfg.blockDim = dim3(IM_THREADS);
    cfg.dynamicSmemBytes = L.total;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, b);
    return e == cudaSuccess ? BTC_OK : cuda_fail(e);
}

template <int NCLS, int NQ>
static int im_launch_nm(const ImBatch &b, int nm, cudaStream_t s)
{
    if (nm == 1) return im_launch<NCLS, NQ, 1>(b, s);
    if (NQ == 1) {
        if (nm == 2) return im_launch<NCLS, 1, 2>(b, s);
        return im_launch<NCLS, 1, 3>(b, s);
    }
    return BTC_ERR_UNSUPPORTED;
}

template <int NCLS>
static int im_launch_nq(const ImBatch &b, int nq, int nm, cudaStream_t s)
{
    if (nq == 1) return im_launch_nm<NCLS, 1>(b, nm, s);
    if (nm != 1) return BTC_ERR_UNSUPPORTED;
    if (nq == 2) return im_launch_nm<NCLS, 2>(b, nm, s);
    if (nq == 3) return im_launch_nm<NCLS, 3>(b, nm, s);
    return BTC_ERR_UNSUPPORTED;
}

int launch_gemv_imma(const LinearArgs *problems, int count, cudaStream_t s)
{
    if (count < 1 || count > IM_MAXP) return BTC_ERR_UNSUPPORTED;
    ImBatch b = {};
    b.count = count;
    int ncls_max = 0, nq_max = 0, m_max = 0, tab_max = 0, it = 0;
    for (int i = 0; i < count; ++i) {
        const LinearArgs &a = problems[i];
        ImProblem &p = b.p[i];
        if (a.M < 1 || a.M > 8 || a.Kb % 4 != 0 || a.v % 4 != 0 || a.v > 20) return BTC_ERR_UNSUPPORTED;
        if ((long long)a.Kb * 32 > IM_STAGE_BYTES) return BTC_ERR_UNSUPPORTED;      // one 16-row tile must fit a stage
        p.x = a.x; p.idx = a.idx; p.alpha = a.alpha; p.mu = a.mu; p.y = a.y;
        const int Kc4 = (a.Kc + 3) / 4 * 4;
        p.tab = a.Cp + 2 * Kc4;                      // byte-lane words follow the two other forms
        p.M = a.M; p.N = a.N; p.K = a.K; p.v = a.v; p.Kc = a.Kc; p.Kb = a.Kb;
        p.x_dt = a.x_dt; p.y_dt = a.y_dt;
        p.nq = (a.Kb + 255) / 256;
        p.ncls = (a.v + 3) / 4;
        p.tiles = (a.N + 15) / 16;
        if (p.ncls > ncls_max) ncls_max = p.ncls;
        if (p.nq > nq_max) nq_max = p.nq;
        if (a.M > m_max) m_max = a.M;
        if (Kc4 * 4 > tab_max) tab_max = Kc4 * 4;
    }
    const int nm = m_max <= 2 ? 1 : (m_max <= 5 ? 2 : 3);
    for (int i = 0; i < count; ++i) {
        ImProblem &p = b.p[i];
        p.tr = (nm == 1 && (long long)p.Kb * 64 <= IM_STAGE_BYTES && p.tiles > 1) ? 2 : 1;
        p.iters = (p.tiles + p.tr - 1) / p.tr;
        p.iter_begin = it;
        it += p.iters;
    }
    b.total_iters = it;
    const int part_ints = (nm == 1 ? IM_TR : 1) * 16 * 8 * nm;
    b.tab_smem_bytes = tab_max;
    if (im_smem_layout(tab_max, part_ints).total > 227u * 1024u) b.tab_smem_bytes = 0;   // gather from global (L1/L2)
    if (ncls_max <= 4) return im_launch_nq<4>(b, nq_max, nm, s);
    return im_launch_nq<5>(b, nq_max, nm, s);
}

int imma_status_read(int *out)
{
    int v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, g_imma_status, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    *out = v;
    return BTC_OK;
}

}  // namespace btc
