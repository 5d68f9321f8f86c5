// Decode path for M <= 8: streams the index matrix once and evaluates every block dot
//     <x_j, C[idx]> = 2 * sum_{bit=1} x  -  sum x          (identity for +-1 codewords)
// with fp32 accumulation (block-dot sum of the paper's appendix "Binary codebook LUT-GEMM").
//
// How sum_{bit=1} x is formed without expanding bits one by one
// -------------------------------------------------------------
// An fp16 bit pattern with a single bit i <= 11 set is the number 2^(i-24) (a subnormal for
// i < 10).  So `word & mask`, where mask keeps one bit per 16-bit half, *is* a pair of fp16
// numbers {0 or 2^(i-24)}: one LOP3 turns two stored weight bits into two usable multiplicands.
// The activations are pre-scaled once per call by the matching 2^-c (c = position class of the
// weight inside its block), so every product equals bit * x * 2^(P0-24) exactly and the sum can be
// taken by the warp-level mma.sync.m16n8k16 (fp16 inputs, exact products, fp32 accumulate):
//     A (16 rows x 16 k)  = masked codeword bits of 16 output rows,
//     B (16 k x 8 cols)   = pre-scaled activations of up to 8 rows of x (cols = m),
//     D (16 x 8, fp32)    = 2^(P0-24) * sum_{bit=1} x  for 16 outputs x 8 activation rows.
// The k dimension of one MMA is permuted so that each thread supplies bits of a block it owns:
// thread (g = lane/4, t = lane%4) owns, for rows g and g+8, the block j0+t of a group of four
// blocks; MMA q of the group consumes weights 4q..4q+3 of those blocks.  Hence every codeword is
// fetched exactly once (one shared-memory gather per index) and every stored bit is touched by
// exactly one LOP3 (two bits per instruction).
//
// The per-layer codeword table in this "MMA layout" (bit of weight t at (t&1)*16 + P0 + (t>>1),
// P0 = 12 - v/2) is written by btc_codebook_pack behind the public words.
//
// Work split: persistent CTAs, 16 warps.  A CTA owns a contiguous range of 16-row tiles; the 16
// warps split K; partial sums meet in shared memory in a fixed order (deterministic).
#include "btc_internal.cuh"

namespace btc {

constexpr int DEC_WARPS = 16;
constexpr int DEC_THREADS = DEC_WARPS * 32;

__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct DecParams {
    LinearArgs a;
    const uint32_t *Cm;      // codeword table in MMA layout, [Kc]
    int tiles;               // ceil(N / 16)
    int L;                   // blocks per warp K-slice (multiple of 4)
    int xs_stride;           // halves per row of the scaled-activation buffer
    int table_in_smem;
};

// Shared memory carve-up (dynamic): [table Kc*4] [xs M*xs_stride*2] [partials 2*16*128*4] [sumx 8*4] [red 8*16*4]
template <int V, int LG, bool BREG>
__global__ void __launch_bounds__(DEC_THREADS, 1)
gemv_decode_kernel(const DecParams p)
{
    constexpr int NQ = V / 4;            // MMAs per group of four blocks
    constexpr int P0 = 12 - V / 2;       // lowest bit position used in each 16-bit half
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const LinearArgs &a = p.a;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;

    uint32_t *s_tab = reinterpret_cast<uint32_t *>(smem_raw);
    const size_t tab_bytes = p.table_in_smem ? (((size_t)a.Kc * 4 + 15) / 16) * 16 : 0;
    __half *s_x = reinterpret_cast<__half *>(smem_raw + tab_bytes);
    const size_t xs_bytes = (((size_t)a.M * p.xs_stride * 2) + 15) / 16 * 16;
    float *s_part = reinterpret_cast<float *>(smem_raw + tab_bytes + xs_bytes);   // [2][16 warps][128]
    float *s_sumx = s_part + 2 * DEC_WARPS * 128;                                    // [8]
    float *s_red = s_sumx + 8;                                                      // [8][16 warps]

    // ---- tile range of this CTA
    const int per = p.tiles / gridDim.x, rem = p.tiles % gridDim.x;
    const int tile_begin = blockIdx.x * per + min((int)blockIdx.x, rem);
    const int tile_end = tile_begin + per + ((int)blockIdx.x < rem ? 1 : 0);

    // ---- this thread's blocks: LG consecutive blocks starting at jb, for rows g and g+8
    const int L = p.L;
    const int lg_run = L / 4;                       // groups per warp slice (<= LG when BREG)
    const int jb = warp * L + t * lg_run;

    // ---- prologue 1: codeword table -> shared memory
    if (p.table_in_smem) {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.Cm);
        uint4 *dst = reinterpret_cast<uint4 *>(s_tab);
        const int n16 = (a.Kc * 4) / 16;
        for (int i = tid; i < n16; i += DEC_THREADS) dst[i] = __ldg(src + i);
        for (int i = n16 * 4 + tid; i < a.Kc; i += DEC_THREADS) s_tab[i] = __ldg(p.Cm + i);
    }
    // ---- prologue 2: x -> x * 2^-(class) as fp16 in shared memory, and sum_k x[m,k]
    for (int m = 0; m < a.M; ++m) {
        float part = 0.f;
        for (int k = tid; k < a.K; k += DEC_THREADS) {
            const float xv = load_as_float(a.x, a.x_dt, (size_t)m * a.K + k);
            part += xv;
            const int cls = (k % V) >> 1;
            s_x[(size_t)m * p.xs_stride + k] = __float2half_rn(ldexpf(xv, -cls));
        }
        part = warp_sum(part);
        if (lane == 0) s_red[m * DEC_WARPS + warp] = part;
    }
    __syncthreads();
    if (tid < a.M) {
        float s = 0.f;
        for (int w = 0; w < DEC_WARPS; ++w) s += s_red[tid * DEC_WARPS + w];   // fixed order
        s_sumx[tid] = s;
    }
    __syncthreads();

    // ---- B fragments (pre-scaled activations of row m = g for this thread's blocks)
    uint32_t breg[BREG ? LG : 1][2 * NQ];
    if (BREG) {
#pragma unroll
        for (int i = 0; i < LG; ++i) {
            const int j = jb + i;
            const bool ok = (i < lg_run) && (j < a.Kb) && (g < a.M);
#pragma unroll
            for (int r = 0; r < 2 * NQ; ++r)
                breg[i][r] = ok ? *reinterpret_cast<const uint32_t *>(s_x + (size_t)g * p.xs_stride + (size_t)j * V + 2 * r) : 0u;
        }
    }

    uint32_t mask0[NQ], mask2[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        mask0[q] = (1u << (P0 + 2 * q)) | (1u << (16 + P0 + 2 * q));
        mask2[q] = (1u << (P0 + 2 * q + 1)) | (1u << (16 + P0 + 2 * q + 1));
    }

    const uint32_t *tab = p.table_in_smem ? s_tab : p.Cm;
    const float unscale = ldexpf(2.0f, 24 - P0);     // 2 * 2^(24-P0): turns D into 2*sum_{bit=1} x

    // ---- index prefetch for the first tile
    uint16_t inext[BREG ? LG : 1][2];
    auto load_idx = [&](int tile, int i, int which) -> uint16_t {
        const int row = min(tile * 16 + g + which * 8, a.N - 1);
        const int j = jb + i;
        return (i < lg_run && j < a.Kb) ? __ldg(a.idx + (size_t)row * a.Kb + j) : (uint16_t)0;
    };
    if (BREG && tile_begin < tile_end) {
#pragma unroll
        for (int i = 0; i < LG; ++i) { inext[i][0] = load_idx(tile_begin, i, 0); inext[i][1] = load_idx(tile_begin, i, 1); }
    }

    int buf = 0;
    for (int tile = tile_begin; tile < tile_end; ++tile, buf ^= 1) {
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        if (BREG) {
            uint16_t icur[LG][2];
#pragma unroll
            for (int i = 0; i < LG; ++i) { icur[i][0] = inext[i][0]; icur[i][1] = inext[i][1]; }
            if (tile + 1 < tile_end) {
#pragma unroll
                for (int i = 0; i < LG; ++i) { inext[i][0] = load_idx(tile + 1, i, 0); inext[i][1] = load_idx(tile + 1, i, 1); }
            }
#pragma unroll
            for (int i = 0; i < LG; ++i) {
                if (i < lg_run) {
                    const uint32_t w0 = p.table_in_smem ? tab[icur[i][0]] : __ldg(tab + icur[i][0]);
                    const uint32_t w1 = p.table_in_smem ? tab[icur[i][1]] : __ldg(tab + icur[i][1]);
#pragma unroll
                    for (int q = 0; q < NQ; ++q)
                        mma_f16_16816(c, w0 & mask0[q], w1 & mask0[q], w0 & mask2[q], w1 & mask2[q],
                                      breg[i][2 * q], breg[i][2 * q + 1]);
                }
            }
        } else {
            // Large K: activations stay in shared memory, indices are read as they are needed.
            for (int i = 0; i < lg_run; ++i) {
                const int j = jb + i;
                const bool okb = (j < a.Kb);
                const uint16_t i0 = load_idx(tile, i, 0), i1 = load_idx(tile, i, 1);
                const uint32_t w0 = p.table_in_smem ? tab[i0] : __ldg(tab + i0);
                const uint32_t w1 = p.table_in_smem ? tab[i1] : __ldg(tab + i1);
                const bool ok = okb && (g < a.M);
                const uint32_t *xb = reinterpret_cast<const uint32_t *>(s_x + (size_t)(ok ? g : 0) * p.xs_stride + (size_t)(okb ? j : 0) * V);
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const uint32_t b0 = ok ? xb[2 * q] : 0u, b1 = ok ? xb[2 * q + 1] : 0u;
                    mma_f16_16816(c, w0 & mask0[q], w1 & mask0[q], w0 & mask2[q], w1 & mask2[q], b0, b1);
                }
            }
        }
        // ---- partial sums of this warp's K-slice -> shared memory: [row 0..15][m 0..7]
        float *mine = s_part + ((size_t)buf * DEC_WARPS + warp) * 128;
        mine[g * 8 + 2 * t] = c[0];
        mine[g * 8 + 2 * t + 1] = c[1];
        mine[(g + 8) * 8 + 2 * t] = c[2];
        mine[(g + 8) * 8 + 2 * t + 1] = c[3];
        __syncthreads();
        if (tid < 128) {
            const int r = tid >> 3, m = tid & 7;
            const int n = tile * 16 + r;
            if (n < a.N && m < a.M) {
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < DEC_WARPS; ++w) s += s_part[((size_t)buf * DEC_WARPS + w) * 128 + tid];
                const float sx = s_sumx[m];
                float y = __half2float(a.alpha[n]) * (s * unscale - sx);
                if (a.mu) y += __half2float(a.mu[n]) * sx;
                store_from_float(a.y, a.y_dt, (size_t)m * a.N + n, y);
            }
        }
        // the other partial buffer is used by the next tile, so one barrier per tile is enough
    }
}

struct DecPlan {
    bool ok;
    int L, lg, xs_stride, table_in_smem;
    size_t smem;
};

static DecPlan plan(const LinearArgs &a)
{
    DecPlan d{};
    d.ok = false;
    if (a.M > 8 || a.v % 4 || a.v < 4 || a.v > 24) return d;
    const int groups = (a.Kb + 3) / 4;
    const int gpw = (groups + DEC_WARPS - 1) / DEC_WARPS;     // groups per warp slice
    d.L = gpw * 4;
    d.lg = gpw;
    d.xs_stride = a.K + 8;                                      // +16 bytes: rows of x land in different banks
    const size_t xs = (((size_t)a.M * d.xs_stride * 2) + 15) / 16 * 16;
    const size_t fixed = xs + (size_t)2 * DEC_WARPS * 128 * 4 + 8 * 4 + 8 * DEC_WARPS * 4;
    const size_t tab = (((size_t)a.Kc * 4 + 15) / 16) * 16;
    const size_t cap = 227 * 1024;
    if (fixed > cap) return d;
    d.table_in_smem = (fixed + tab <= cap) && a.Kc <= 32768;
    d.smem = fixed + (d.table_in_smem ? tab : 0);
    d.ok = true;
    return d;
}

template <int V, int LG, bool BREG>
static int launch_one(const DecParams &p, size_t smem, int grid, cudaStream_t s)
{
    auto kern = gemv_decode_kernel<V, LG, BREG>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    kern<<<grid, DEC_THREADS, smem, s>>>(p);
    return cuda_check_launch();
}

template <int V>
static int launch_v(const DecParams &p, const DecPlan &d, int grid, cudaStream_t s)
{
    if (d.lg <= 1) return launch_one<V, 1, true>(p, d.smem, grid, s);
    if (d.lg <= 2) return launch_one<V, 2, true>(p, d.smem, grid, s);
    if (d.lg <= 4) return launch_one<V, 4, true>(p, d.smem, grid, s);
    if (d.lg <= 8 && V <= 16) return launch_one<V, 8, true>(p, d.smem, grid, s);
    return launch_one<V, 1, false>(p, d.smem, grid, s);
}

static int sm_count()
{
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

int launch_gemv_decode(const LinearArgs &a, cudaStream_t s)
{
    const DecPlan d = plan(a);
    if (!d.ok) return BTC_ERR_UNSUPPORTED;
    DecParams p;
    p.a = a;
    p.Cm = a.Cp + (a.Kc + 3) / 4 * 4;   // MMA-layout words follow the public words (16-byte aligned)
    p.tiles = (a.N + 15) / 16;
    p.L = d.L;
    p.xs_stride = d.xs_stride;
    p.table_in_smem = d.table_in_smem;
    const int grid = p.tiles < sm_count() ? p.tiles : sm_count();
    switch (a.v) {
    case 4: return launch_v<4>(p, d, grid, s);
    case 8: return launch_v<8>(p, d, grid, s);
    case 12: return launch_v<12>(p, d, grid, s);
    case 16: return launch_v<16>(p, d, grid, s);
    case 20: return launch_v<20>(p, d, grid, s);
    case 24: return launch_v<24>(p, d, grid, s);
    default: return BTC_ERR_UNSUPPORTED;
    }
}

size_t gemv_decode_workspace_bytes(int, int, int, int, int) { return 0; }

}  // namespace btc
