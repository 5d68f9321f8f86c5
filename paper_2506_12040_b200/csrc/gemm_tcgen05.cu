// Tensor-core path: y[M,N] = x[M,K] * W^[N,K]^T with W^ = alpha * C[idx] (+ mu), for large M.
//
// The contraction runs on the 5th-generation tensor cores (tcgen05.mma, kind::f16, fp32 accumulators in tensor
// memory).  The weight tile is the A operand (128 rows = UMMA M), x is the B operand (BM rows = UMMA N, loaded by TMA
// with the 128-byte swizzle), so the accumulator holds y^T: tensor-memory lane = output feature n, column = activation
// row m, and a warp stores 32 consecutive n for one m (coalesced).  The decoded tile is pure +-1 and the row scale is
// applied in the fp32 epilogue, which is exact for a row-wise alpha.
//
// Two kernels: gemm_v16t_kernel (v = 16; decoded weights go straight into tensor memory, see its header) and
// gemm_tcgen05_kernel (any v; one thread per weight row writes the +-1 tile into shared memory):
//   warp 0     TMA producer: x tiles [BM rows x 64 k] -> shared memory
//   warp 1     MMA issuer: one elected thread issues tcgen05.mma for every 64-wide k step
//   warp 2     allocates / frees tensor memory
//   warps 4-7  decode producers: thread r expands the indices of weight row n0+r for the current 64-wide k step into
//              +-1 bf16 (or fp16) in the swizzled K-major layout the MMA reads; afterwards the same warps run the
//              epilogue: tcgen05.ld, scale by alpha_n in fp32 (+ mu_n * sum_k x[m,k]), store y.
//
// Every mbarrier wait is bounded: after ~2 s of polling the CTA raises a status word, stops waiting and runs to
// completion (the output is then undefined and btc_device_status reports the timeout).
#include <cuda.h>
#include "btc_internal.cuh"

namespace btc {

constexpr int G_BN = 128;          // weight rows per tile (UMMA M)
constexpr int G_BK = 64;           // k per stage: 64 x 2 bytes = one 128-byte swizzle row
constexpr int G_THREADS = 256;
constexpr uint32_t G_A_BYTES = G_BN * G_BK * 2;

__device__ int g_gemm_status = 0;  // 0 = ok, 7 = a bounded wait ran out

// ------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and latches *abort_flag) when the deadline passes.  BACKOFF: sleep between polls;
// every role but the MMA issuer uses it, because a warp that spins takes issue slots from the one thread whose
// instruction stream paces the tensor core.
template <bool BACKOFF = true>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    const long long t0 = clock64();
    int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (BACKOFF) __nanosleep(spins < 8 ? 32 : 128);
        if ((++spins & 63) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > 4000000000LL) {   // ~2 s at 2 GHz
                *abort_flag = 1;
                atomicExch(&g_gemm_status, (int)BTC_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major, 128-byte-swizzled operand tile whose rows are 128 bytes: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);          // start address, 16-byte units
    d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                            // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
    return d;
}

struct GemmParams {
    LinearArgs a;
    const float *sumx;       // [M] row sums of x (only read when mu != nullptr)
    int k_tiles;             // ceil(K / 64)
};

// sum_k x[m,k] in fp32, one warp per row (needed only for the mean term).
__global__ void rowsum_kernel(const void *x, int x_dt, int M, int K, float *out)
{
    const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (m >= M) return;
    float s = 0.f;
    for (int k = threadIdx.x & 31; k < K; k += 32) s += load_as_float(x, x_dt, (size_t)m * K + k);
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) out[m] = s;
}

template <int BM, int STAGES>
__global__ void __launch_bounds__(G_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_x, const GemmParams p)
{
    constexpr uint32_t B_BYTES = BM * G_BK * 2;
    constexpr uint32_t STAGE_BYTES = G_A_BYTES + B_BYTES;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // carve: stages (1024-byte aligned), then barriers
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_gen + (size_t)STAGES * STAGE_BYTES);
    // bars: [0,S) full_x, [S,2S) full_w, [2S,3S) empty, [3S] accum
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(bars + 3 * STAGES + 1);
    volatile int *s_abort = reinterpret_cast<volatile int *>(s_tmem + 1);

    const LinearArgs &a = p.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * G_BN;
    const int m0 = blockIdx.y * BM;
    const int KT = p.k_tiles;
    const bool is_bf16 = (a.x_dt == BTC_BF16);

    auto bar_full_x = [&](int s) { return smem_u32(bars + s); };
    auto bar_full_w = [&](int s) { return smem_u32(bars + STAGES + s); };
    auto bar_empty = [&](int s) { return smem_u32(bars + 2 * STAGES + s); };
    const uint32_t bar_accum = smem_u32(bars + 3 * STAGES);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full_x(s), 1);
            mbar_init(bar_full_w(s), 128);
            mbar_init(bar_empty(s), 1);
        }
        mbar_init(bar_accum, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) tmem_alloc(smem_u32(s_tmem), BM);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = *s_tmem;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (x tiles)
        if (lane == 0) {
            for (int kt = 0; kt < KT; ++kt) {
                const int s = kt % STAGES;
                const uint32_t ph = (kt / STAGES) & 1;
                if (kt >= STAGES) mbar_wait(bar_empty(s), ph ^ 1, s_abort);
                mbar_expect_tx(bar_full_x(s), B_BYTES);
                const uint32_t dst = smem_base + s * STAGE_BYTES + G_A_BYTES;
                tma_load_2d(dst, &tmap_x, kt * G_BK, m0, bar_full_x(s));
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // kind::f16 instruction descriptor: D = f32, A/B = bf16 or f16, both K-major, M = 128, N = BM
            uint32_t idesc = (1u << 4) | ((uint32_t)(BM >> 3) << 17) | ((uint32_t)(G_BN >> 4) << 24);
            if (is_bf16) idesc |= (1u << 7) | (1u << 10);
            for (int kt = 0; kt < KT; ++kt) {
                const int s = kt % STAGES;
                const uint32_t ph = (kt / STAGES) & 1;
                mbar_wait<false>(bar_full_x(s), ph, s_abort);
                mbar_wait<false>(bar_full_w(s), ph, s_abort);
                tc_fence_after();
                const uint32_t a_addr = smem_base + s * STAGE_BYTES;
                const uint64_t adesc = make_smem_desc(a_addr);
                const uint64_t bdesc = make_smem_desc(a_addr + G_A_BYTES);
#pragma unroll
                for (int k = 0; k < G_BK / 16; ++k)      // +32 bytes per 16-wide k step inside the swizzle row
                    umma_f16(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, (kt | k) ? 1u : 0u);
                umma_commit(bar_empty(s));               // frees the stage when these MMAs have read it
            }
            umma_commit(bar_accum);                      // accumulator complete
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ decode producers (weights -> A tile)
        const int r = tid - 128;                          // row inside the tile, also the TMEM lane
        const int n = min(n0 + r, a.N - 1);
        const uint16_t *irow = a.idx + (size_t)n * a.Kb;
        const uint32_t one2 = is_bf16 ? 0x3F803F80u : 0x3C003C00u;
        const int v = a.v;
        for (int kt = 0; kt < KT; ++kt) {
            const int s = kt % STAGES;
            const uint32_t ph = (kt / STAGES) & 1;
            // 64 weight bits of this row for k in [k0, k0+64), gathered from the public codeword words
            const int k0 = kt * G_BK;
            const int jf = k0 / v;
            const int jl = min((k0 + G_BK - 1) / v, a.Kb - 1);
            uint64_t win = 0;
            for (int j = jf; j <= jl; ++j) {
                const uint64_t w = __ldg(a.Cp + __ldg(irow + j));
                const int off = j * v - k0;
                win |= (off >= 0) ? (w << off) : (w >> (-off));
            }
            const uint64_t neg = ~win;                    // sign bit set where the weight is -1
            if (kt >= STAGES) mbar_wait(bar_empty(s), ph ^ 1, s_abort);
            unsigned char *arow = smem_gen + (size_t)s * STAGE_BYTES + (size_t)r * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t b = (uint32_t)(neg >> (8 * c)) & 0xFFu;
                uint4 q;
                q.x = one2 | ((b & 1u) << 15) | ((b & 2u) << 30);
                q.y = one2 | ((b & 4u) << 13) | ((b & 8u) << 28);
                q.z = one2 | ((b & 16u) << 11) | ((b & 32u) << 26);
                q.w = one2 | ((b & 64u) << 9) | ((b & 128u) << 24);
                *reinterpret_cast<uint4 *>(arow + ((c ^ (r & 7)) << 4)) = q;   // 128-byte swizzle
            }
            fence_proxy_async_smem();                     // make the generic-proxy writes visible to the MMA
            mbar_arrive(bar_full_w(s));
        }
        // ------------------------------------------------------------ epilogue
        mbar_wait(bar_accum, 0, s_abort);
        tc_fence_after();
        const int nrow = n0 + r;
        const float al = __half2float(a.alpha[n]);
        const float mu = a.mu ? __half2float(a.mu[n]) : 0.f;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
#pragma unroll 1
        for (int c0 = 0; c0 < BM; c0 += 32) {
            uint32_t rr[32];
            tmem_ld32(tmem_d + lane_base + c0, rr);
            tmem_ld_wait();
            if (nrow < a.N) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int m = m0 + c0 + i;
                    if (m < a.M) {
                        float y = al * __uint_as_float(rr[i]);
                        if (a.mu) y += mu * p.sumx[m];
                        store_from_float(a.y, a.y_dt, (size_t)m * a.N + nrow, y);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*s_abort) {
        // give copies that may still be in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 2) tmem_dealloc(tmem_d, BM);
}

// ------------------------------------------------------------------------------------ v = 16: shared declarations
// For v = 16 a 64-wide k step is four blocks.  The codeword table of the "fp16 layout" keeps the bit of weight t at
// (t & 1) * 16 + 4 + (t >> 1), so ((~w << (11 - j)) & 0x80008000) | {1.0, 1.0} is the pair of weights (2j, 2j+1) as +-1
// in bf16 / fp16: one shift and one LOP3 per pair.  Index tiles (128 rows x 64 blocks = 16 k steps, 128-byte swizzle)
// arrive by TMA; the table is bulk-copied into shared memory when it fits.
constexpr int G2_DWARPS = 16;                    // decode warps (four groups of four)
constexpr int G2_THREADS = 128 + G2_DWARPS * 32;
constexpr uint32_t G2_IDX_BYTES = 128 * 128;     // one index tile

struct Gemm2Params {
    LinearArgs a;
    const float *sumx;
    const uint32_t *tab;     // fp16-layout codeword words [Kc4]
    int k_tiles;
    int tab_bytes;           // > 0: table staged in shared memory
};

struct SplitArgs {
    int split_tiles;         // k tiles (a multiple of 16: whole index tiles) per CTA along grid.z
    float *part;             // raw partial sums [grid.z][M][N]
};

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------ v = 16 and v = 20, weights in tensor memory
// With both operands in shared memory the kernel above is bound by shared-memory bandwidth: per 64-wide k step the
// tensor core reads the A and B tiles while the decode warps write 16 KB of A and TMA writes the x tile, more than
// the 128 bytes per clock an SM's shared memory delivers (66 % of the MMA rate at best with 256-row x tiles, 50 % with
// 128-row ones).  Here the decoded +-1 tile never touches shared memory: each decode thread owns one weight row =
// one tensor-memory lane, expands the row's 64 weights of a k step into 32 registers and stores them with
// tcgen05.st into a ring of A tiles in tensor memory (32 columns per k step); the MMAs take A from tensor memory and
// only the x tile from shared memory.
//   warp 0 TMA producer (x tiles, index tiles, table) | warp 1 MMA issuer | warp 2 tensor-memory allocation
//   warps 4-19: four groups of four warps; group g expands the k steps g, g + 4, ...; then all 16 run the epilogue.
// Tensor memory (512 columns): accumulator in columns [0, BM), A ring of STAGES x 32 columns from column 256.
constexpr int G4_A_COL0 = 256;

__device__ __forceinline__ void umma_f16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
           "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
           "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
           "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// SPLIT: the CTAs of a tile share K along grid.z and leave raw partial sums in p.part (a separate instantiation, so
// that the unsplit kernel carries none of it).
// v = 20: the 64 weights of step S of a super-block are the weight pairs 2 S .. 2 S + 31 of its four blocks (ten pairs each);
// in the fp16-layout word of a 20-bit codeword pair j sits at bits (2 + j, 18 + j).
template <int S>
__device__ __forceinline__ void expand_v20(const uint32_t (&w)[4], uint32_t one2, uint32_t (&regs)[32])
{
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int q = 2 * S + i, c = q / 10, j = q - 10 * c;
        regs[i] = ((w[c] << (13 - j)) & 0x80008000u) | one2;
    }
}

template <int BM, int STAGES, int KS, bool SPLIT, int V>
__global__ void __launch_bounds__(G2_THREADS, 1)
gemm_v16t_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_i, const Gemm2Params p, const SplitArgs sp)
{
    constexpr uint32_t B_BYTES = BM * G_BK * 2;                    // one x tile (64 k); a stage holds KS of them
    constexpr uint32_t STAGE_BYTES = KS * B_BYTES;
    constexpr int ACOLS = 32 * KS;                                 // tensor-memory columns of a stage's A tile
    // An index tile of 64 blocks covers 64 * V weights = V k steps: 16 for v = 16 (four whole blocks per step); 20 for
    // v = 20, where a step takes 64 weights out of four consecutive blocks, starting 0, 4, 8, 12 or 16 weights into the
    // first (five steps = sixteen blocks, then the pattern repeats).
    constexpr int KPT = V;
    static_assert(V == 16 || V == 20, "index tiles of 64 blocks and whole k steps");
    // With 128-row x tiles an MMA runs for 64 clk, less than it takes one thread to issue it next to sixteen busy decode
    // warps; then two threads issue (warp 1: even stages into accumulator 0; warp 3: odd stages into accumulator 1 in
    // columns [128, 256)) and the epilogue adds the two accumulators.
    constexpr int NACC = (BM == 128) ? 2 : 1;
    static_assert(BM * ((BM == 128) ? 2 : 1) <= G4_A_COL0, "accumulators and A ring must not overlap");
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    unsigned char *s_idx = smem_gen + (size_t)STAGES * STAGE_BYTES;                 // 2 index tiles
    uint32_t *s_tab = reinterpret_cast<uint32_t *>(s_idx + 2 * G2_IDX_BYTES);
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(s_tab) + ((p.tab_bytes + 15) & ~15));
    // One ring of STAGES stages holds both operands of a k step: the x tile in shared memory and the A tile in tensor
    // memory.  full[s]: the TMA arrival (with its bytes) plus the four decode warps; empty[s]: the MMAs' commit.
    // bars: [0,S) full, [S,2S) empty, accum, full_i[2], empty_i[2], tab_full
    static_assert(STAGES % 4 == 0 && STAGES * ACOLS <= 512 - G4_A_COL0 && KPT % KS == 0, "a decode group must meet a stage in consecutive phases");
    constexpr int NB = 2 * STAGES + 6;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(bars + NB);
    volatile int *s_abort = reinterpret_cast<volatile int *>(s_tmem + 1);

    const LinearArgs &a = p.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * G_BN, m0 = blockIdx.y * BM;
    // a CTA covers the k tiles [kt_first, kt_first + KT): all of them, or its share along grid.z (whole index tiles)
    const int kt_first = SPLIT ? blockIdx.z * sp.split_tiles : 0;
    const int KT = SPLIT ? min(sp.split_tiles, p.k_tiles - kt_first) : p.k_tiles;
    const int NS = (KT + KS - 1) / KS;                              // stages' worth of k steps
    const bool is_bf16 = (a.x_dt == BTC_BF16);
    auto bar_full = [&](int s) { return smem_u32(bars + s); };
    auto bar_empty = [&](int s) { return smem_u32(bars + STAGES + s); };
    const uint32_t bar_accum = smem_u32(bars + 2 * STAGES);
    auto bar_full_i = [&](int b) { return smem_u32(bars + 2 * STAGES + 1 + b); };
    auto bar_empty_i = [&](int b) { return smem_u32(bars + 2 * STAGES + 3 + b); };
    const uint32_t bar_tab = smem_u32(bars + 2 * STAGES + 5);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full(s), 1 + 4); mbar_init(bar_empty(s), 1); }
        mbar_init(bar_accum, NACC);
        for (int b = 0; b < 2; ++b) { mbar_init(bar_full_i(b), 1); mbar_init(bar_empty_i(b), G2_DWARPS); }
        mbar_init(bar_tab, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) tmem_alloc(smem_u32(s_tmem), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = *s_tmem;
    if (SPLIT) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the reduce kernel may take its place early

    if (warp == 0) {
        if (lane == 0) {
            if (p.tab_bytes > 0) {
                mbar_expect_tx(bar_tab, (uint32_t)p.tab_bytes);
                bulk_g2s(smem_u32(s_tab), p.tab, (uint32_t)p.tab_bytes, bar_tab);
            }
            for (int ks = 0; ks < NS; ++ks) {
                const int kt0 = ks * KS;
                if (kt0 % KPT == 0) {
                    const int it = kt0 / KPT, ib = it & 1;
                    if (it >= 2 && !mbar_wait(bar_empty_i(ib), ((it >> 1) & 1) ^ 1, s_abort)) break;
                    mbar_expect_tx(bar_full_i(ib), G2_IDX_BYTES);
                    tma_load_2d(smem_u32(s_idx + (size_t)ib * G2_IDX_BYTES), &tmap_i, (kt_first / KPT) * 64 + it * 64, n0, bar_full_i(ib));
                }
                const int s = ks % STAGES;
                if (ks >= STAGES && !mbar_wait(bar_empty(s), ((ks / STAGES) & 1) ^ 1, s_abort)) break;
                mbar_expect_tx(bar_full(s), STAGE_BYTES);
#pragma unroll
                for (int j = 0; j < KS; ++j)             // (a box past K arrives as zeros)
                    tma_load_2d(smem_base + s * STAGE_BYTES + j * B_BYTES, &tmap_x, (kt_first + kt0 + j) * G_BK, m0, bar_full(s));
            }
        }
    } else if (warp == 1 || (NACC == 2 && warp == 3)) {
        if (lane == 0) {
            const int me = (warp == 1) ? 0 : 1;                    // which accumulator / which stages
            uint32_t idesc = (1u << 4) | ((uint32_t)(BM >> 3) << 17) | ((uint32_t)(G_BN >> 4) << 24);
            if (is_bf16) idesc |= (1u << 7) | (1u << 10);
            const uint32_t d_tm = tmem_d + me * BM;
            for (int ks = me; ks < NS; ks += NACC) {
                const int s = ks % STAGES;
                if (!mbar_wait<false>(bar_full(s), (ks / STAGES) & 1, s_abort)) break;
                tc_fence_after();
                const uint32_t a_tm = tmem_d + G4_A_COL0 + s * ACOLS;
#pragma unroll
                for (int j = 0; j < KS; ++j) {
                    const uint64_t bdesc = make_smem_desc(smem_base + s * STAGE_BYTES + j * B_BYTES);
#pragma unroll
                    for (int k = 0; k < G_BK / 16; ++k)
                        umma_f16_ts(d_tm, a_tm + 32 * j + 8 * k, bdesc + 2 * k, idesc, (ks >= NACC || j || k) ? 1u : 0u);
                }
                umma_commit(bar_empty(s));
            }
            umma_commit(bar_accum);
        }
    } else if (warp >= 4) {
        const int r = (tid - 128) & 127;               // weight row of the tile = tensor-memory lane
        const int grp = (tid - 128) >> 7;              // k steps grp, grp + 4, ...: STAGES is a multiple of 4, so a stage is always
                                                       // met by the same group, phase after phase: its parity waits are unambiguous
        const uint32_t one2 = is_bf16 ? 0x3F803F80u : 0x3C003C00u;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const bool tab_smem = p.tab_bytes > 0;
        if (tab_smem && !mbar_wait(bar_tab, 0, s_abort)) { /* fall through: waits below bail out */ }
        bool ok = true;
        int cur_it = -1;
        for (int ks = grp; ks < NS && ok; ks += 4) {
            const int kt0 = ks * KS;
            const int it = kt0 / KPT, ib = it & 1;
            if (it != cur_it) {
                if (!mbar_wait(bar_full_i(ib), (it >> 1) & 1, s_abort)) { ok = false; break; }
                cur_it = it;
            }
            // the four indices per k step of this row.  v = 16: columns (kt % 16) * 4 .. + 3 of the index tile (8 bytes);
            // v = 20: step s of super-block q (16 blocks) starts in block 16 q + 3 s
            uint32_t w[KS][4];
            int spos[KS];
#pragma unroll
            for (int j = 0; j < KS; ++j) {
                const int ktl = (kt0 + j) % KPT;
                const unsigned char *irow_s = s_idx + (size_t)ib * G2_IDX_BYTES + (size_t)r * 128;
                uint32_t i4[4];
                if (V == 16) {
                    const int boff = ktl * 8;
                    const uint2 quad = *reinterpret_cast<const uint2 *>(irow_s + ((((boff >> 4) & 7) ^ (r & 7)) << 4) + (boff & 15));
                    i4[0] = quad.x & 0xffffu; i4[1] = quad.x >> 16; i4[2] = quad.y & 0xffffu; i4[3] = quad.y >> 16;
                    spos[j] = 0;
                } else {
                    const int sb = ktl / 5, sp5 = ktl - 5 * sb;
                    spos[j] = sp5;
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const int boff = (16 * sb + 3 * sp5 + b) * 2;
                        i4[b] = *reinterpret_cast<const uint16_t *>(irow_s + ((((boff >> 4) & 7) ^ (r & 7)) << 4) + (boff & 15));
                    }
                }
#pragma unroll
                for (int b = 0; b < 4; ++b) w[j][b] = ~(tab_smem ? s_tab[i4[b]] : __ldg(p.tab + i4[b]));
            }
            if (((ks + 4) * KS) / KPT != it || ks + 4 >= NS) {     // this group's last stage in the index tile
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty_i(ib));
            }
            const int sa = ks % STAGES;
            if (ks >= STAGES && !mbar_wait(bar_empty(sa), ((ks / STAGES) & 1) ^ 1, s_abort)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int j = 0; j < KS; ++j) {
                // register i holds the weights 2i, 2i+1 of the k step (K elements 2i, 2i+1 of this row of A)
                uint32_t regs[32];
                if (V == 16) {
#pragma unroll
                    for (int b = 0; b < 4; ++b)
#pragma unroll
                        for (int i = 0; i < 8; ++i) regs[8 * b + i] = ((w[j][b] << (11 - i)) & 0x80008000u) | one2;
                } else {
                    switch (spos[j]) {
                    case 0: expand_v20<0>(w[j], one2, regs); break;
                    case 1: expand_v20<1>(w[j], one2, regs); break;
                    case 2: expand_v20<2>(w[j], one2, regs); break;
                    case 3: expand_v20<3>(w[j], one2, regs); break;
                    default: expand_v20<4>(w[j], one2, regs); break;
                    }
                }
                tmem_st32(tmem_d + lane_base + G4_A_COL0 + sa * ACOLS + 32 * j, regs);
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_full(sa));
        }
        // ------------------------------------------------------------ epilogue: four warps per lane quadrant
        if (ok && mbar_wait(bar_accum, 0, s_abort)) {
            tc_fence_after();
            const int wl = warp - 4;
            const int q4 = wl & 3, quarter = wl >> 2;
            const int nrow = n0 + q4 * 32 + lane;
            const int nc = min(nrow, a.N - 1);
            const float al = __half2float(a.alpha[nc]);
            const float mu = a.mu ? __half2float(a.mu[nc]) : 0.f;
#pragma unroll 1
            for (int c0 = quarter * (BM / 4); c0 < (quarter + 1) * (BM / 4); c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(tmem_d + lane_base + c0, rr);
                tmem_ld_wait();
                if (NACC == 2 && NS > 1) {                         // (with a single stage accumulator 1 was never written)
                    uint32_t r2[32];
                    tmem_ld32(tmem_d + lane_base + BM + c0, r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) rr[i] = __float_as_uint(__uint_as_float(rr[i]) + __uint_as_float(r2[i]));
                }
                if (nrow < a.N) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int m = m0 + c0 + i;
                        if (m < a.M) {
                            if (SPLIT) {                           // K split: the reduce kernel applies alpha and mu
                                sp.part[((size_t)blockIdx.z * a.M + m) * a.N + nrow] = __uint_as_float(rr[i]);
                            } else {
                                float y = al * __uint_as_float(rr[i]);
                                if (a.mu) y += mu * p.sumx[m];
                                store_from_float(a.y, a.y_dt, (size_t)m * a.N + nrow, y);
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*s_abort) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 2) tmem_dealloc(tmem_d, 512);
}

// y = alpha * (sum of the K splits' partial sums, in split order) + mu * sum_k x.
__global__ void splitk_reduce_kernel(const float *__restrict__ part, int splits, int M, int N, const __half *__restrict__ alpha,
                                     const __half *__restrict__ mu, const float *__restrict__ sumx, void *__restrict__ y, int y_dt)
{
    // launched with programmatic stream serialisation: the blocks are resident before the split kernel has finished, and
    // wait here until all of it has completed and its partial sums are visible
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t MN = (size_t)M * N;
    if (i >= MN) return;
    const int n = (int)(i % N), m = (int)(i / N);
    float acc = 0.f;
    for (int z = 0; z < splits; ++z) acc += part[(size_t)z * MN + i];
    float v = __half2float(alpha[n]) * acc;
    if (mu) v += __half2float(mu[n]) * sumx[m];
    store_from_float(y, y_dt, i, v);
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

static encode_tiled_fn get_encode()
{
    static encode_tiled_fn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(ptr);
    }
    return fn;
}

template <int BM, int STAGES>
static int launch_cfg(const CUtensorMap &tm, const GemmParams &p, cudaStream_t s)
{
    constexpr size_t smem = (size_t)STAGES * (G_A_BYTES + BM * G_BK * 2) + 1024 + (3 * STAGES + 1) * 8 + 16;
    auto kern = gemm_tcgen05_kernel<BM, STAGES>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    dim3 grid((p.a.N + G_BN - 1) / G_BN, (p.a.M + BM - 1) / BM);
    kern<<<grid, G_THREADS, smem, s>>>(tm, p);
    return cuda_check_launch();
}

template <int BM, int STAGES, int KS, bool SPLIT, int V = 16>
static int launch_v16t(const CUtensorMap &tm, const CUtensorMap &ti, const Gemm2Params &p, const SplitArgs &sp, cudaStream_t s)
{
    const size_t smem = (size_t)STAGES * KS * (BM * G_BK * 2) + 1024 + 2 * G2_IDX_BYTES + ((p.tab_bytes + 15) & ~15) +
                        (2 * STAGES + 6) * 8 + 16;
    auto kern = gemm_v16t_kernel<BM, STAGES, KS, SPLIT, V>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    dim3 grid((p.a.N + G_BN - 1) / G_BN, (p.a.M + BM - 1) / BM, SPLIT ? (p.k_tiles + sp.split_tiles - 1) / sp.split_tiles : 1);
    kern<<<grid, G2_THREADS, smem, s>>>(tm, ti, p, sp);
    return cuda_check_launch();
}

// K splits for a launch of `tiles` CTAs over `k_tiles` k tiles: as many as keep the grid within the SM count, each a
// whole number of index tiles (16 k tiles).  Returns k tiles per split.
static int splitk_tiles(int tiles, int k_tiles, int *splits)
{
    *splits = 1;
    if (tiles > 74 || k_tiles < 64) return k_tiles;
    int want = 148 / tiles;
    if (want > 8) want = 8;
    int per = ((k_tiles + want - 1) / want + 15) / 16 * 16;
    if (per < 16) per = 16;
    const int n = (k_tiles + per - 1) / per;
    if (n < 2) return k_tiles;
    *splits = n;
    return per;
}

// Tile width in rows of x for a (M, N) problem: 128 or 256, whichever needs less time under a wave model -- CTAs run in
// rounds of one per SM, and a 256-row tile takes about 1.6 times as long as a 128-row one (it amortises the weight
// decode over twice the rows; measured at M = 2048 against M = 512).
static int gemm_bm(int M, int N)
{
    if (M <= 128) return 128;
    const long long rows = (N + 127) / 128, sms = 148;
    const long long t128 = ((M + 127) / 128) * rows, t256 = ((M + 255) / 256) * rows;
    const double c128 = (double)((t128 + sms - 1) / sms), c256 = 1.6 * (double)((t256 + sms - 1) / sms);
    return c256 < c128 ? 256 : 128;
}

size_t gemm_tcgen05_workspace_min(int M)
{
    return M > 8 ? (size_t)M * sizeof(float) : 0;   // row sums of x for the mean term
}

// 5 <= M <= 8 with few tiles and a long K (above all the 11008-wide down projection): the split tensor-core launch beats
// the fp16 decode kernel (measured 17 us against 30 us for 4096 x 11008), so the decode entry point tries it first.
bool gemm_tcgen05_small_m_pays(int M, int N, int K, int v)
{
    if (M < 5 || M > 8 || v != 16 || K % 16 || (K / v) % 8) return false;
    int splits = 1;
    const int k_tiles = (K + G_BK - 1) / G_BK;
    splitk_tiles((N + 127) / 128, k_tiles, &splits);
    return splits > 1 && (k_tiles >= 128 || (k_tiles >= 64 && M >= 6));   // (4096 x 4096 at M = 8: 10 us against 12.5 us)
}

// The minimum plus, where the launch would otherwise leave most SMs idle (v = 16, few tiles, long K), room for the
// partial sums of a K split.  With less than this (but at least the minimum) the kernels run without the split.
size_t gemm_tcgen05_workspace_bytes(int M, int N, int K, int v, int)
{
    size_t w = gemm_tcgen05_workspace_min(M);
    const bool small = gemm_tcgen05_small_m_pays(M, N, K, v);
    if (small) w = (size_t)M * sizeof(float);
    if ((M > 8 || small) && v == 16 && (K / v) % 8 == 0) {
        const int BM = gemm_bm(M, N);
        int splits = 1;
        splitk_tiles(((N + 127) / 128) * ((M + BM - 1) / BM), (K + G_BK - 1) / G_BK, &splits);
        if (splits > 1) w = ((w + 255) & ~(size_t)255) + (size_t)splits * M * N * sizeof(float);
    }
    return w;
}

int launch_gemm_tcgen05(const LinearArgs &a, cudaStream_t s, bool small_m)
{
    if (a.M <= 8 && !small_m) return BTC_ERR_UNSUPPORTED;      // the decode path is the better kernel there
    if (a.M <= 8 && (!gemm_tcgen05_small_m_pays(a.M, a.N, a.K, a.v) || !a.workspace ||
                     a.workspace_bytes < gemm_tcgen05_workspace_bytes(a.M, a.N, a.K, a.v, a.Kc)))
        return BTC_ERR_UNSUPPORTED;                            // (only with room for the K split)
    if (a.K % 8) return BTC_ERR_UNSUPPORTED;                   // TMA row pitch must be a multiple of 16 bytes
    encode_tiled_fn enc = get_encode();
    if (!enc) return BTC_ERR_UNSUPPORTED;
    const int BM = gemm_bm(a.M, a.N);

    CUtensorMap tm;
    const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
    const cuuint64_t strides[1] = {(cuuint64_t)a.K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)G_BK, (cuuint32_t)BM};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = a.x_dt == BTC_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    CUresult r = enc(&tm, dt, 2, const_cast<void *>(a.x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue);

    GemmParams p;
    p.a = a;
    p.k_tiles = (a.K + G_BK - 1) / G_BK;
    p.sumx = nullptr;
    if (a.mu) {
        if (!a.workspace || a.workspace_bytes < (size_t)a.M * sizeof(float)) return BTC_ERR_WORKSPACE;
        float *sx = reinterpret_cast<float *>(a.workspace);
        rowsum_kernel<<<(a.M + 7) / 8, 256, 0, s>>>(a.x, a.x_dt, a.M, a.K, sx);
        int rc = cuda_check_launch();
        if (rc != BTC_OK) return rc;
        p.sumx = sx;
    }
    if ((a.v == 16 && a.Kb % 8 == 0) || (a.v == 20 && a.Kb % 16 == 0)) {
        // v = 16, and v = 20 with K a multiple of 320: index tiles by TMA, table in shared memory when it fits, weights
        // through tensor memory
        CUtensorMap ti;
        const cuuint64_t idims[2] = {(cuuint64_t)a.Kb, (cuuint64_t)a.N};
        const cuuint64_t istr[1] = {(cuuint64_t)a.Kb * 2};
        const cuuint32_t ibox[2] = {64, 128};
        if (enc(&ti, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<uint16_t *>(a.idx), idims, istr, ibox, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS) {
            Gemm2Params q;
            q.a = a; q.sumx = p.sumx; q.k_tiles = p.k_tiles;
            const int Kc4 = (a.Kc + 3) / 4 * 4;
            q.tab = a.Cp + Kc4;
            // shared memory holds only x tiles (4 stages of 32 KB either way), index tiles and the table
            const size_t fixed_t = (size_t)4 * (256 * G_BK * 2) + 1024 + 2 * G2_IDX_BYTES + 512;
            q.tab_bytes = (fixed_t + (size_t)Kc4 * 4 <= 227u * 1024u) ? Kc4 * 4 : 0;
            // few tiles and a long K: split K over the idle SMs when the caller's workspace has room for the partial sums
            SplitArgs sp = {q.k_tiles, nullptr};
            int splits = 1;
            const int per = a.v == 16 ? splitk_tiles(((a.N + 127) / 128) * ((a.M + BM - 1) / BM), q.k_tiles, &splits) : q.k_tiles;
            if (a.v == 20)                                         // (no K split here: its index tiles are 20 k steps)
                return (BM == 256) ? launch_v16t<256, 4, 1, false, 20>(tm, ti, q, sp, s) : launch_v16t<128, 4, 2, false, 20>(tm, ti, q, sp, s);
            if (splits > 1) {
                const size_t off = ((size_t)a.M * sizeof(float) + 255) & ~(size_t)255;   // (row sums of x come first)
                const size_t need = off + (size_t)splits * a.M * a.N * sizeof(float);
                if (a.workspace && a.workspace_bytes >= need && reinterpret_cast<uintptr_t>(a.workspace) % 16 == 0) {
                    sp.split_tiles = per;
                    sp.part = reinterpret_cast<float *>(static_cast<char *>(a.workspace) + off);
                } else {
                    splits = 1;
                }
            }
            if (splits == 1) return (BM == 256) ? launch_v16t<256, 4, 1, false>(tm, ti, q, sp, s) : launch_v16t<128, 4, 2, false>(tm, ti, q, sp, s);
            const int rc = (BM == 256) ? launch_v16t<256, 4, 1, true>(tm, ti, q, sp, s) : launch_v16t<128, 4, 2, true>(tm, ti, q, sp, s);
            if (rc != BTC_OK) return rc;
            const size_t mn = (size_t)a.M * a.N;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)((mn + 255) / 256));
            cfg.blockDim = dim3(256);
            cfg.stream = s;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            at[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = at;
            cfg.numAttrs = 1;
            const float *part = sp.part;
            const cudaError_t e = cudaLaunchKernelEx(&cfg, splitk_reduce_kernel, part, splits, a.M, a.N, a.alpha, a.mu, q.sumx, a.y, a.y_dt);
            return e == cudaSuccess ? BTC_OK : cuda_fail(e);
        }
    }
    if (BM == 256) return launch_cfg<256, 4>(tm, p, s);
    return launch_cfg<128, 6>(tm, p, s);
}

}  // namespace btc

extern "C" BTC_API int btc_device_status_reset(void)
{
    const int zero = 0;
    cudaError_t e = cudaMemcpyToSymbol(btc::g_gemm_status, &zero, sizeof(int));
    if (e != cudaSuccess) return btc::cuda_fail(e);
    int rc = btc::index_status_reset();
    if (rc != BTC_OK) return rc;
    rc = btc::wide_status_reset();
    if (rc != BTC_OK) return rc;
    return btc::imma_status_reset();
}

extern "C" BTC_API int btc_selftest_bounded_wait(void *stream)
{
    return btc::imma_selftest_wait((cudaStream_t)stream);
}

extern "C" BTC_API int btc_device_status(int *status_host)
{
    if (!status_host) return BTC_ERR_NULL;
    int v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, btc::g_gemm_status, sizeof(int));
    if (e != cudaSuccess) return btc::cuda_fail(e);
    int v2 = 0;
    const int rc = btc::imma_status_read(&v2);
    if (rc != BTC_OK) return rc;
    int v3 = 0;
    const int rc3 = btc::index_status_read(&v3);
    if (rc3 != BTC_OK) return rc3;
    int v4 = 0;
    const int rc4 = btc::wide_status_read(&v4);
    if (rc4 != BTC_OK) return rc4;
    *status_host = v ? v : (v2 ? v2 : (v4 ? v4 : v3));
    return BTC_OK;
}

// ---------------------------------------------------------------------------------------------
// btc_linear_gemm for callers that cannot allocate: the row-sum scratch of the mean term lives in
// a fixed array of the device image instead of a caller-supplied workspace.
//
// In host code `g_static_scratch` is only a handle for the runtime, not a device address, so it
// must never be passed to a kernel as is; its address on the current device comes from
// cudaGetSymbolAddress, looked up once per device and cached.
#include <mutex>

namespace btc {

static __device__ __align__(256) unsigned char g_static_scratch[BTC_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static void *g_static_scratch_addr[MAX_DEVICES] = {};
static std::mutex g_static_scratch_mutex;

// Device address of g_static_scratch on the current device (cached per device); no allocation.
static int static_scratch_address(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= MAX_DEVICES) return BTC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        if (!p) return cuda_fail(cudaErrorInvalidSymbol);
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return BTC_OK;
}

}  // namespace btc

extern "C" BTC_API int btc_linear_gemm_static_scratch(const void *x, int x_dtype, const uint16_t *idx,
                                                      const uint32_t *C_packed, const void *alpha,
                                                      const void *mu, const btc_transform *T, void *y,
                                                      int y_dtype, int M, int N, int K, int v, int Kc,
                                                      void *stream)
{
    if (T) return BTC_ERR_UNSUPPORTED;
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || M < 1 || N < 1 || K < 1 || K % v) return BTC_ERR_SHAPE;
    if (btc::gemm_tcgen05_workspace_min(M) > (size_t)BTC_STATIC_SCRATCH_BYTES) return BTC_ERR_WORKSPACE;
    void *scratch = nullptr;
    const int rc = btc::static_scratch_address(&scratch);
    if (rc != BTC_OK) return rc;
    // Only the part the kernels cannot do without is handed on (the row sums of x), so that no launch below ever
    // takes the K split and parks partial sums of y in the shared array.
    const size_t usable = (btc::gemm_tcgen05_workspace_min(M) + 255) / 256 * 256;
    return btc_linear_gemm(x, x_dtype, idx, C_packed, alpha, mu, nullptr, y, y_dtype, M, N, K, v, Kc, scratch,
                           usable, stream);
}
