// Integer form of the decode path for M <= 2 in its one-CTA-per-SM geometry: the same arithmetic as the integer form of
// gemv_imma.cu (see the header there: mma.sync.m16n8k32 u8 x s8 over masked codeword bits and three base-256 digits of
// block-fixed-point activations; block dot <x_j, C[idx]> = 2 * sum_{bit=1} x - sum x of the paper's appendix "Binary
// codebook LUT-GEMM"), with a different work split that is the faster of the two for plain launches at M <= 2
// (uint16 index containers, dense 16-bit activations, y overwritten): measured 14.5 us against 16.5 us for the fused
// 7-layer decode step.  Everything else (M = 3..8, dense-packed indices, fp32 activations, column-range views, adding to
// y) is only in gemv_imma.cu.
//
// Why it is faster there.  A "row group" is 32 rows of one layer; a CTA (one per SM) owns a contiguous, cost-weighted
// range of row groups.  Layers wider than 256 blocks are cut into K-parts of 256 blocks; a CTA walks up to IM_RC of its
// row groups part by part.
//   warps 0..15  compute: warp w owns K-slice w % 8 of the part and tile w / 8 of the row group; the two warps of a
//                slice build its activation fragments together (half the quantisation work per warp of the two-CTA
//                geometry, where both CTAs of an SM rebuild the same slices); lane (g = lane / 4, t = lane % 4)
//                supplies two rows of the tile and 8 consecutive blocks; digit d of row m sits in column 3 m + d.
//   warp 16      producer: TMA boxes (64 blocks x 32 rows, 128-byte swizzle) of the index matrix into a shared ring,
//                bulk copy of the codeword table.
//   warps 17,18  epilogue: add the K-slices' integer digit sums in a fixed order, recombine them, add the K-parts,
//                apply alpha (and mu, both staged in shared memory once per chunk of row groups), store y -- while the
//                compute warps are already on the next row group, so a launch has no serial reduce phase.
// (Kept from the first version of the kernel: the template still carries the geometry for more rows of x, which is
// not instantiated.)  Every mbarrier wait is bounded; when one runs out the CTA raises a status word and drains.
#include <cuda.h>
#include "btc_internal.cuh"

namespace btc {
namespace wide {

constexpr int IM_CWARPS = 16;                   // compute warps
constexpr int IM_EWARPS = 2;                    // epilogue warps (four would cap the kernel at 80 registers: spills)
constexpr int IM_THREADS = (IM_CWARPS + 1 + IM_EWARPS) * 32;
constexpr int IM_STAGES = 8;                     // most index stages a launch may use (fewer when shared memory is short)
constexpr int IM_BOX_COLS = 64;                 // blocks per TMA box row: 128 bytes, the swizzle span
constexpr int IM_STAGE_BYTES = 16 * 1024;       // one iteration's indices: 4 boxes of 32 rows x 128 bytes
constexpr int IM_PW = 256;                      // blocks per K-part (16 per compute warp)
constexpr int IM_RC = 16;                       // row groups a CTA walks part by part at a time

__device__ int g_wide_status = 0;

struct ImProblem {
    const void *x;
    const uint16_t *idx;
    const uint32_t *tab;      // byte-lane codeword words [Kc]
    const uint16_t *tab16;    // the same squeezed into 16 bits (v <= 16)
    const __half *alpha;
    const __half *mu;         // may be nullptr
    void *y;
    int M, N, K, v, Kc, Kb;
    int x_dt, y_dt;
    int parts;                // ceil(Kb / IM_PW)
    int groups;               // row groups: ceil(N / (16 * TRK))
    int ncls;                 // v / 4
    int cost;                 // cost of one row group (blocks, plus the per-part fragment rebuild; see launch_gemv_imma)
    int per, rem;             // groups / cta_count and groups % cta_count
    int cta_begin, cta_count; // the CTAs that work on this layer (no CTA works on two layers: each switch would cost a
                              // table load and a fragment rebuild, and the slowest CTA sets the launch's time)
};

struct ImBatch {
    CUtensorMap map[IM_MAXP]; // idx of each layer as a 2-D tensor {K/v, N} of 16-bit words, box {64, rows}, 128-byte swizzle
    ImProblem p[IM_MAXP];
    int count;
    int tab_smem_bytes;       // bytes reserved for the codeword table (0: gather from global memory)
    int tab_head;             // entries of every table that are staged there; the rest is gathered from global memory
                              // (L1/L2): a table of 65536 codewords does not fit, and with frequency-ordered codebooks
                              // the head serves most lookups
    int stages;               // index stages in the ring (2 .. IM_STAGES)
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
// Bounded wait, called by all 32 lanes of a warp together; the answer is the same in every lane (a vote), so the
// full-mask shuffles, MMAs and __syncwarp that follow never see a split warp.  False once ~1 s has passed or the
// CTA-wide abort flag is up.  A waiting warp backs off with nanosleep so that it does not take issue slots from the
// warps it is waiting for.
__device__ __forceinline__ bool im_mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                             long long limit_clk = 2000000000LL) {
    bool ok = im_mbar_try(bar, parity);
    if (!__all_sync(0xffffffffu, ok)) {
        const long long t0 = clock64();
        int spins = 0;
        for (;;) {
            ok = im_mbar_try(bar, parity);
            if (__all_sync(0xffffffffu, ok)) break;
            __nanosleep(spins < 4 ? 20 : 100);
            if ((++spins & 255) == 0) {
                bool give_up = (*abort_flag != 0);
                if (!give_up && clock64() - t0 > limit_clk) {
                    *abort_flag = 1;
                    atomicExch(&g_wide_status, (int)BTC_ERR_TIMEOUT);
                    give_up = true;
                }
                if (__any_sync(0xffffffffu, give_up)) return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void im_bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void im_tma_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void im_mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Two 16-bit indices packed in one word -> the shared addresses base + 4 * index of both.
__device__ __forceinline__ void im_pair_addr(uint32_t pair, uint32_t base, uint32_t &lo, uint32_t &hi) {
    asm("{\n\t.reg .u16 l, h;\n\t"
        "mov.b32 {l, h}, %2;\n\t"
        "mad.wide.u16 %0, l, 4, %3;\n\t"
        "mad.wide.u16 %1, h, 4, %3;\n\t}"
        : "=r"(lo), "=r"(hi) : "r"(pair), "r"(base));
}
__device__ __forceinline__ uint32_t im_lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void im_named_bar(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
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

// Shared-memory layout (dynamic), offsets computed identically on host and device.
struct ImSmem {
    uint32_t bars;        // mbarriers: full[S], empty[S], part_full[2], part_empty[2], tab_full, tab_free
    uint32_t misc;        // abort flag, per-part scale slots
    uint32_t rowsc;       // alpha and mu of the rows of the current chunk, float [2][IM_RC * 32]
    uint32_t planes;      // per compute warp: digit planes of its K-slice of one row of x
    uint32_t tab;         // codeword table
    uint32_t ring;        // index stages
    uint32_t part;        // partial sums, two buffers: digit sums int [16 warps][16 rows][8 cols] (M <= 2), else partial dot
                          // products float [tile][16 rows][m][K-slice]
    uint32_t acc;         // dot products summed over K-parts, float [IM_RC][rows][cols / 2]
    uint32_t total;
};
constexpr int IM_NBARS = 2 * IM_STAGES + 6;
constexpr int IM_SLOTS = 4;                      // scale slots: K-parts whose partial sums may still be in flight
struct ImScale { float inv; float sx; };         // per (slot, compute warp, row m of x): 1/scale (a power of two), and
                                                 // the warp's share of sum_k x over the slice
constexpr int IM_MISC_BYTES = 16 + IM_SLOTS * IM_CWARPS * 8 * (int)sizeof(ImScale) + IM_CWARPS * 4;
constexpr int IM_PLANE_WORDS = 3 * (IM_PW + 64) * 5;   // all K-slices: 3 digits x (256 blocks + skew) x (v / 4 <= 5) words

__host__ __device__ inline ImSmem im_smem_layout(int tab_bytes, int cols, int rows, int stages)
{
    ImSmem L;
    uint32_t o = 0;
    L.bars = o; o += IM_NBARS * 8;
    o = (o + 15u) & ~15u;
    L.misc = o; o += IM_MISC_BYTES;
    o = (o + 15u) & ~15u;
    L.rowsc = o; o += 2u * IM_RC * 32u * 4u;
    L.planes = o; o += IM_PLANE_WORDS * 4;
    o = (o + 127u) & ~127u;
    L.tab = o; o += (uint32_t)tab_bytes;
    o = (o + 1023u) & ~1023u;                     // swizzled TMA boxes want 1024-byte alignment
    L.ring = o; o += (uint32_t)stages * IM_STAGE_BYTES;
    // cols == 8 (M <= 2): a 16 x 8 tile of digit sums per compute warp; else one float per (warp, row, m)
    L.part = o; o += 2u * IM_CWARPS * 16u * (uint32_t)(cols == 8 ? 8 : (cols == 16 ? 5 : 8)) * 4u;
    L.acc = o; o += (uint32_t)IM_RC * (uint32_t)rows * (uint32_t)(cols / 2) * 4u;
    L.total = o;
    return L;
}

// Row groups [lo, hi) of layer P that fall to CTA b: the layer's cta_count CTAs split its row groups evenly (the first
// `rem` of them take one more); per and rem come from the host, so no division runs here.
__device__ __forceinline__ void im_group_range(const ImProblem &P, int b, int &lo, int &hi)
{
    lo = hi = 0;
    const int r = b - P.cta_begin;
    if (r < 0 || r >= P.cta_count) return;
    lo = r * P.per + min(r, P.rem);
    hi = lo + P.per + (r < P.rem ? 1 : 0);
}

// TAB_MODE 0: tables gathered from global memory; 1: whole tables in shared memory; 2: the first tab_head entries in
// shared memory, the rest from global memory; 3: whole tables in shared memory as 16-bit halves (v <= 16; a table of
// 65536 codewords then takes 128 KB), widened by `h | (h << 12)` after the gather.
template <int NCLS, int NM, int TAB_MODE>
__global__ void __launch_bounds__(IM_THREADS, 1)
gemv_imma_kernel(const __grid_constant__ ImBatch batch)
{
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int TRK = (NM == 1) ? 2 : 1;               // 16-row tiles per row group
    constexpr int ROWS = TRK * 16;
    constexpr int COLS = 8 * NM;
    constexpr int KS = 16 / TRK;                         // K-slices of a part; warp w: slice w % KS, tile w / KS
    constexpr int SLICE = IM_PW / KS;                    // blocks per slice
    constexpr int BPL = SLICE / 4;                       // blocks per lane
    constexpr int MAXM = (NM == 1) ? 2 : (NM == 2 ? 5 : 8);
    const ImSmem L = im_smem_layout(batch.tab_smem_bytes, COLS, ROWS, batch.stages);
    const int NST = batch.stages;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + L.misc);
    ImScale *s_scale = reinterpret_cast<ImScale *>(smem + L.misc + 16);           // [IM_SLOTS][16 warps][8]
    float *s_xmax = reinterpret_cast<float *>(smem + L.misc + 16 + IM_SLOTS * IM_CWARPS * 8 * sizeof(ImScale));   // [16 warps]
    uint32_t *s_planes = reinterpret_cast<uint32_t *>(smem + L.planes);
    uint32_t *s_tab = reinterpret_cast<uint32_t *>(smem + L.tab);
    unsigned char *s_ring = smem + L.ring;
    // Who recombines the three digit sums of a (K-slice, row, m): with M <= 2 the compute warps set the pace, so they
    // hand over their raw 16 x 8 integer tiles and the epilogue warps recombine; with more rows of x the epilogue
    // would fall behind, so each compute warp recombines its own sums and hands over one float per (row, m).
    constexpr bool FPART = (NM > 1);
    constexpr int TILE_INTS = 16 * COLS;                 // one compute warp's integer tile
    float *s_part = reinterpret_cast<float *>(smem + L.part);
    int *s_parti = reinterpret_cast<int *>(smem + L.part);
    float *s_acc = reinterpret_cast<float *>(smem + L.acc);
    float *s_alpha = reinterpret_cast<float *>(smem + L.rowsc), *s_mu = s_alpha + IM_RC * 32;
    constexpr int ACC_M = COLS / 2;                      // floats per row of s_acc (>= MAXM)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto bar_full = [&](int s) { return im_smem_u32(bars + s); };
    auto bar_empty = [&](int s) { return im_smem_u32(bars + IM_STAGES + s); };
    auto bar_pfull = [&](int b) { return im_smem_u32(bars + 2 * IM_STAGES + b); };
    auto bar_pempty = [&](int b) { return im_smem_u32(bars + 2 * IM_STAGES + 2 + b); };
    const uint32_t bar_tabfull = im_smem_u32(bars + 2 * IM_STAGES + 4);
    const uint32_t bar_tabfree = im_smem_u32(bars + 2 * IM_STAGES + 5);

    if (tid == 0) {
        for (int s = 0; s < NST; ++s) { im_mbar_init(bar_full(s), 1); im_mbar_init(bar_empty(s), IM_CWARPS); }
        for (int b = 0; b < 2; ++b) { im_mbar_init(bar_pfull(b), IM_CWARPS); im_mbar_init(bar_pempty(b), IM_EWARPS); }
        im_mbar_init(bar_tabfull, 1);
        im_mbar_init(bar_tabfree, IM_CWARPS);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr bool tab_smem = TAB_MODE != 0;             // (part of) the codeword table is staged in shared memory
    const uint32_t tab_head = (uint32_t)batch.tab_head;

    // All three roles walk the same sequence: layers pi (those with row groups for this CTA, counted
    // by ps), chunks [c0, c1) of at most IM_RC row groups, K-parts j (counted by pc), row groups r; li
    // counts iterations.
    if (warp == IM_CWARPS) {
        // ============================================================ producer
        int li = 0, ps = 0;
        int s = 0;                                             // ring stage li % NST; rph = (li / NST) & 1
        uint32_t rph = 0;
        bool ok = true;
        for (int pi = 0; pi < batch.count && ok; ++pi) {
            const ImProblem &P = batch.p[pi];
            int glo, ghi;
            im_group_range(P, (int)blockIdx.x, glo, ghi);
            if (glo >= ghi) continue;
            if (tab_smem) {
                if (ps > 0 && !im_mbar_wait(bar_tabfree, (ps - 1) & 1, s_abort)) break;
                if (lane == 0) {
                    const uint32_t bytes = TAB_MODE == 3 ? (uint32_t)((P.Kc + 7) / 8 * 8 * 2)
                                                         : (uint32_t)(min((P.Kc + 3) / 4 * 4, batch.tab_head) * 4);
                    im_mbar_expect_tx(bar_tabfull, bytes);
                    im_bulk_g2s(im_smem_u32(s_tab), TAB_MODE == 3 ? static_cast<const void *>(P.tab16) : static_cast<const void *>(P.tab),
                                bytes, bar_tabfull);
                }
            }
            ++ps;
            for (int c0 = glo; c0 < ghi && ok; c0 += IM_RC) {
                const int c1 = min(c0 + IM_RC, ghi);
                for (int j = 0; j < P.parts && ok; ++j) {
                    const int pw = min(IM_PW, P.Kb - j * IM_PW);          // blocks of this part
                    for (int r = c0; r < c1; ++r, ++li) {
                        if (li >= NST && !im_mbar_wait(bar_empty(s), rph ^ 1u, s_abort)) { ok = false; break; }
                        // boxes of 64 blocks x ROWS rows; rows past N and blocks past K/v arrive as zeros
                        const int nbox = (pw + IM_BOX_COLS - 1) / IM_BOX_COLS;
                        constexpr uint32_t BOX_BYTES = ROWS * 128;
                        if (lane == 0) im_mbar_expect_tx(bar_full(s), (uint32_t)nbox * BOX_BYTES);
                        __syncwarp();
                        if (lane < nbox)
                            im_tma_2d(im_smem_u32(s_ring + (size_t)s * IM_STAGE_BYTES + (size_t)lane * BOX_BYTES), &batch.map[pi],
                                      j * IM_PW + lane * IM_BOX_COLS, r * ROWS, bar_full(s));
                        if (++s == NST) { s = 0; rph ^= 1u; }
                    }
                }
            }
        }
    } else if (warp > IM_CWARPS) {
        // ============================================================ epilogue (two warps)
        // 64 threads = ROWS rows x SPLIT groups of compute warps; the groups of a row sit in adjacent lanes.
        constexpr int SPLIT = (IM_EWARPS * 32) / ROWS;         // 2 or 4
        constexpr int WPG = KS / SPLIT;                        // compute warps (K-slices) per group: 4
        const int et = (warp - IM_CWARPS - 1) * 32 + lane;
        const int R = et / SPLIT, grp = et % SPLIT;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        int li = 0, pc = 0;
        bool ok = true;
        for (int pi = 0; pi < batch.count && ok; ++pi) {
            const ImProblem &P = batch.p[pi];
            int glo, ghi;
            im_group_range(P, (int)blockIdx.x, glo, ghi);
            if (glo >= ghi) continue;
            const float unshift2 = 2.0f / (float)(1 << (P.ncls - 1));
            for (int c0 = glo; c0 < ghi && ok; c0 += IM_RC) {
                const int c1 = min(c0 + IM_RC, ghi);
                float sxtot[MAXM];                               // sum_k x[m, k] over the parts seen so far
#pragma unroll
                for (int m = 0; m < MAXM; ++m) sxtot[m] = 0.f;
                // alpha / mu of this thread's row in every row group of the chunk go to shared memory once per chunk (each
                // thread reads back only what it wrote, so no barrier is needed): the loads, a trip to DRAM, overlap the
                // compute warps' fragment build instead of sitting in every iteration's chain
                if (grp == 0) {
                    unsigned short ab[IM_RC], mb[IM_RC];
#pragma unroll
                    for (int i = 0; i < IM_RC; ++i) {                // all loads in flight together
                        const int n = (c0 + i) * ROWS + R;
                        ab[i] = 0; mb[i] = 0;
                        if (i < c1 - c0 && n < P.N) {
                            ab[i] = __ldg(reinterpret_cast<const unsigned short *>(P.alpha) + n);
                            if (P.mu) mb[i] = __ldg(reinterpret_cast<const unsigned short *>(P.mu) + n);
                        }
                    }
#pragma unroll
                    for (int i = 0; i < IM_RC; ++i) {
                        s_alpha[i * ROWS + R] = __half2float(__ushort_as_half(ab[i]));
                        s_mu[i * ROWS + R] = __half2float(__ushort_as_half(mb[i]));
                    }
                }
                for (int j = 0; j < P.parts && ok; ++j, ++pc) {
                    const bool last = (j == P.parts - 1);
                    const ImScale *sc = s_scale + (size_t)(pc % IM_SLOTS) * IM_CWARPS * 8;
                    float sxp[MAXM];                             // sum_k x[m, k] over this part (fixed order of warps)
#pragma unroll
                    for (int m = 0; m < MAXM; ++m) sxp[m] = 0.f;
                    for (int r = c0; r < c1; ++r, ++li) {
                        const int buf = li & 1;
                        const int n = r * ROWS + R;
                        const bool live = (n < P.N) && (grp == 0);
                        if (!im_mbar_wait(bar_pfull(buf), (li >> 1) & 1, s_abort)) { ok = false; break; }
                        const float al = s_alpha[(r - c0) * ROWS + R], mu = s_mu[(r - c0) * ROWS + R];
                        if (r == c0) {
#pragma unroll
                            for (int m = 0; m < MAXM; ++m)
                                if (m < P.M)
                                    for (int w = 0; w < IM_CWARPS; ++w) sxp[m] += sc[w * 8 + m].sx;
#pragma unroll
                            for (int m = 0; m < MAXM; ++m) sxtot[m] += sxp[m];
                        }
                        float *accrow = s_acc + ((size_t)(P.parts > 1 ? (r - c0) : 0) * ROWS + R) * ACC_M;
                        float dots[MAXM];
                        if constexpr (FPART) {
                            // row R lies in tile R / 16; its K-slices' partial dot products sit side by side
                            const float *base = s_part + ((((size_t)buf * TRK + (R >> 4)) * 16 + (R & 15)) * MAXM) * KS + grp * WPG;
#pragma unroll
                            for (int m = 0; m < MAXM; ++m) {
                                dots[m] = 0.f;
                                if (m < P.M) {
                                    const float4 q = *reinterpret_cast<const float4 *>(base + m * KS);
                                    dots[m] = ((q.x + q.y) + q.z) + q.w;
                                }
                            }
                        } else {
                            // row R lies in tile R / 16, written by the compute warps (R / 16) * KS + slice
                            const int *base = s_parti + ((size_t)buf * IM_CWARPS + (R >> 4) * KS + grp * WPG) * TILE_INTS + (size_t)(R & 15) * COLS;
#pragma unroll
                            for (int m = 0; m < MAXM; ++m) dots[m] = 0.f;
#pragma unroll
                            for (int w = 0; w < WPG; ++w) {
                                int pv[COLS];
#pragma unroll
                                for (int c4 = 0; c4 < COLS / 4; ++c4) {
                                    if (c4 * 4 < 3 * P.M) {                 // columns 3 m + d, m < M
                                        const int4 q = *reinterpret_cast<const int4 *>(base + (size_t)w * TILE_INTS + c4 * 4);
                                        pv[c4 * 4] = q.x; pv[c4 * 4 + 1] = q.y; pv[c4 * 4 + 2] = q.z; pv[c4 * 4 + 3] = q.w;
                                    } else {
                                        pv[c4 * 4] = pv[c4 * 4 + 1] = pv[c4 * 4 + 2] = pv[c4 * 4 + 3] = 0;
                                    }
                                }
#pragma unroll
                                for (int m = 0; m < MAXM; ++m) {
                                    if (m < P.M) {
                                        // each digit sum is below 2^24 in magnitude, so the conversions are exact
                                        const float T = ((float)pv[3 * m + 2] * 256.0f + (float)pv[3 * m + 1]) * 256.0f + (float)pv[3 * m];
                                        dots[m] += T * sc[(grp * WPG + w) * 8 + m].inv;
                                    }
                                }
                            }
                        }
                        __syncwarp();
                        if (lane == 0) im_mbar_arrive(bar_pempty(buf));
#pragma unroll
                        for (int m = 0; m < MAXM; ++m) {
                            if (m < P.M) {
#pragma unroll
                                for (int o = 1; o < SPLIT; o <<= 1) dots[m] += __shfl_xor_sync(0xffffffffu, dots[m], o);
                                float dot = dots[m] * unshift2 - sxp[m];        // 2 * sum_{bit=1} x - sum x over this part
                                if (grp == 0) {
                                    if (j > 0) dot += accrow[m];
                                    if (!last) accrow[m] = dot;
                                }
                                if (last && live) {
                                    const float yv = al * dot + mu * sxtot[m];
                                    store_from_float(P.y, P.y_dt, (size_t)m * P.N + n, yv);
                                }
                            }
                        }
                    }
                }
            }
        }
    } else {
        // ============================================================ compute warps
        const int g = lane >> 2, t = lane & 3;
        constexpr float MAGIC = 12582912.0f;                   // 1.5 * 2^23: float -> int by addition
        constexpr int MAGIC_BITS = 0x4B400000;
        const int ks = warp % KS, rh = warp / KS;             // K-slice and tile of this warp
        // MMA row g (and g + 8) carries tile row sg (and sg + 8): neighbouring g differ in bit 2 of the row, so the
        // eight lanes of a shared-memory phase read distinct swizzled chunks
        const int sg = ((g & 1) << 2) | (g >> 1);
        // digit planes of a slice: block b, class c of digit d at word d * PSW + (b + b / BPL) * NCLS + c; the skew
        // puts the lanes of a fragment read (t: blocks BPL apart, d: planes) on different banks
        constexpr int PSW = (SLICE + 4) * NCLS;
        uint32_t *planes = s_planes + ks * (3 * PSW);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        int li = 0, ps = 0, pc = 0;
        int s = 0;                                             // ring stage li % NST; rph = (li / NST) & 1
        uint32_t rph = 0;
        bool ok = true;
        for (int pi = 0; pi < batch.count && ok; ++pi) {
            const ImProblem &P = batch.p[pi];
            int glo, ghi;
            im_group_range(P, (int)blockIdx.x, glo, ghi);
            if (glo >= ghi) continue;
            const int M = P.M, K = P.K, Kb = P.Kb, v = P.v;
            const int cmax = P.ncls - 1;
            const int PBITS = 22 - cmax;                       // |X| <= 2^PBITS
            const int ngroups = SLICE * v / 8;                 // groups of 8 activations in a slice (<= 80)
            bool tab_ready = !tab_smem;
            const uint32_t *gtab = P.tab;                      // (s_tab is named directly below so that its loads are shared-memory loads)

            for (int c0 = glo; c0 < ghi && ok; c0 += IM_RC) {
                const int c1 = min(c0 + IM_RC, ghi);
                for (int j = 0; j < P.parts && ok; ++j, ++pc) {
                    const int pw = min(IM_PW, Kb - j * IM_PW);
                    const int jb0 = j * IM_PW + ks * SLICE;         // first block of this warp's slice
                    const bool wvalid = ks * SLICE + BPL * t < pw;  // this lane's blocks exist (pw % 8 == 0)
                    const int kend = (j * IM_PW + pw) * v;          // end of the part in x
                    // byte offset of this lane's index chunk inside a stage (128-byte swizzle: 16-byte chunk c of row q
                    // sits at chunk c ^ (q & 7)); rows sg and sg + 8 of tile rh
                    const int boff = (ks * SLICE + BPL * t) * 2;
                    const int irow = rh * 16 + sg;
                    const uint32_t idx_off = (uint32_t)(boff >> 7) * (ROWS * 128) + (uint32_t)irow * 128
                                             + ((((boff >> 4) & 7) ^ (irow & 7)) << 4) + (boff & 15);
                    ImScale *scale_out = s_scale + ((size_t)(pc % IM_SLOTS) * IM_CWARPS + warp) * 8;

                    // ---- B fragments for this part.  The warp's slice of each row of x (16 blocks) is
                    //      quantised with its own scale: X = rint(x * 2^(PBITS - e)), 2^e > max |x| of the slice.
                    uint32_t breg[BPL][NCLS][NM];
#pragma unroll
                    for (int e = 0; e < BPL; ++e)
#pragma unroll
                        for (int c = 0; c < NCLS; ++c)
#pragma unroll
                            for (int nm = 0; nm < NM; ++nm) breg[e][c][nm] = 0u;
                    // The TRK warps of a slice share its planes: each quantises every TRK-th group of 8 activations.
                    constexpr int NU = (SLICE * 20 / 8 + 32 * TRK - 1) / (32 * TRK);   // groups per lane (v <= 20)
                    auto slice_sync = [&]() {
                        if (TRK == 1) __syncwarp();
                        else im_named_bar(1 + ks, TRK * 32);
                    };
                    for (int m = 0; m < M; ++m) {
                        const uint16_t *xrow = reinterpret_cast<const uint16_t *>(P.x) + (size_t)m * K;
                        uint4 q4[NU];
                        float amax = 0.f;
#pragma unroll
                        for (int u = 0; u < NU; ++u) {
                            const int gi = lane + 32 * (rh + TRK * u);
                            const int k0 = jb0 * v + 8 * gi;
                            q4[u] = make_uint4(0u, 0u, 0u, 0u);
                            if (gi < ngroups && k0 < kend) q4[u] = __ldg(reinterpret_cast<const uint4 *>(xrow + k0));
                            const uint32_t wds[4] = {q4[u].x, q4[u].y, q4[u].z, q4[u].w};
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj) {
                                float lo, hi;
                                im_unpack2(wds[jj], P.x_dt, lo, hi);
                                amax = fmaxf(amax, fmaxf(fabsf(lo), fabsf(hi)));
                            }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                        if (TRK > 1) {
                            if (lane == 0) s_xmax[warp] = amax;
                            slice_sync();
                            amax = fmaxf(s_xmax[ks], s_xmax[ks + KS]);
                        }
                        // amax = f * 2^e with f in [1, 2) (a float from fp16 / bf16 is normal or zero): |x| < 2^(e+1)
                        const int ex = max((int)((__float_as_uint(amax) >> 23) & 0xffu) - 127 + 1, -100);   // (clamped: bf16 can be tinier)
                        const float sc = (amax > 0.f) ? __uint_as_float((uint32_t)(127 + PBITS - ex) << 23) : 1.0f;
                        const float inv = (amax > 0.f) ? __uint_as_float((uint32_t)(127 - PBITS + ex) << 23) : 1.0f;
                        int xs = 0;
#pragma unroll
                        for (int u = 0; u < NU; ++u) {
                            const int gi = lane + 32 * (rh + TRK * u);
                            if (gi < ngroups) {
                                const uint32_t wds[4] = {q4[u].x, q4[u].y, q4[u].z, q4[u].w};
                                int blk = (8 * gi) / v;                  // block of the group's first activation in the slice
                                int cpos = 8 * gi - blk * v;             // and its position in that block
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const int c = cpos >> 2;
                                    const int wi = (blk + blk / BPL) * NCLS + c;
                                    cpos += 4;
                                    if (cpos >= v) { cpos -= v; ++blk; }
                                    const uint32_t sh = 1u << (cmax - c);
                                    const uint32_t off = 0x8080u - (uint32_t)MAGIC_BITS * sh;    // arithmetic modulo 2^32
                                    float f0, f1, f2, f3;
                                    im_unpack2(wds[2 * h], P.x_dt, f0, f1);
                                    im_unpack2(wds[2 * h + 1], P.x_dt, f2, f3);
                                    const uint32_t b0 = (uint32_t)__float_as_int(f0 * sc + MAGIC), b1 = (uint32_t)__float_as_int(f1 * sc + MAGIC);
                                    const uint32_t b2 = (uint32_t)__float_as_int(f2 * sc + MAGIC), b3 = (uint32_t)__float_as_int(f3 * sc + MAGIC);
                                    xs += (int)(b0 + b1 + b2 + b3 - 4u * (uint32_t)MAGIC_BITS);
                                    // Y = X * 2^(cmax - c) + 0x8080: byte d of Y is balanced digit d of X * 2^(cmax-c), + 0x80 for d < 2
                                    const uint32_t y0 = b0 * sh + off, y1 = b1 * sh + off, y2 = b2 * sh + off, y3 = b3 * sh + off;
#pragma unroll
                                    for (int d = 0; d < 3; ++d) {
                                        const uint32_t sel = (uint32_t)d | ((uint32_t)(4 + d) << 4);
                                        const uint32_t lo2 = __byte_perm(y0, y1, sel), hi2 = __byte_perm(y2, y3, sel);
                                        planes[d * PSW + wi] = __byte_perm(lo2, hi2, 0x5410) ^ (d < 2 ? 0x80808080u : 0u);
                                    }
                                }
                            }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) xs += __shfl_xor_sync(0xffffffffu, xs, o);
                        if (lane == 0) {
                            ImScale o2;
                            o2.inv = inv;
                            o2.sx = (float)xs * inv;                     // this warp's share of sum_k x over the slice
                            scale_out[m] = o2;
                        }
                        slice_sync();
#pragma unroll
                        for (int nm = 0; nm < NM; ++nm) {
                            const int col = g + 8 * nm;
                            const int mc = col / 3, d = col - 3 * mc;
                            if (mc == m && wvalid) {
                                const uint32_t *src = planes + d * PSW + (BPL * t + t) * NCLS;
#pragma unroll
                                for (int e = 0; e < BPL; ++e) {
                                    if (NCLS == 4) {
                                        const uint4 q = *reinterpret_cast<const uint4 *>(src + e * 4);
                                        breg[e][0][nm] = q.x; breg[e][1][nm] = q.y; breg[e][2][nm] = q.z; breg[e][NCLS - 1][nm] = q.w;
                                    } else {
#pragma unroll
                                        for (int c = 0; c < NCLS; ++c) breg[e][c][nm] = src[e * NCLS + c];
                                    }
                                }
                            }
                        }
                        slice_sync();
                    }
                    if (!tab_ready) {
                        if (!im_mbar_wait(bar_tabfull, ps & 1, s_abort)) { ok = false; break; }
                        tab_ready = true;
                    }

                    // ---- the row groups of the chunk, for this part
                    // Loads this lane's indices of the next row group from the ring (tile rows sg and sg + 8 of tile rh;
                    // 128-byte swizzle: 16-byte chunk c of row q sits at chunk c ^ (q & 7)) and frees the stage.
                    uint32_t ia[BPL / 2], ib[BPL / 2];
                    auto load_indices = [&]() -> bool {
                        if (!im_mbar_wait(bar_full(s), rph, s_abort)) return false;
                        const unsigned char *stage = s_ring + (size_t)s * IM_STAGE_BYTES;
#pragma unroll
                        for (int i = 0; i < BPL / 2; ++i) { ia[i] = 0u; ib[i] = 0u; }
                        if (wvalid) {
                            const unsigned char *pa = stage + idx_off;
                            const unsigned char *pb = pa + 8 * 128;                 // row + 8: same row & 7
                            if (BPL == 8) {
                                const uint4 qa = *reinterpret_cast<const uint4 *>(pa), qb = *reinterpret_cast<const uint4 *>(pb);
                                ia[0] = qa.x; ia[1] = qa.y; ia[BPL / 2 - 2] = qa.z; ia[BPL / 2 - 1] = qa.w;
                                ib[0] = qb.x; ib[1] = qb.y; ib[BPL / 2 - 2] = qb.z; ib[BPL / 2 - 1] = qb.w;
                            } else {
                                const uint2 qa = *reinterpret_cast<const uint2 *>(pa), qb = *reinterpret_cast<const uint2 *>(pb);
                                ia[0] = qa.x; ia[1] = qa.y;
                                ib[0] = qb.x; ib[1] = qb.y;
                            }
                        }
                        // the index loads must have RETURNED before the stage is handed back: the arrive does not wait for
                        // loads in flight, and the producer's next copy into this stage can land within a few hundred clocks
#pragma unroll
                        for (int i = 0; i < BPL / 2; ++i) asm volatile("" :: "r"(ia[i]), "r"(ib[i]) : "memory");
                        __syncwarp();
                        if (lane == 0) im_mbar_arrive(bar_empty(s));
                        if (++s == NST) { s = 0; rph ^= 1u; }
                        return true;
                    };
                    if (!load_indices()) { ok = false; break; }
                    for (int r = c0; r < c1; ++r, ++li) {
                        constexpr int CH = 2;        // accumulation chains: an MMA need not wait for the previous one
                        int accs[CH][NM][4];
                        int (&acc)[NM][4] = accs[0];
#pragma unroll
                        for (int nm = 0; nm < NM; ++nm)
#pragma unroll
                            for (int i = 0; i < 4; ++i)
#pragma unroll
                                for (int ch = 0; ch < CH; ++ch) accs[ch][nm][i] = 0;
                        if (ks * SLICE < pw) {                      // warp-uniform: the slice is not empty
#pragma unroll
                            for (int e4 = 0; e4 < BPL; e4 += 4) {
                                uint32_t w0[4], w1[4];
                                if (TAB_MODE == 1) {
                                    // whole table in shared memory: one multiply-add per index gives its address
                                    const uint32_t tb = im_smem_u32(s_tab);
#pragma unroll
                                    for (int ep = 0; ep < 2; ++ep) {
                                        uint32_t a0, a1, b0, b1;
                                        im_pair_addr(ia[(e4 >> 1) + ep], tb, a0, a1);
                                        im_pair_addr(ib[(e4 >> 1) + ep], tb, b0, b1);
                                        w0[2 * ep] = im_lds32(a0); w0[2 * ep + 1] = im_lds32(a1);
                                        w1[2 * ep] = im_lds32(b0); w1[2 * ep + 1] = im_lds32(b1);
                                    }
                                } else {
#pragma unroll
                                    for (int e = 0; e < 4; ++e) {
                                        const uint32_t pa = ia[(e4 + e) >> 1], pb = ib[(e4 + e) >> 1];
                                        const uint32_t i0 = (e & 1) ? (pa >> 16) : (pa & 0xffffu);
                                        const uint32_t i1 = (e & 1) ? (pb >> 16) : (pb & 0xffffu);
                                        if (TAB_MODE == 3) {
                                            const uint32_t h0 = reinterpret_cast<const uint16_t *>(s_tab)[i0];
                                            const uint32_t h1 = reinterpret_cast<const uint16_t *>(s_tab)[i1];
                                            w0[e] = h0 | (h0 << 12); w1[e] = h1 | (h1 << 12);
                                        }
                                        else if (TAB_MODE == 0) { w0[e] = __ldg(gtab + i0); w1[e] = __ldg(gtab + i1); }
                                        else {
                                            w0[e] = i0 < tab_head ? s_tab[i0] : __ldg(gtab + i0);
                                            w1[e] = i1 < tab_head ? s_tab[i1] : __ldg(gtab + i1);
                                        }
                                    }
                                }
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
#pragma unroll
                                    for (int cp = 0; cp < NCLS / 2; ++cp) {
                                        const uint32_t ma = 0x01010101u << (2 * cp), mb = 0x01010101u << (2 * cp + 1);
#pragma unroll
                                        for (int nm = 0; nm < NM; ++nm)
                                            im_mma_u8s8(accs[((e & 1) * 2 + (cp & 1)) % CH][nm], w0[e] & ma, w1[e] & ma, w0[e] & mb, w1[e] & mb,
                                                        breg[e4 + e][2 * cp][nm], breg[e4 + e][2 * cp + 1][nm]);
                                    }
                                }
                                if (NCLS & 1) {
                                    const uint32_t ml = 0x01010101u << (NCLS - 1);
#pragma unroll
                                    for (int ep = 0; ep < 2; ++ep)
#pragma unroll
                                        for (int nm = 0; nm < NM; ++nm)
                                            im_mma_u8s8(acc[nm], w0[2 * ep] & ml, w1[2 * ep] & ml, w0[2 * ep + 1] & ml,
                                                        w1[2 * ep + 1] & ml, breg[e4 + 2 * ep][NCLS - 1][nm], breg[e4 + 2 * ep + 1][NCLS - 1][nm]);
                                }
                            }
                        }
                        // the next row group's indices are fetched while this one's MMAs drain (their codewords are in
                        // registers by now), so the barrier round trip is off the critical path
                        if (r + 1 < c1 && !load_indices()) { ok = false; break; }
                        // likewise the wait for the partial-sum buffer: its round trip overlaps the MMAs' drain
                        const int buf = li & 1;
                        if (li >= 2 && !im_mbar_wait(bar_pempty(buf), ((li >> 1) & 1) ^ 1, s_abort)) { ok = false; break; }
#pragma unroll
                        for (int nm = 0; nm < NM; ++nm)
#pragma unroll
                            for (int i = 0; i < 4; ++i)
#pragma unroll
                                for (int ch = 1; ch < CH; ++ch) acc[nm][i] += accs[ch][nm][i];
                        if constexpr (FPART) {
                            // The three digit sums of (row, m) sit in columns 3 m .. 3 m + 2, spread over the lanes of a quad:
                            // they are brought together by shuffles, recombined (each is below 2^24 in magnitude, so the
                            // conversions are exact), scaled by the slice's 2^-s and stored as one float per (row, m).
                            float *mine = s_part + (((size_t)buf * TRK + rh) * 16) * MAXM * KS + ks;
#pragma unroll
                            for (int m = 0; m < MAXM; ++m) {
                                if (m < M) {                                // warp-uniform
                                    int dlo[3], dhi[3];
#pragma unroll
                                    for (int d = 0; d < 3; ++d) {
                                        const int col = 3 * m + d;          // a constant once unrolled
                                        const int src = (lane & ~3) | ((col & 7) >> 1);
                                        dlo[d] = __shfl_sync(0xffffffffu, acc[col >> 3][col & 1], src);
                                        dhi[d] = __shfl_sync(0xffffffffu, acc[col >> 3][2 + (col & 1)], src);
                                    }
                                    if (t == (m & 3)) {
                                        const float inv = scale_out[m].inv;
                                        const float Tlo = ((float)dlo[2] * 256.0f + (float)dlo[1]) * 256.0f + (float)dlo[0];
                                        const float Thi = ((float)dhi[2] * 256.0f + (float)dhi[1]) * 256.0f + (float)dhi[0];
                                        mine[(sg * MAXM + m) * KS] = Tlo * inv;
                                        mine[((sg + 8) * MAXM + m) * KS] = Thi * inv;
                                    }
                                }
                            }
                        } else {
                            int *mine = s_parti + ((size_t)buf * IM_CWARPS + warp) * TILE_INTS;
                            if (2 * t < 3 * M) {                        // columns 3 m + d, m < M: the others are never read
                                *reinterpret_cast<int2 *>(mine + sg * COLS + 2 * t) = make_int2(acc[0][0], acc[0][1]);
                                *reinterpret_cast<int2 *>(mine + (sg + 8) * COLS + 2 * t) = make_int2(acc[0][2], acc[0][3]);
                            }
                        }
                        __syncwarp();
                        if (lane == 0) im_mbar_arrive(bar_pfull(buf));
                    }
                }
            }
            ++ps;
            if (tab_smem && ok) {
                __syncwarp();
                if (lane == 0) im_mbar_arrive(bar_tabfree);
            }
        }
    }
    // A CTA that gave up on a wait may still have copies in flight into its shared memory: let them land before it goes.
    if (*s_abort) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000LL) __nanosleep(1000);
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*im_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static im_encode_fn im_get_encode()
{
    static im_encode_fn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<im_encode_fn>(ptr);
    }
    return fn;
}

// Tensor map of an index matrix {K/v, N} (16-bit words), box {64, rows}, 128-byte swizzle.  Encoding goes through the
// driver and costs about a microsecond; a decode step re-uses the same matrices call after call, so the last few
// maps are kept per host thread, keyed by everything the encoding depends on.
static bool im_tensor_map(im_encode_fn enc, const uint16_t *idx, int Kb, int N, int rows, CUtensorMap *out)
{
    struct Entry { const uint16_t *idx; int Kb, N, rows; CUtensorMap map; };
    constexpr int SLOTS = 64;
    thread_local Entry cache[SLOTS];
    thread_local int used = 0, next = 0;
    for (int i = 0; i < used; ++i)
        if (cache[i].idx == idx && cache[i].Kb == Kb && cache[i].N == N && cache[i].rows == rows) { *out = cache[i].map; return true; }
    const cuuint64_t dims[2] = {(cuuint64_t)Kb, (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)Kb * 2};
    const cuuint32_t box[2] = {(cuuint32_t)IM_BOX_COLS, (cuuint32_t)rows};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap m;
    if (enc(&m, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<uint16_t *>(idx), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    Entry &e = cache[next];
    e.idx = idx; e.Kb = Kb; e.N = N; e.rows = rows; e.map = m;
    next = (next + 1) % SLOTS;
    if (used < SLOTS) ++used;
    *out = m;
    return true;
}

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

// Gives every layer a whole number of CTAs so that the largest load of any CTA -- ceil(groups / CTAs) row groups times
// the layer's cost per row group; row groups are not divisible -- is as small as the budget allows, and returns the
// grid size.  Smallest feasible load by bisection; a load T needs ceil(groups / floor(T / cost)) CTAs of a layer.
static int im_assign_ctas(ImBatch &b, int budget)
{
    auto ctas_needed = [&](long long T) {
        long long sum = 0;
        for (int i = 0; i < b.count; ++i) {
            const long long per = T / b.p[i].cost;                    // row groups one CTA may take
            if (per < 1) return (long long)1 << 40;
            sum += (b.p[i].groups + per - 1) / per;
        }
        return sum;
    };
    long long lo = 1, hi = 0;
    for (int i = 0; i < b.count; ++i) {
        const long long all = (long long)b.p[i].groups * b.p[i].cost;
        if (all > hi) hi = all;                                       // one CTA per layer always fits (budget >= count)
    }
    while (lo < hi) {
        const long long mid = (lo + hi) / 2;
        if (ctas_needed(mid) <= budget) hi = mid; else lo = mid + 1;
    }
    int sum = 0;
    for (int i = 0; i < b.count; ++i) {
        const long long per = lo / b.p[i].cost;
        b.p[i].cta_count = (int)((b.p[i].groups + per - 1) / per);
        sum += b.p[i].cta_count;
    }
    while (sum < budget) {                          // spare CTAs: more SMs streaming, where the average load is highest
        int best = -1;
        for (int i = 0; i < b.count; ++i)
            if (b.p[i].cta_count < b.p[i].groups &&
                (best < 0 || (double)b.p[i].groups * b.p[i].cost / b.p[i].cta_count >
                                 (double)b.p[best].groups * b.p[best].cost / b.p[best].cta_count)) best = i;
        if (best < 0) break;
        ++b.p[best].cta_count; ++sum;
    }
    int begin = 0;
    for (int i = 0; i < b.count; ++i) {
        b.p[i].cta_begin = begin;
        begin += b.p[i].cta_count;
        b.p[i].per = b.p[i].groups / b.p[i].cta_count;
        b.p[i].rem = b.p[i].groups % b.p[i].cta_count;
    }
    return begin;
}

template <int NCLS, int NM, int TS>
static int im_launch(ImBatch &b, int groups_total, cudaStream_t s)
{
    constexpr int TRK = (NM == 1) ? 2 : 1;
    const ImSmem L = im_smem_layout(b.tab_smem_bytes, 8 * NM, TRK * 16, b.stages);
    auto kern = gemv_imma_kernel<NCLS, NM, TS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total);
    if (e != cudaSuccess) return cuda_fail(e);
    cudaLaunchConfig_t cfg = {};
    const int sms = im_sm_count();
    const int grid = im_assign_ctas(b, groups_total < sms ? groups_total : sms);
    cfg.gridDim = dim3((unsigned)grid);
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

template <int NCLS, int TS>
static int im_launch_nm(ImBatch &b, int nm, int groups_total, cudaStream_t s)
{
    if (nm != 1) return BTC_ERR_UNSUPPORTED;                // only the one-MMA form (M <= 2) is built here
    return im_launch<NCLS, 1, TS>(b, groups_total, s);
}

int launch(const LinearArgs *problems, int count, cudaStream_t s)
{
    if (count < 1 || count > IM_MAXP) return BTC_ERR_UNSUPPORTED;
    im_encode_fn enc = im_get_encode();
    if (!enc) return BTC_ERR_UNSUPPORTED;
    ImBatch b = {};
    b.count = count;
    int ncls_max = 0, m_max = 0, tab_max = 0, tab16_max = 0, v_max = 0;
    for (int i = 0; i < count; ++i) {
        const LinearArgs &a = problems[i];
        // covered: M <= 2, v a multiple of 4 up to 20, K/v a multiple of 8 (16-byte rows for the bulk copies)
        if (a.M < 1 || a.M > 2 || a.v % 4 != 0 || a.v > 20 || a.Kb % 8 != 0 || a.K > (1 << 20)) return BTC_ERR_UNSUPPORTED;
        // 16-bit activations, uint16 index containers, dense rows, overwrite: everything else is the other kernel's
        if (a.x_dt == BTC_F32 || a.idx_bits || a.x_stride || a.idx_stride || a.accumulate) return BTC_ERR_UNSUPPORTED;
        if (a.M > m_max) m_max = a.M;
    }
    const int nm = m_max <= 2 ? 1 : (m_max <= 5 ? 2 : 3);
    const int rows = (nm == 1) ? 32 : 16;
    int groups_total = 0;
    for (int i = 0; i < count; ++i) {
        const LinearArgs &a = problems[i];
        ImProblem &p = b.p[i];
        p.x = a.x; p.idx = a.idx; p.alpha = a.alpha; p.mu = a.mu; p.y = a.y;
        const int Kc4 = (a.Kc + 3) / 4 * 4;
        p.tab = a.Cp + 2 * Kc4;                      // byte-lane words follow the two other forms
        p.tab16 = reinterpret_cast<const uint16_t *>(a.Cp + 3 * (size_t)Kc4);
        p.M = a.M; p.N = a.N; p.K = a.K; p.v = a.v; p.Kc = a.Kc; p.Kb = a.Kb;
        p.x_dt = a.x_dt; p.y_dt = a.y_dt;
        p.parts = (a.Kb + IM_PW - 1) / IM_PW;
        p.groups = (a.N + rows - 1) / rows;
        p.ncls = a.v / 4;
        if (!im_tensor_map(enc, a.idx, a.Kb, a.N, rows, &b.map[i]))
            return BTC_ERR_UNSUPPORTED;                     // shape the tensor map cannot describe: other kernels take it
        // measured: an iteration (one row group x one part of up to 256 blocks) costs about the same whatever the
        // part's width, and rebuilding the activation fragments for a part costs ~1.5 iterations, shared by the
        // (few) row groups a CTA walks with it; a single-part layer rebuilds only once per CTA
        p.cost = p.parts > 1 ? p.parts * (IM_PW + 110) : a.Kb + 40;
        groups_total += p.groups;
        if (p.ncls > ncls_max) ncls_max = p.ncls;
        if (Kc4 * 4 > tab_max) tab_max = Kc4 * 4;
        if ((a.Kc + 7) / 8 * 16 > tab16_max) tab16_max = (a.Kc + 7) / 8 * 16;
        if (a.v > v_max) v_max = a.v;
    }
    // the whole table in shared memory when it fits beside at least four index stages; else, for v <= 16, as 16-bit
    // halves beside at least two; else as much of its head as fits
    int mode = 1;
    b.tab_smem_bytes = tab_max;
    b.tab_head = tab_max / 4;
    if (im_smem_layout(tab_max, 8 * nm, rows, 4).total > 227u * 1024u) {
        if (v_max <= 16 && im_smem_layout(tab16_max, 8 * nm, rows, 2).total <= 227u * 1024u) {
            mode = 3;
            b.tab_smem_bytes = tab16_max;
        } else {
            mode = 2;
            int head_bytes = tab_max;
            while (head_bytes > 0 && im_smem_layout(head_bytes, 8 * nm, rows, 4).total > 227u * 1024u) head_bytes -= 4096;
            if (head_bytes <= 0) { mode = 0; head_bytes = 0; }
            b.tab_smem_bytes = head_bytes;
            b.tab_head = head_bytes / 4;
        }
    }
    b.stages = IM_STAGES;
    while (b.stages > 2 && im_smem_layout(b.tab_smem_bytes, 8 * nm, rows, b.stages).total > 227u * 1024u) --b.stages;
    if (ncls_max <= 4) {
        if (mode == 1) return im_launch_nm<4, 1>(b, nm, groups_total, s);
        if (mode == 3) return im_launch_nm<4, 3>(b, nm, groups_total, s);
        if (mode == 2) return im_launch_nm<4, 2>(b, nm, groups_total, s);
        return im_launch_nm<4, 0>(b, nm, groups_total, s);
    }
    if (mode == 1) return im_launch_nm<5, 1>(b, nm, groups_total, s);
    if (mode == 2) return im_launch_nm<5, 2>(b, nm, groups_total, s);
    return im_launch_nm<5, 0>(b, nm, groups_total, s);
}

}  // namespace wide

int launch_gemv_imma_wide(const LinearArgs *problems, int count, cudaStream_t s)
{
    return wide::launch(problems, count, s);
}

int wide_status_reset()
{
    const int zero = 0;
    cudaError_t e = cudaMemcpyToSymbol(wide::g_wide_status, &zero, sizeof(int));
    return e == cudaSuccess ? BTC_OK : cuda_fail(e);
}

int wide_status_read(int *out)
{
    int v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, wide::g_wide_status, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    *out = v;
    return BTC_OK;
}

}  // namespace btc
