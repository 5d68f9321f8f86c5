// Decode path for small M (1..8): streams the index matrices of up to IM_MAXP independent layers
// once and evaluates every block dot
//     <x_j, C[idx]> = 2 * sum_{bit=1} x  -  sum x            (identity for +-1 codewords)
// (block-dot sum of the paper's appendix "Binary codebook LUT-GEMM") on the warp-level MMA, in one of
// two forms.
//
// Integer form (M <= 2).  One output needs K sign applications.  At the HBM rate an SM receives 180
// weights per clock (v = 16), while its plain ALUs issue 64 integer lane-operations per clock; of the
// warp-level MMAs that run natively here, mma.sync.m16n8k32 (u8 x s8 -> s32) takes the most weights per
// expansion instruction:
//   A (16 rows x 32 k, u8) = masked codeword bits: the codeword table stores weight t at bit (t >> 2)
//       of byte (t & 3), so `word & (0x01010101 << c)` IS the four bytes {0 or 2^c} of weights
//       4c .. 4c+3: one LOP3 expands four weights.
//   B (32 k x 8 cols, s8)  = the activations as three balanced base-256 digits of a block-fixed-point
//       integer: X = rint(x * 2^s), |X| <= 2^(22 - cmax), with s chosen per K-slice (512 activations
//       of one row of x at v = 16) from its largest magnitude, pre-shifted by (cmax - c) so that every
//       product is bit * X * 2^cmax; digit d of row m sits in column 4 m + d, so that both rows of x
//       see the same lanes and the same order of fp32 operations.
//   D (16 x 8, s32)        = exact partial sums.
// The three digit sums of a (slice, output) are recombined in fp32 (each is below 2^24, so the
// conversions are exact), scaled by 2^-s and added over the slices; then alpha (and mu) are applied.
// Roundings: the quantisation of x (2^-20 of the slice's largest magnitude for v = 16) and a handful
// of fp32 operations per output.
//
// fp16 form (3 <= M <= 8): see the comment at its branch in the kernel.  Masked codeword bits act as
// fp16 numbers on mma.sync.m16n8k16 against the activations themselves (eight rows of x are the eight
// columns of B), fp32 accumulation; twice the expansion instructions per weight, but no digits and a
// cost that does not grow with M.
//
// Work split.  A tile is 16 output rows of one layer; a CTA owns a contiguous, cost-weighted range of
// tiles of ONE layer (no CTA works on two layers: each switch would cost a table load).  Layers wider
// than one K-part (256 blocks; 128 in the fp16 form) are walked part by part over chunks of RC tiles, so
// the activation fragments change only once per part.
//   warps 0..7   compute: warp w owns K-slice w of the part (32 blocks; 16 in the fp16 form); lane
//                (g = lane / 4, t = lane % 4) supplies two rows of the tile and BPL consecutive blocks;
//                its activations stay in registers as MMA B fragments.  A tile's codewords are looked
//                up while the previous tile's MMAs are in flight.  The slice's share of every (row, m)
//                is parked in shared memory as one float; after the last part of a chunk the eight
//                warps meet once, add the slices in a fixed order, apply alpha (and mu) and store y.
//   warp 8       producer: TMA boxes (64 blocks x 16 rows, 128-byte swizzle) of the index matrix into
//                a shared ring of (tile, part) stages; bulk copy of the codeword table.
// Two CTAs fit an SM (shared memory and registers are sized for it), so while the CTAs of one launch
// compute, those of the next launch on the stream (programmatic dependent launch) already pull their
// indices and table into shared memory; only the activations are read after the dependency wait.
// Every mbarrier wait is bounded; when one runs out the CTA raises a status word and drains.
#include <cuda.h>
#include "btc_internal.cuh"

namespace btc {

constexpr int IM_CWARPS = 8;                    // compute warps = K-slices of a part
constexpr int IM_THREADS = (IM_CWARPS + 1) * 32;
constexpr int IM_STAGES = 12;                   // most index stages a launch may use (fewer when shared memory is short)
constexpr int IM_BOX_COLS = 64;                 // blocks per TMA box row: 128 bytes, the swizzle span
constexpr int IM_BOX_BYTES = 16 * 128;          // one box: 16 rows x 128 bytes

__device__ int g_imma_status = 0;

struct ImProblem {
    const void *x;
    const void *idx;          // uint16 [N, K/v], or rows of dense ib-bit fields
    const uint32_t *tab;      // byte-lane codeword words [Kc]
    const uint16_t *tab16;    // the same squeezed into 16 bits (v <= 16)
    const __half *alpha;
    const __half *mu;         // may be nullptr
    void *y;
    int M, N, K, v, Kc, Kb;
    int xs;                   // elements from one row of x to the next (K unless x is a column range of a wider matrix)
    int acc;                  // 1: add to what y holds (a further term of a sum of layers); y is fp32 then
    int x_dt, y_dt;
    int parts;                // ceil(Kb / part width)
    int groups;               // tiles: ceil(N / 16)
    int ncls;                 // v / 4
    int cost, fixed;          // cost of one tile and of a CTA's set-up for this layer (see launch_gemv_imma)
    int per, rem;             // groups / cta_count and groups % cta_count
    int cta_begin, cta_count; // the CTAs that work on this layer
};

struct ImBatch {
    CUtensorMap map[IM_MAXP]; // idx of each layer as a 2-D tensor {K/v, N} of 16-bit words, box {64, 16}, 128-byte swizzle
    ImProblem p[IM_MAXP];
    int count;
    int tab_smem_bytes;       // bytes reserved for the codeword table (0: gather from global memory)
    int tab_head;             // entries of every table that are staged there; the rest is gathered from global memory
                              // (L1/L2): a table of 65536 20-bit codewords does not fit, and with frequency-ordered
                              // codebooks the head serves most lookups
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
                    atomicExch(&g_imma_status, (int)BTC_ERR_TIMEOUT);
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
__device__ __forceinline__ void im_mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint64_t b) {
    asm volatile(
        "{\n\t.reg .b32 b0, b1;\n\t"
        "mov.b64 {b0, b1}, %8;\n\t"
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {b0,b1}, {%0,%1,%2,%3};\n\t}"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "l"(b));
}
__device__ __forceinline__ void im_mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint64_t b) {
    asm volatile(
        "{\n\t.reg .b32 b0, b1;\n\t"
        "mov.b64 {b0, b1}, %8;\n\t"
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {b0,b1}, {%0,%1,%2,%3};\n\t}"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "l"(b));
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
// NF consecutive IB-bit fields starting at field f0 of a packed row in shared memory (row: 4-byte aligned).  The words
// that hold them are read aligned and shifted into place; one word past the last needed bit may be read (the stage
// keeps 16 spare bytes for it).
template <int IB, int NF>
__device__ __forceinline__ void im_unpack_fields(const unsigned char *row, int f0, uint32_t (&f)[NF])
{
    constexpr int NW = (NF * IB + 31) / 32;                // words of the aligned bit string
    const uint32_t bit0 = (uint32_t)f0 * IB;
    const uint32_t *wp = reinterpret_cast<const uint32_t *>(row) + (bit0 >> 5);
    const uint32_t sh = bit0 & 31u;
    uint32_t w[NW + 1], a[NW + 1];
#pragma unroll
    for (int k = 0; k <= NW; ++k) w[k] = wp[k];
#pragma unroll
    for (int k = 0; k < NW; ++k) a[k] = __funnelshift_r(w[k], w[k + 1], sh);
    a[NW] = 0u;
#pragma unroll
    for (int i = 0; i < NF; ++i) {
        constexpr uint32_t mask = (1u << IB) - 1u;
        const int lo = (i * IB) >> 5, s = (i * IB) & 31;
        f[i] = __funnelshift_r(a[lo], a[lo + 1], s) & mask;
    }
}
// Codeword of index i: from the shared table (32-bit words, or 16-bit halves widened by h | (h << 12)), its shared
// head, or global memory, as TAB_MODE says.
template <int TAB_MODE>
__device__ __forceinline__ uint32_t im_codeword(uint32_t i, const uint32_t *s_tab, const uint32_t *gtab, uint32_t tab_head)
{
    if (TAB_MODE == 1) return s_tab[i];
    if (TAB_MODE == 3) {
        const uint32_t h = reinterpret_cast<const uint16_t *>(s_tab)[i];
        return h | (h << 12);
    }
    if (TAB_MODE == 0) return __ldg(gtab + i);
    return i < tab_head ? s_tab[i] : __ldg(gtab + i);
}
__device__ __forceinline__ void im_named_bar(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Eight consecutive activations of a row of x starting at element k0 (a multiple of 8) as floats.
__device__ __forceinline__ void im_load8(const void *xrow, int dt, int k0, float (&f)[8])
{
    if (dt == BTC_F32) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(xrow) + k0));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(xrow) + k0) + 1);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    } else {
        const uint4 q = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(xrow) + k0));
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (dt == BTC_F16) {
                const float2 p = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
                f[2 * i] = p.x; f[2 * i + 1] = p.y;
            } else {
                f[2 * i] = __uint_as_float(w[i] << 16);
                f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
            }
        }
    }
}

// Eight fp16 (dt = BTC_F16) or bf16 numbers held in a uint4 -> floats.
__device__ __forceinline__ void im_cvt8(const uint4 &q, int dt, float *f)
{
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (dt == BTC_F16) {
            const float2 p = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
            f[2 * i] = p.x; f[2 * i + 1] = p.y;
        } else {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
}

// Block-fixed-point scale of one K-slice of a row of x from the largest magnitude any lane saw (reduced over the warp
// here): X = rint(x * sc) has |X| <= 2^pbits, inv = 1 / sc, both powers of two.  A slice of zeros gives sc = inv = 0;
// a slice holding an inf or a nan gives inv = nan, so every output of that row of x becomes a nan, as the exact product
// would.
__device__ __forceinline__ void im_slice_scale(float amax, int pbits, float &sc, float &inv)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    // amax = f * 2^e with f in [1, 2) (a float widened from fp16 / bf16 is normal or zero; an fp32 subnormal counts
    // as tiny): |x| < 2^(e+1)
    const int ex = max((int)((__float_as_uint(amax) >> 23) & 0xffu) - 127 + 1, -100);
    const bool nz = amax > 0.f && amax < 3.0e38f;
    sc = nz ? __uint_as_float((uint32_t)(127 + pbits - ex) << 23) : 0.0f;
    inv = nz ? __uint_as_float((uint32_t)(127 - pbits + ex) << 23) : (amax == 0.f ? 0.0f : __uint_as_float(0x7fc00000u));
}

// Shared-memory layout (dynamic), offsets computed identically on host and device.
struct ImSmem {
    uint32_t bars;        // mbarriers: full[S], empty[S], tab_full
    uint32_t misc;        // abort flag; per compute warp and row m of x: its share of sum_k x
    uint32_t planes;      // per compute warp: digit planes of its K-slice of one row of x
    uint32_t tab;         // codeword table
    uint32_t ring;        // index stages
    uint32_t part;        // partial dot products, float [tile of the chunk][16 rows][MAXM][8 slices]
    uint32_t total;
};
constexpr int IM_NBARS = 2 * IM_STAGES + 1;
constexpr int IM_MISC_BYTES = 16 + IM_CWARPS * 8 * 4;

// NM = 1: the integer form (M <= 2, one MMA per A fragment).  NM = 0: the fp16 form (M <= 8).
template <int NM> struct ImShape {
    static constexpr int PW = (NM == 1) ? 256 : 128;           // blocks per K-part
    static constexpr int SLICE = PW / IM_CWARPS;               // blocks per compute warp
    static constexpr int BPL = SLICE / 4;                      // blocks per lane
    static constexpr int MAXM = (NM == 1) ? 2 : 8;
    static constexpr int RC = 12;                              // tiles a CTA walks part by part at a time
    static constexpr int PROW = RC * 16 + 4;                   // NM = 0: floats per (slice, m) row of the partial sums
};

// Bytes of one index stage: a (tile, part) of 16 rows.  ib = 0: 16-bit containers, boxes of 64 blocks x 16 rows with the
// 128-byte swizzle.  ib > 0: dense ib-bit fields (Section 4.3's index width), one unswizzled box of 16 rows x
// part_width * ib / 8 bytes, plus one spare 16 bytes because a lane's last aligned word may lie just past its row.
__host__ __device__ constexpr int im_stage_bytes(int nm, int ib)
{
    return ib == 0 ? (nm == 1 ? 256 : 128) / IM_BOX_COLS * IM_BOX_BYTES
                   : (16 * ((nm == 1 ? 256 : 128) * ib / 8) + 16 + 127) / 128 * 128;
}

__host__ __device__ inline ImSmem im_smem_layout(int tab_bytes, int nm, int stages, int ib = 0)
{
    const int slice = (nm == 1 ? 256 : 128) / IM_CWARPS;
    const int maxm = nm == 1 ? 2 : 8;
    const int rc = 12;
    const int stage_bytes = im_stage_bytes(nm, ib);
    ImSmem L;
    uint32_t o = 0;
    L.bars = o; o += IM_NBARS * 8;
    o = (o + 15u) & ~15u;
    L.misc = o; o += IM_MISC_BYTES;
    o = (o + 15u) & ~15u;
    L.planes = o;
    if (nm != 0) o += (uint32_t)IM_CWARPS * 3u * (uint32_t)(slice + 4) * 5u * 4u;   // 3 digits x (blocks + skew) x (v / 4 <= 5) words
    o = (o + 15u) & ~15u;
    L.part = o;
    o += (nm == 0) ? (uint32_t)IM_CWARPS * (uint32_t)maxm * (uint32_t)(rc * 16 + 4) * 4u
                   : (uint32_t)rc * 16u * (uint32_t)maxm * IM_CWARPS * 4u;
    o = (o + 127u) & ~127u;
    L.tab = o; o += (uint32_t)tab_bytes;
    o = (o + 1023u) & ~1023u;                     // swizzled TMA boxes want 1024-byte alignment
    L.ring = o; o += (uint32_t)stages * (uint32_t)stage_bytes;
    L.total = o;
    return L;
}

// Tiles [lo, hi) of layer P that fall to CTA b: the layer's cta_count CTAs split its tiles evenly (the first
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
template <int NCLS, int NM, int TAB_MODE, int IB>
__global__ void __launch_bounds__(IM_THREADS, 2)
gemv_imma_kernel(const __grid_constant__ ImBatch batch)
{
    extern __shared__ __align__(128) unsigned char smem[];
    using S = ImShape<NM>;
    constexpr int PW = S::PW, SLICE = S::SLICE, BPL = S::BPL, MAXM = S::MAXM, RC = S::RC;
    constexpr int STAGE_BYTES = im_stage_bytes(NM, IB);
    constexpr int ROWB = PW * IB / 8;                     // bytes of one row of a packed stage (IB > 0)
    const ImSmem L = im_smem_layout(batch.tab_smem_bytes, NM, batch.stages, IB);
    const int NST = batch.stages;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + L.misc);
    float *s_sx = reinterpret_cast<float *>(smem + L.misc + 16);                  // [8 warps][8]
    uint32_t *s_planes = reinterpret_cast<uint32_t *>(smem + L.planes);
    uint32_t *s_tab = reinterpret_cast<uint32_t *>(smem + L.tab);
    unsigned char *s_ring = smem + L.ring;
    float *s_part = reinterpret_cast<float *>(smem + L.part);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto bar_full = [&](int s) { return im_smem_u32(bars + s); };
    auto bar_empty = [&](int s) { return im_smem_u32(bars + IM_STAGES + s); };
    const uint32_t bar_tabfull = im_smem_u32(bars + 2 * IM_STAGES);

    if (tid == 0) {
        for (int s = 0; s < NST; ++s) { im_mbar_init(bar_full(s), 1); im_mbar_init(bar_empty(s), IM_CWARPS); }
        im_mbar_init(bar_tabfull, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr bool tab_smem = TAB_MODE != 0;             // (part of) the codeword table is staged in shared memory
    const uint32_t tab_head = (uint32_t)batch.tab_head;

    // the one layer this CTA works on, and its tiles
    int pi = 0, glo = 0, ghi = 0;
    for (; pi < batch.count; ++pi) {
        im_group_range(batch.p[pi], (int)blockIdx.x, glo, ghi);
        if (glo < ghi) break;
    }
    if (pi < batch.count) {
        const ImProblem &P = batch.p[pi];
        // Both roles walk the same sequence: chunks [c0, c1) of at most RC tiles, K-parts j, tiles r.
        if (warp == IM_CWARPS) {
            // ============================================================ producer
            if (tab_smem && lane == 0) {
                const uint32_t bytes = TAB_MODE == 3 ? (uint32_t)((P.Kc + 7) / 8 * 8 * 2)
                                                     : (uint32_t)(min((P.Kc + 3) / 4 * 4, batch.tab_head) * 4);
                im_mbar_expect_tx(bar_tabfull, bytes);
                im_bulk_g2s(im_smem_u32(s_tab), TAB_MODE == 3 ? static_cast<const void *>(P.tab16) : static_cast<const void *>(P.tab),
                            bytes, bar_tabfull);
            }
            int li = 0, s = 0;                                     // ring stage li % NST; rph = (li / NST) & 1
            uint32_t rph = 0;
            bool ok = true;
            for (int c0 = glo; c0 < ghi && ok; c0 += RC) {
                const int c1 = min(c0 + RC, ghi);
                for (int j = 0; j < P.parts && ok; ++j) {
                    // every stage is filled whole (boxes of 64 blocks x 16 rows): rows past N and blocks past K/v arrive
                    // as zeros, so a consumer never meets an index left behind by an earlier stage
                    constexpr int nbox = PW / IM_BOX_COLS;
                    for (int r = c0; r < c1; ++r, ++li) {
                        if (li >= NST && !im_mbar_wait(bar_empty(s), rph ^ 1u, s_abort)) { ok = false; break; }
                        if constexpr (IB == 0) {
                            if (lane == 0) im_mbar_expect_tx(bar_full(s), (uint32_t)nbox * IM_BOX_BYTES);
                            __syncwarp();
                            if (lane < nbox)
                                im_tma_2d(im_smem_u32(s_ring + (size_t)s * STAGE_BYTES + (size_t)lane * IM_BOX_BYTES), &batch.map[pi],
                                          j * PW + lane * IM_BOX_COLS, r * 16, bar_full(s));
                        } else {
                            // dense fields: the part of 16 rows is one box of 32-bit words (coordinates in words)
                            if (lane == 0) {
                                im_mbar_expect_tx(bar_full(s), 16u * ROWB);
                                im_tma_2d(im_smem_u32(s_ring + (size_t)s * STAGE_BYTES), &batch.map[pi], j * (ROWB / 4), r * 16, bar_full(s));
                            }
                        }
                        if (++s == NST) { s = 0; rph ^= 1u; }
                    }
                }
            }
        } else {
            // ============================================================ compute warps
            if constexpr (NM == 0) {
            // ---- fp16 form (M <= 8).  An fp16 bit pattern with one bit p <= 14 set is the number 2^(p-24), so the
            // codeword word of the "fp16 layout" (weight t at bit (t & 1) * 16 + P0 + (t >> 1), P0 = 12 - v/2) masked
            // with one bit per half IS a pair of multiplicands {0 or 2^(P0+i-24)} for the weights 2i, 2i+1: one LOP3
            // per two weights, no conversion.  mma.sync.m16n8k16 (fp16 x fp16 -> fp32):
            //   A (16 rows x 16 k) = masked codeword bits: lane (g, t) supplies, for rows g and g + 8, four weights
            //       (class c = weights 4c .. 4c+3) of a block it owns; the four lanes of a quad own four blocks;
            //   B (16 k x 8 cols)  = the activations of row m = column, as fp16, scaled per K-slice by 2^(E-i) so that
            //       every product is bit * x * 2^(E+P0-24) exactly (E from the slice's largest magnitude: no overflow);
            //   D (16 x 8, fp32)   = sums over set bits for 16 outputs x 8 rows of x, fp32 accumulation.
            // The sum of the slice's activations (for the identity's "- sum x" and the mean term) comes from the same
            // MMAs with all mask bits as A.  The cost does not depend on M.
            const int g = lane >> 2, t = lane & 3;
            const int ks = warp;
            const int sg = ((g & 1) << 2) | (g >> 1);
            const int M = P.M, K = P.K, Kb = P.Kb, v = P.v;
            const int P0 = 12 - v / 2;
            constexpr int PROW = S::PROW;
            uint32_t pm[2 * NCLS];                                 // mask of pair i: bit P0 + i of both halves
#pragma unroll
            for (int i = 0; i < 2 * NCLS; ++i) pm[i] = (2 * i < v) ? (0x00010001u << (P0 + i)) : 0u;
            const uint32_t *gtab = P.tab;
            const int xsz = (P.x_dt == BTC_F32) ? 4 : 2;
            bool tab_ready = !tab_smem;
            bool ok = true;
            int s = 0;
            uint32_t rph = 0;
            const int boff = (ks * SLICE + BPL * t) * 2;
            const uint32_t idx_off = (uint32_t)(boff >> 7) * IM_BOX_BYTES + (uint32_t)sg * 128
                                     + ((((boff >> 4) & 7) ^ (sg & 7)) << 4) + (boff & 15);
            const int ct = tid;
            for (int c0 = glo; c0 < ghi; c0 += RC) {
                const int c1 = min(c0 + RC, ghi);
                const int nrows = (c1 - c0) * 16;
                const int nout = nrows * M;
                constexpr int OPT = (RC * 16 * MAXM + IM_CWARPS * 32 - 1) / (IM_CWARPS * 32);
                unsigned short areg[OPT], mreg[OPT];
#pragma unroll
                for (int q = 0; q < OPT; ++q) {
                    const int o = ct + q * (IM_CWARPS * 32);
                    areg[q] = 0; mreg[q] = 0;
                    if (o < nout) {
                        const int n = c0 * 16 + (o % nrows);
                        if (n < P.N) {
                            areg[q] = __ldg(reinterpret_cast<const unsigned short *>(P.alpha) + n);
                            if (P.mu) mreg[q] = __ldg(reinterpret_cast<const unsigned short *>(P.mu) + n);
                        }
                    }
                }
                if (c0 == glo) asm volatile("griddepcontrol.wait;" ::: "memory");
                float sx0 = 0.f, sx1 = 0.f;                        // lanes g = 0: this slice's sum_k x[m, k], m = 2t, 2t+1

                for (int j = 0; j < P.parts; ++j) {
                    const int pw = min(PW, Kb - j * PW);
                    const bool wvalid = ks * SLICE + BPL * t < pw;
                    // ---- B fragments: lane (g = m, t) reads the activations of row m for its own BPL blocks
                    uint64_t breg[BPL][NCLS];
                    const bool has = wvalid && g < M;
                    const unsigned char *xrow = reinterpret_cast<const unsigned char *>(P.x) + (size_t)g * P.xs * xsz;
                    // 16-bit activations: all of this lane's loads are issued before anything uses them; with v = 16 a
                    // lane's four blocks are 128 contiguous bytes, read 16 bytes (two classes) at a time
                    uint2 raw[BPL][NCLS];
                    const bool x16 = P.x_dt != BTC_F32;
                    if (NCLS == 4 && v == 16) {
#pragma unroll
                        for (int e = 0; e < BPL; ++e)
#pragma unroll
                            for (int c = 0; c < NCLS; c += 2) {
                                uint4 q = make_uint4(0u, 0u, 0u, 0u);
                                if (x16 && has)
                                    q = __ldg(reinterpret_cast<const uint4 *>(
                                        xrow + ((size_t)(j * PW + ks * SLICE + BPL * t + e) * 16 + 4 * c) * 2));
                                raw[e][c] = make_uint2(q.x, q.y);
                                raw[e][c + 1] = make_uint2(q.z, q.w);
                            }
                    } else {
#pragma unroll
                        for (int e = 0; e < BPL; ++e)
#pragma unroll
                            for (int c = 0; c < NCLS; ++c) {
                                raw[e][c] = make_uint2(0u, 0u);
                                if (x16 && has && 4 * c < v)
                                    raw[e][c] = __ldg(reinterpret_cast<const uint2 *>(
                                        xrow + ((size_t)(j * PW + ks * SLICE + BPL * t + e) * v + 4 * c) * 2));
                            }
                    }
                    // the four activations of class c of this lane's block e, as floats (fp32 activations are read from
                    // memory twice: once for the largest magnitude, once to scale; the second read is served by L1)
                    auto x4 = [&](int e, int c, float (&f)[4]) {
                        f[0] = f[1] = f[2] = f[3] = 0.f;
                        if (x16) {
                            const uint2 q = raw[e][c];
                            if (P.x_dt == BTC_F16) {
                                const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&q.x));
                                const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&q.y));
                                f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
                            } else {
                                f[0] = __uint_as_float(q.x << 16); f[1] = __uint_as_float(q.x & 0xffff0000u);
                                f[2] = __uint_as_float(q.y << 16); f[3] = __uint_as_float(q.y & 0xffff0000u);
                            }
                        } else if (has && 4 * c < v) {
                            const size_t k0 = (size_t)(j * PW + ks * SLICE + BPL * t + e) * v + 4 * c;
                            const float4 q = __ldg(reinterpret_cast<const float4 *>(xrow + k0 * 4));
                            f[0] = q.x; f[1] = q.y; f[2] = q.z; f[3] = q.w;
                        }
                    };
                    float amax = 0.f;
#pragma unroll
                    for (int e = 0; e < BPL; ++e)
#pragma unroll
                        for (int c = 0; c < NCLS; ++c) {
                            float f[4];
                            x4(e, c, f);
                            amax = fmaxf(fmaxf(amax, fmaxf(fabsf(f[0]), fabsf(f[1]))), fmaxf(fabsf(f[2]), fabsf(f[3])));
                        }
                    // largest magnitude of (row m, slice): over the four lanes of the quad
                    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
                    // amax = f * 2^e, f in [1, 2): x * 2^(14 - e) stays below 2^15
                    int E = 14 - ((int)((__float_as_uint(amax) >> 23) & 0xffu) - 127);
                    E = min(max(E, -90), 100);
#pragma unroll
                    for (int e = 0; e < BPL; ++e) {
#pragma unroll
                        for (int c = 0; c < NCLS; ++c) {
                            float f[4];
                            x4(e, c, f);
                            const float s0 = __uint_as_float((uint32_t)(127 + E - 2 * c) << 23);        // 2^(E - i), i = 2c
                            const float s1 = __uint_as_float((uint32_t)(127 + E - 2 * c - 1) << 23);    // i = 2c + 1
                            const __half2 h0 = __floats2half2_rn(f[0] * s0, f[1] * s0);
                            const __half2 h1 = __floats2half2_rn(f[2] * s1, f[3] * s1);
                            breg[e][c] = (uint64_t)(*reinterpret_cast<const uint32_t *>(&h0))
                                         | ((uint64_t)(*reinterpret_cast<const uint32_t *>(&h1)) << 32);
                        }
                    }
                    // scale of the two output columns this lane holds (m = 2t, 2t+1): 2^(24 - E_m - P0)
                    const int Elo = __shfl_sync(0xffffffffu, E, 8 * t), Ehi = __shfl_sync(0xffffffffu, E, 8 * t + 4);
                    const float us_lo = __uint_as_float((uint32_t)(127 + 24 - Elo - P0) << 23);
                    const float us_hi = __uint_as_float((uint32_t)(127 + 24 - Ehi - P0) << 23);
                    {   // sum of the slice's activations: the same MMAs with every mask bit as A
                        float sa[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int e = 0; e < BPL; ++e)
#pragma unroll
                            for (int c = 0; c < NCLS; ++c)
                                im_mma_f16(sa, pm[2 * c], pm[2 * c], pm[2 * c + 1], pm[2 * c + 1], breg[e][c]);
                        sx0 += sa[0] * us_lo;
                        sx1 += sa[1] * us_hi;
                    }
                    if (!tab_ready) {
                        ok &= im_mbar_wait(bar_tabfull, 0, s_abort);
                        tab_ready = true;
                    }
                    uint32_t w0[BPL], w1[BPL];
                    auto fetch = [&]() {
                        ok &= im_mbar_wait(bar_full(s), rph, s_abort);
                        if constexpr (IB > 0) {
                            uint32_t fa[BPL], fb[BPL];
                            const unsigned char *st = s_ring + (size_t)s * STAGE_BYTES;
                            im_unpack_fields<IB, BPL>(st + sg * ROWB, ks * SLICE + BPL * t, fa);
                            im_unpack_fields<IB, BPL>(st + (sg + 8) * ROWB, ks * SLICE + BPL * t, fb);
                            if (!ok) {
#pragma unroll
                                for (int e = 0; e < BPL; ++e) { fa[e] = 0u; fb[e] = 0u; }
                            }
                            // (the loads must have returned before the stage is handed back: see below)
#pragma unroll
                            for (int e = 0; e < BPL; ++e) asm volatile("" :: "r"(fa[e]), "r"(fb[e]) : "memory");
                            __syncwarp();
                            if (lane == 0) im_mbar_arrive(bar_empty(s));
                            if (++s == NST) { s = 0; rph ^= 1u; }
#pragma unroll
                            for (int e = 0; e < BPL; ++e) {
                                w0[e] = im_codeword<TAB_MODE>(fa[e], s_tab, gtab, tab_head);
                                w1[e] = im_codeword<TAB_MODE>(fb[e], s_tab, gtab, tab_head);
                            }
                            return;
                        }
                        const unsigned char *pa = s_ring + (size_t)s * STAGE_BYTES + idx_off;
                        uint2 qa = *reinterpret_cast<const uint2 *>(pa), qb = *reinterpret_cast<const uint2 *>(pa + 8 * 128);
                        if (!ok) { qa = make_uint2(0u, 0u); qb = qa; }
                        // the index loads must have RETURNED before the stage is handed back: the arrive below does not
                        // wait for loads in flight, and the producer's next copy into this stage may land within a few
                        // hundred clocks when it comes from L2 (seen as stale half boxes before this line was here)
                        asm volatile("" :: "r"(qa.x), "r"(qa.y), "r"(qb.x), "r"(qb.y) : "memory");
                        __syncwarp();
                        if (lane == 0) im_mbar_arrive(bar_empty(s));
                        if (++s == NST) { s = 0; rph ^= 1u; }
                        const uint32_t ia[2] = {qa.x, qa.y}, ib[2] = {qb.x, qb.y};
                        if constexpr (TAB_MODE == 1) {
                            const uint32_t tb = im_smem_u32(s_tab);
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                uint32_t a0, a1, b0, b1;
                                im_pair_addr(ia[i], tb, a0, a1);
                                im_pair_addr(ib[i], tb, b0, b1);
                                w0[2 * i] = im_lds32(a0); w0[2 * i + 1] = im_lds32(a1);
                                w1[2 * i] = im_lds32(b0); w1[2 * i + 1] = im_lds32(b1);
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < BPL; ++e) {
                                const uint32_t i0 = (e & 1) ? (ia[e >> 1] >> 16) : (ia[e >> 1] & 0xffffu);
                                const uint32_t i1 = (e & 1) ? (ib[e >> 1] >> 16) : (ib[e >> 1] & 0xffffu);
                                w0[e] = im_codeword<TAB_MODE>(i0, s_tab, gtab, tab_head);
                                w1[e] = im_codeword<TAB_MODE>(i1, s_tab, gtab, tab_head);
                            }
                        }
                    };
                    fetch();
                    for (int r = c0; r < c1; ++r) {
                        float acc[2][4];
#pragma unroll
                        for (int ch = 0; ch < 2; ++ch)
#pragma unroll
                            for (int i = 0; i < 4; ++i) acc[ch][i] = 0.f;
                        if (ks * SLICE < pw) {
#pragma unroll
                            for (int e = 0; e < BPL; ++e)
#pragma unroll
                                for (int c = 0; c < NCLS; ++c)
                                    im_mma_f16(acc[(e * NCLS + c) & 1], w0[e] & pm[2 * c], w1[e] & pm[2 * c], w0[e] & pm[2 * c + 1],
                                               w1[e] & pm[2 * c + 1], breg[e][c]);
                        }
                        if (r + 1 < c1) fetch();
                        // rows sg, sg + 8 x columns m = 2t, 2t+1: one float per (slice, m, row); later parts add up
                        if (2 * t < M) {
                            const int rl = (r - c0) * 16 + sg;
                            float *q0 = s_part + (size_t)(ks * MAXM + 2 * t) * PROW + rl, *q1 = q0 + PROW;
                            const float v00 = (acc[0][0] + acc[1][0]) * us_lo, v01 = (acc[0][1] + acc[1][1]) * us_hi;
                            const float v10 = (acc[0][2] + acc[1][2]) * us_lo, v11 = (acc[0][3] + acc[1][3]) * us_hi;
                            if (j == 0) { q0[0] = v00; q1[0] = v01; q0[8] = v10; q1[8] = v11; }
                            else { q0[0] += v00; q1[0] += v01; q0[8] += v10; q1[8] += v11; }
                        }
                    }
                }
                if (g == 0) { s_sx[ks * 8 + 2 * t] = sx0; s_sx[ks * 8 + 2 * t + 1] = sx1; }
                im_named_bar(1, IM_CWARPS * 32);
                if (ok && !*s_abort) {
#pragma unroll
                    for (int q = 0; q < OPT; ++q) {
                        const int o = ct + q * (IM_CWARPS * 32);
                        if (o < nout) {
                            const int m = o / nrows, rl = o - m * nrows;
                            const int n = c0 * 16 + rl;
                            float dot1 = 0.f, sx = 0.f;
#pragma unroll
                            for (int w = 0; w < IM_CWARPS; ++w) {
                                dot1 += s_part[(size_t)(w * MAXM + m) * PROW + rl];
                                sx += s_sx[w * 8 + m];
                            }
                            if (n < P.N) {
                                const float al = __half2float(__ushort_as_half(areg[q])), mu = __half2float(__ushort_as_half(mreg[q]));
                                float yv = al * (2.0f * dot1 - sx) + mu * sx;
                                if (P.acc) yv += reinterpret_cast<const float *>(P.y)[(size_t)m * P.N + n];
                                store_from_float(P.y, P.y_dt, (size_t)m * P.N + n, yv);
                            }
                        }
                    }
                }
                if (c1 < ghi) im_named_bar(1, IM_CWARPS * 32);
            }
            } else {
            const int g = lane >> 2, t = lane & 3;
            constexpr float MAGIC = 12582912.0f;                   // 1.5 * 2^23: float -> int by addition
            constexpr int MAGIC_BITS = 0x4B400000;
            const int ks = warp;                                   // K-slice of this warp
            // MMA row g (and g + 8) carries tile row sg (and sg + 8): neighbouring g differ in bit 2 of the row, so the
            // eight lanes of a shared-memory phase read distinct swizzled chunks
            const int sg = ((g & 1) << 2) | (g >> 1);
            // digit planes of a slice: block b, class c of digit d at word d * PSW + (b + b / BPL) * NCLS + c; the skew
            // puts the lanes of a fragment read (t: blocks BPL apart, d: planes) on different banks
            constexpr int PSW = (SLICE + 4) * NCLS;
            uint32_t *planes = s_planes + ks * (3 * (SLICE + 4) * 5);
            const int M = P.M, K = P.K, Kb = P.Kb, v = P.v;
            const int cmax = P.ncls - 1;
            const int PBITS = 22 - cmax;                           // |X| <= 2^PBITS
            const int ngroups = SLICE * v / 8;                     // groups of 8 activations in a slice (<= 80)
            const float unshift2 = 2.0f / (float)(1 << cmax);
            const uint32_t *gtab = P.tab;
            const int xsz = (P.x_dt == BTC_F32) ? 4 : 2;
            bool tab_ready = !tab_smem;
            bool ok = true;
            int li = 0, s = 0;
            uint32_t rph = 0;
            // byte offset of this lane's index chunk inside a stage (128-byte swizzle: 16-byte chunk c of row q sits
            // at chunk c ^ (q & 7)); rows sg and sg + 8
            const int boff = (ks * SLICE + BPL * t) * 2;
            const uint32_t idx_off = (uint32_t)(boff >> 7) * IM_BOX_BYTES + (uint32_t)sg * 128
                                     + ((((boff >> 4) & 7) ^ (sg & 7)) << 4) + (boff & 15);
            const int ct = tid;                                    // 0 .. 255: position among the compute threads

            for (int c0 = glo; c0 < ghi; c0 += RC) {
                const int c1 = min(c0 + RC, ghi);
                const int nrows = (c1 - c0) * 16;
                const int nout = nrows * M;                        // outputs of this chunk: (m, tile row) pairs
                // alpha / mu of the outputs this thread will finish (static data: the loads are issued ahead of the
                // dependency wait and of the chunk's work, and land while it runs)
                constexpr int OPT = (RC * 16 * MAXM + IM_CWARPS * 32 - 1) / (IM_CWARPS * 32);   // outputs per thread
                unsigned short areg[OPT], mreg[OPT];
#pragma unroll
                for (int q = 0; q < OPT; ++q) {
                    const int o = ct + q * (IM_CWARPS * 32);
                    areg[q] = 0; mreg[q] = 0;
                    if (o < nout) {
                        const int n = c0 * 16 + (o % nrows);
                        if (n < P.N) {
                            areg[q] = __ldg(reinterpret_cast<const unsigned short *>(P.alpha) + n);
                            if (P.mu) mreg[q] = __ldg(reinterpret_cast<const unsigned short *>(P.mu) + n);
                        }
                    }
                }
                if (c0 == glo) asm volatile("griddepcontrol.wait;" ::: "memory");
                float sxw[MAXM];                                   // this warp's share of sum_k x[m, k] (lane 0)
#pragma unroll
                for (int m = 0; m < MAXM; ++m) sxw[m] = 0.f;

                for (int j = 0; j < P.parts; ++j) {
                    const int pw = min(PW, Kb - j * PW);
                    const int jb0 = j * PW + ks * SLICE;            // first block of this warp's slice
                    const bool wvalid = ks * SLICE + BPL * t < pw;  // this lane's blocks exist (pw % 8 == 0)
                    const int kend = (j * PW + pw) * v;             // end of the part in x

                    // ---- B fragments for this part.  The warp's slice of each row of x is quantised with its own
                    //      scale: X = rint(x * 2^(PBITS - e)), 2^e > max |x| of the slice.
                    // (kept as 64-bit values: the two registers of an MMA's B operand then always sit in an aligned pair)
                    constexpr int NPAIR = (NCLS + 1) / 2;
                    uint64_t breg[BPL][NPAIR][NM];
                    float invs[MAXM];
#pragma unroll
                    for (int e = 0; e < BPL; ++e)
#pragma unroll
                        for (int c = 0; c < NPAIR; ++c)
#pragma unroll
                            for (int nm = 0; nm < NM; ++nm) breg[e][c][nm] = 0ull;
#pragma unroll
                    for (int m = 0; m < MAXM; ++m) invs[m] = 0.f;
                    constexpr int NU = (SLICE * 20 / 8 + 31) / 32;  // groups of 8 activations per lane (v <= 20)
                    const bool fast16 = (NM == 1 && NCLS == 4 && v == 16);   // lane = block of the slice: no index arithmetic
                    // 16-bit activations of the fast path: row m + 1 is fetched while row m is quantised
                    const bool pf16 = fast16 && P.x_dt != BTC_F32;
                    const bool pin = ks * SLICE + lane < pw;
                    const size_t pk0 = (size_t)(jb0 + lane) * 16;
                    uint4 cur0 = make_uint4(0u, 0u, 0u, 0u), cur1 = cur0;
                    if (pf16 && pin) {
                        const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(P.x) + pk0);
                        cur0 = __ldg(src);
                        cur1 = __ldg(src + 1);
                    }
#pragma unroll 1
                    for (int m = 0; m < M; ++m) {
                        const unsigned char *xrow = reinterpret_cast<const unsigned char *>(P.x) + (size_t)m * P.xs * xsz;
                        float inv;
                        int xs = 0;
                        uint4 nxt0 = make_uint4(0u, 0u, 0u, 0u), nxt1 = nxt0;
                        if (pf16 && pin && m + 1 < M) {
                            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(P.x) + (size_t)(m + 1) * P.xs + pk0);
                            nxt0 = __ldg(src);
                            nxt1 = __ldg(src + 1);
                        }
                        if (fast16) {
                            float xf[16];
                            const bool in = ks * SLICE + lane < pw;
#pragma unroll
                            for (int i = 0; i < 16; ++i) xf[i] = 0.f;
                            if (pf16) {
                                im_cvt8(cur0, P.x_dt, &xf[0]);
                                im_cvt8(cur1, P.x_dt, &xf[8]);
                            } else if (in) {
                                im_load8(xrow, P.x_dt, (jb0 + lane) * 16, *reinterpret_cast<float (*)[8]>(&xf[0]));
                                im_load8(xrow, P.x_dt, (jb0 + lane) * 16 + 8, *reinterpret_cast<float (*)[8]>(&xf[8]));
                            }
                            float amax = 0.f;
#pragma unroll
                            for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(xf[i]));
                            float sc;
                            im_slice_scale(amax, PBITS, sc, inv);
                            uint32_t bq[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                bq[i] = (uint32_t)__float_as_int(xf[i] * sc + MAGIC);
                                xs += (int)(bq[i] - (uint32_t)MAGIC_BITS);
                            }
                            uint32_t dg[3][4];                       // digit d of the four activations of class c, one byte each
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const uint32_t sh = 1u << (3 - c);
                                const uint32_t off = 0x8080u - (uint32_t)MAGIC_BITS * sh;        // arithmetic modulo 2^32
                                // Y = X * 2^(cmax - c) + 0x8080: byte d of Y is balanced digit d of X * 2^(cmax-c), + 0x80 for d < 2
                                const uint32_t y0 = bq[4 * c] * sh + off, y1 = bq[4 * c + 1] * sh + off;
                                const uint32_t y2 = bq[4 * c + 2] * sh + off, y3 = bq[4 * c + 3] * sh + off;
                                const uint32_t t0 = __byte_perm(y0, y1, 0x5140), t1 = __byte_perm(y2, y3, 0x5140);
                                const uint32_t t2 = __byte_perm(y0, y1, 0x0062), t3 = __byte_perm(y2, y3, 0x0062);
                                dg[0][c] = __byte_perm(t0, t1, 0x5410) ^ 0x80808080u;
                                dg[1][c] = __byte_perm(t0, t1, 0x7632) ^ 0x80808080u;
                                dg[2][c] = __byte_perm(t2, t3, 0x5410);
                            }
#pragma unroll
                            for (int d = 0; d < 3; ++d)
                                *reinterpret_cast<uint4 *>(planes + d * PSW + (lane + (lane >> 3)) * 4) =
                                    make_uint4(dg[d][0], dg[d][1], dg[d][2], dg[d][3]);
                        } else {
                            float xf[NU][8];
                            float amax = 0.f;
#pragma unroll
                            for (int u = 0; u < NU; ++u) {
                                const int gi = lane + 32 * u;
                                const int k0 = jb0 * v + 8 * gi;
#pragma unroll
                                for (int i = 0; i < 8; ++i) xf[u][i] = 0.f;
                                if (gi < ngroups && k0 < kend) im_load8(xrow, P.x_dt, k0, xf[u]);
#pragma unroll
                                for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(xf[u][i]));
                            }
                            float sc;
                            im_slice_scale(amax, PBITS, sc, inv);
#pragma unroll
                            for (int u = 0; u < NU; ++u) {
                                const int gi = lane + 32 * u;
                                if (gi < ngroups) {
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
                                        const uint32_t b0 = (uint32_t)__float_as_int(xf[u][4 * h] * sc + MAGIC);
                                        const uint32_t b1 = (uint32_t)__float_as_int(xf[u][4 * h + 1] * sc + MAGIC);
                                        const uint32_t b2 = (uint32_t)__float_as_int(xf[u][4 * h + 2] * sc + MAGIC);
                                        const uint32_t b3 = (uint32_t)__float_as_int(xf[u][4 * h + 3] * sc + MAGIC);
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
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) xs += __shfl_xor_sync(0xffffffffu, xs, o);
#pragma unroll
                        for (int mm = 0; mm < MAXM; ++mm)
                            if (mm == m) { invs[mm] = inv; sxw[mm] += (float)xs * inv; }
                        __syncwarp();
#pragma unroll
                        for (int nm = 0; nm < NM; ++nm) {
                            const int col = g + 8 * nm;
                            const int mc = col >> 2, d = col & 3;     // column 4 m + d
                            if (mc == m && d < 3 && wvalid) {
                                const uint32_t *src = planes + d * PSW + (BPL * t + t) * NCLS;
#pragma unroll
                                for (int e = 0; e < BPL; ++e) {
                                    if (NCLS == 4) {
                                        const uint4 q = *reinterpret_cast<const uint4 *>(src + e * 4);
                                        breg[e][0][nm] = (uint64_t)q.x | ((uint64_t)q.y << 32);
                                        breg[e][NPAIR - 1][nm] = (uint64_t)q.z | ((uint64_t)q.w << 32);
                                    } else {
#pragma unroll
                                        for (int c = 0; c < NCLS / 2; ++c)
                                            breg[e][c][nm] = (uint64_t)src[e * NCLS + 2 * c] | ((uint64_t)src[e * NCLS + 2 * c + 1] << 32);
                                        // the odd class of two neighbouring blocks shares one MMA: block e even holds the pair
                                        if ((NCLS & 1) && !(e & 1))
                                            breg[e][NPAIR - 1][nm] = (uint64_t)src[e * NCLS + NCLS - 1] | ((uint64_t)src[(e + 1) * NCLS + NCLS - 1] << 32);
                                    }
                                }
                            }
                        }
                        __syncwarp();
                        cur0 = nxt0; cur1 = nxt1;
                    }
                    if (!tab_ready) {
                        ok &= im_mbar_wait(bar_tabfull, 0, s_abort);
                        tab_ready = true;
                    }

                    // ---- the tiles of the chunk, for this part.  A tile's codewords are fetched (index stage -> registers ->
                    //      table lookups) while the previous tile's MMAs are still in flight.
                    uint32_t w0[BPL], w1[BPL];                      // codewords of rows sg and sg + 8, this lane's blocks
                    auto fetch = [&]() {
                        uint32_t ia[BPL / 2], ib[BPL / 2];
                        ok &= im_mbar_wait(bar_full(s), rph, s_abort);
                        if constexpr (IB > 0) {
                            uint32_t fa[BPL], fb[BPL];
                            const unsigned char *st = s_ring + (size_t)s * STAGE_BYTES;
                            im_unpack_fields<IB, BPL>(st + sg * ROWB, ks * SLICE + BPL * t, fa);
                            im_unpack_fields<IB, BPL>(st + (sg + 8) * ROWB, ks * SLICE + BPL * t, fb);
                            if (!ok) {
#pragma unroll
                                for (int e = 0; e < BPL; ++e) { fa[e] = 0u; fb[e] = 0u; }
                            }
                            // (the loads must have returned before the stage is handed back: see the fp16 form)
#pragma unroll
                            for (int e = 0; e < BPL; ++e) asm volatile("" :: "r"(fa[e]), "r"(fb[e]) : "memory");
                            __syncwarp();
                            if (lane == 0) im_mbar_arrive(bar_empty(s));
                            if (++s == NST) { s = 0; rph ^= 1u; }
#pragma unroll
                            for (int e = 0; e < BPL; ++e) {
                                w0[e] = im_codeword<TAB_MODE>(fa[e], s_tab, gtab, tab_head);
                                w1[e] = im_codeword<TAB_MODE>(fb[e], s_tab, gtab, tab_head);
                            }
                            return;
                        }
                        {
                            // (every stage is filled whole: blocks past the part and rows past N arrive as zeros)
                            const unsigned char *pa = s_ring + (size_t)s * STAGE_BYTES + idx_off;
                            const unsigned char *pb = pa + 8 * 128;                 // row + 8: same row & 7
                            const uint4 qa = *reinterpret_cast<const uint4 *>(pa), qb = *reinterpret_cast<const uint4 *>(pb);
                            ia[0] = qa.x; ia[1] = qa.y; ia[2] = qa.z; ia[3] = qa.w;
                            ib[0] = qb.x; ib[1] = qb.y; ib[2] = qb.z; ib[3] = qb.w;
                        }
                        if (!ok) {                                  // a wait gave up: the stage may hold anything
#pragma unroll
                            for (int i = 0; i < BPL / 2; ++i) { ia[i] = 0u; ib[i] = 0u; }
                        }
                        // the index loads must have returned before the stage is handed back (see the fp16 form)
#pragma unroll
                        for (int i = 0; i < BPL / 2; ++i) asm volatile("" :: "r"(ia[i]), "r"(ib[i]) : "memory");
                        __syncwarp();
                        if (lane == 0) im_mbar_arrive(bar_empty(s));
                        if (++s == NST) { s = 0; rph ^= 1u; }
                        if constexpr (TAB_MODE == 1) {
                            // whole table in shared memory as 32-bit words: each pair of packed indices becomes two
                            // shared addresses by one widening multiply-add per index (base + 4 * idx)
                            const uint32_t tb = im_smem_u32(s_tab);
#pragma unroll
                            for (int i = 0; i < BPL / 2; ++i) {
                                uint32_t a0, a1, b0, b1;
                                im_pair_addr(ia[i], tb, a0, a1);
                                im_pair_addr(ib[i], tb, b0, b1);
                                w0[2 * i] = im_lds32(a0); w0[2 * i + 1] = im_lds32(a1);
                                w1[2 * i] = im_lds32(b0); w1[2 * i + 1] = im_lds32(b1);
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < BPL; ++e) {
                                const uint32_t pa = ia[e >> 1], pb = ib[e >> 1];
                                const uint32_t i0 = (e & 1) ? (pa >> 16) : (pa & 0xffffu);
                                const uint32_t i1 = (e & 1) ? (pb >> 16) : (pb & 0xffffu);
                                w0[e] = im_codeword<TAB_MODE>(i0, s_tab, gtab, tab_head);
                                w1[e] = im_codeword<TAB_MODE>(i1, s_tab, gtab, tab_head);
                            }
                        }
                    };
                    fetch();
                    for (int r = c0; r < c1; ++r, ++li) {
                        constexpr int CH = 2;        // accumulation chains: an MMA need not wait for the previous one
                        int accs[CH][NM][4];
#pragma unroll
                        for (int ch = 0; ch < CH; ++ch)
#pragma unroll
                            for (int nm = 0; nm < NM; ++nm)
#pragma unroll
                                for (int i = 0; i < 4; ++i) accs[ch][nm][i] = 0;
                        int (&acc)[NM][4] = accs[0];
                        if (ks * SLICE < pw) {                      // warp-uniform: the slice is not empty
#pragma unroll
                            for (int e = 0; e < BPL; ++e) {
#pragma unroll
                                for (int cp = 0; cp < NCLS / 2; ++cp) {
                                    const uint32_t ma = 0x01010101u << (2 * cp), mb = 0x01010101u << (2 * cp + 1);
#pragma unroll
                                    for (int nm = 0; nm < NM; ++nm)
                                        im_mma_u8s8(accs[((e & 1) * 2 + (cp & 1)) % CH][nm], w0[e] & ma, w1[e] & ma, w0[e] & mb, w1[e] & mb,
                                                    breg[e][cp][nm]);
                                }
                            }
                            if (NCLS & 1) {
                                const uint32_t ml = 0x01010101u << (NCLS - 1);
#pragma unroll
                                for (int ep = 0; ep < BPL / 2; ++ep)
#pragma unroll
                                    for (int nm = 0; nm < NM; ++nm)
                                        im_mma_u8s8(accs[ep % CH][nm], w0[2 * ep] & ml, w1[2 * ep] & ml, w0[2 * ep + 1] & ml,
                                                    w1[2 * ep + 1] & ml, breg[2 * ep][NPAIR - 1][nm]);
                            }
                        }
                        if (r + 1 < c1) fetch();
#pragma unroll
                        for (int nm = 0; nm < NM; ++nm)
#pragma unroll
                            for (int i = 0; i < 4; ++i)
#pragma unroll
                                for (int ch = 1; ch < CH; ++ch) acc[nm][i] += accs[ch][nm][i];
                        // The three digit sums of a (row, m) are recombined (each is below 2^24 in magnitude, so the
                        // conversions are exact), scaled by the slice's 2^-s and parked as one float per (row, m, slice);
                        // later parts add to what the same thread left there.
                        float *mine = s_part + ((size_t)(r - c0) * 16 * MAXM) * IM_CWARPS + ks;
                        {
                            // columns 4 m + d: lane t = 2 m holds digits 0 and 1, lane 2 m + 1 holds digit 2 (and an empty column)
                            const float wa = (t & 1) ? 65536.0f : 1.0f, wb = (t & 1) ? 0.0f : 256.0f;
                            float plo = fmaf((float)acc[0][1], wb, (float)acc[0][0] * wa);
                            float phi = fmaf((float)acc[0][3], wb, (float)acc[0][2] * wa);
                            plo += __shfl_xor_sync(0xffffffffu, plo, 1);
                            phi += __shfl_xor_sync(0xffffffffu, phi, 1);
                            const int m = t >> 1;
                            if (!(t & 1) && m < M) {
                                const float iv = m ? invs[MAXM > 1 ? 1 : 0] : invs[0];
                                float *qlo = mine + (sg * MAXM + m) * IM_CWARPS, *qhi = mine + ((sg + 8) * MAXM + m) * IM_CWARPS;
                                if (j == 0) { *qlo = plo * iv; *qhi = phi * iv; }
                                else { *qlo += plo * iv; *qhi += phi * iv; }
                            }
                        }
                    }
                }
                if (lane == 0) {
#pragma unroll
                    for (int m = 0; m < MAXM; ++m) s_sx[ks * 8 + m] = sxw[m];
                }
                // ---- the eight slices meet: add them in a fixed order, apply alpha (and mu), store
                im_named_bar(1, IM_CWARPS * 32);
                if (ok && !*s_abort) {
#pragma unroll
                    for (int q = 0; q < OPT; ++q) {
                        const int o = ct + q * (IM_CWARPS * 32);
                        if (o < nout) {
                            const int m = o / nrows, rl = o - m * nrows;
                            const int n = c0 * 16 + rl;
                            const float4 p0 = *reinterpret_cast<const float4 *>(s_part + ((size_t)rl * MAXM + m) * IM_CWARPS);
                            const float4 p1 = *reinterpret_cast<const float4 *>(s_part + ((size_t)rl * MAXM + m) * IM_CWARPS + 4);
                            const float dot1 = ((((((p0.x + p0.y) + p0.z) + p0.w) + p1.x) + p1.y) + p1.z) + p1.w;
                            float sx = 0.f;
#pragma unroll
                            for (int w = 0; w < IM_CWARPS; ++w) sx += s_sx[w * 8 + m];
                            if (n < P.N) {
                                const float al = __half2float(__ushort_as_half(areg[q])), mu = __half2float(__ushort_as_half(mreg[q]));
                                const float dot = dot1 * unshift2 - sx;         // 2 * sum_{bit=1} x - sum x
                                float yv = al * dot + mu * sx;
                                if (P.acc) yv += reinterpret_cast<const float *>(P.y)[(size_t)m * P.N + n];
                                store_from_float(P.y, P.y_dt, (size_t)m * P.N + n, yv);
                            }
                        }
                    }
                }
                if (c1 < ghi) im_named_bar(1, IM_CWARPS * 32);      // the next chunk overwrites what was just read
            }
            }
        }
    } else {
        // (a CTA without work: the launch never creates one, but the dependency contract holds anyway)
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

// Tensor map of an index matrix {K/v, N} (16-bit words), box {64, 16}, 128-byte swizzle.  Encoding goes through the
// driver and costs about a microsecond; a decode step re-uses the same matrices call after call, so the last few
// maps are kept per host thread, keyed by everything the encoding depends on.
static bool im_tensor_map(im_encode_fn enc, const void *idx, int Kb, int N, int ib, size_t pitch, int box_words, CUtensorMap *out)
{
    struct Entry { const void *idx; int Kb, N, ib, box; size_t pitch; CUtensorMap map; };
    constexpr int SLOTS = 64;
    thread_local Entry cache[SLOTS];
    thread_local int used = 0, next = 0;
    for (int i = 0; i < used; ++i)
        if (cache[i].idx == idx && cache[i].Kb == Kb && cache[i].N == N && cache[i].ib == ib && cache[i].box == box_words && cache[i].pitch == pitch) { *out = cache[i].map; return true; }
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap m;
    if (ib == 0) {
        const cuuint64_t dims[2] = {(cuuint64_t)Kb, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)pitch};          // bytes from row to row (Kb * 2 unless idx is a column range)
        const cuuint32_t box[2] = {(cuuint32_t)IM_BOX_COLS, 16u};
        if (enc(&m, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void *>(idx), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    } else {
        // dense ib-bit fields: rows of `pitch` bytes seen as 32-bit words; one box = a part of 16 rows, no swizzle
        const cuuint64_t dims[2] = {(cuuint64_t)(pitch / 4), (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)pitch};
        const cuuint32_t box[2] = {(cuuint32_t)box_words, 16u};
        if (enc(&m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(idx), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    Entry &e = cache[next];
    e.idx = idx; e.Kb = Kb; e.N = N; e.ib = ib; e.box = box_words; e.pitch = pitch; e.map = m;
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

// Gives every layer a whole number of CTAs so that the largest load of any CTA -- ceil(tiles / CTAs) tiles times
// the layer's cost per tile, plus the layer's set-up cost; tiles are not divisible -- is as small as the budget
// allows, and returns the grid size.  Smallest feasible load by bisection; a load T needs
// ceil(tiles / floor((T - fixed) / cost)) CTAs of a layer.
static int im_assign_ctas(ImBatch &b, int budget)
{
    auto tiles_per_cta = [&](int i, long long T) { return (T - b.p[i].fixed) / b.p[i].cost; };
    auto ctas_needed = [&](long long T) {
        long long sum = 0;
        for (int i = 0; i < b.count; ++i) {
            const long long per = tiles_per_cta(i, T);                // tiles one CTA may take
            if (per < 1) return (long long)1 << 40;
            sum += (b.p[i].groups + per - 1) / per;
        }
        return sum;
    };
    long long lo = 1, hi = 0;
    for (int i = 0; i < b.count; ++i) {
        const long long all = (long long)b.p[i].groups * b.p[i].cost + b.p[i].fixed;
        if (all > hi) hi = all;                                       // one CTA per layer always fits (budget >= count)
    }
    while (lo < hi) {
        const long long mid = (lo + hi) / 2;
        if (ctas_needed(mid) <= budget) hi = mid; else lo = mid + 1;
    }
    int sum = 0;
    for (int i = 0; i < b.count; ++i) {
        const long long per = tiles_per_cta(i, lo);
        b.p[i].cta_count = (int)((b.p[i].groups + per - 1) / per);
        sum += b.p[i].cta_count;
    }
    while (sum < budget) {                          // spare CTAs: more SMs streaming, where the average load is highest
        int best = -1;
        for (int i = 0; i < b.count; ++i)
            if (b.p[i].cta_count < b.p[i].groups &&
                (best < 0 || (double)b.p[i].groups * b.p[i].cost / b.p[i].cta_count + b.p[i].fixed >
                                 (double)b.p[best].groups * b.p[best].cost / b.p[best].cta_count + b.p[best].fixed)) best = i;
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

template <int NCLS, int NM, int TS, int IB>
static int im_launch(ImBatch &b, int groups_total, cudaStream_t s)
{
    const ImSmem L = im_smem_layout(b.tab_smem_bytes, NM, b.stages, IB);
    auto kern = gemv_imma_kernel<NCLS, NM, TS, IB>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total);
    if (e != cudaSuccess) return cuda_fail(e);
    cudaLaunchConfig_t cfg = {};
    // CTAs that can be resident at once: two per SM when the shared memory asked for allows it
    const int per_sm = (2u * (L.total + 1024u) <= 228u * 1024u) ? 2 : 1;
    const int slots = im_sm_count() * per_sm;
    const int grid = im_assign_ctas(b, groups_total < slots ? groups_total : slots);
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
static int im_launch_nm(ImBatch &b, int nm, int ib, int groups_total, cudaStream_t s)
{
    if (ib != 0) {
        // dense indices: built for the widths of the v = 16 codebooks of 4096 and 8192 centroids, whole table in
        // shared memory
        if constexpr (NCLS == 4 && (TS == 1 || TS == 3)) {
            if (nm == 1) {
                if (ib == 12) return im_launch<4, 1, TS, 12>(b, groups_total, s);
                if (ib == 13) return im_launch<4, 1, TS, 13>(b, groups_total, s);
            } else if (TS == 1) {
                if (ib == 12) return im_launch<4, 0, 1, 12>(b, groups_total, s);
                if (ib == 13) return im_launch<4, 0, 1, 13>(b, groups_total, s);
            }
        }
        return BTC_ERR_UNSUPPORTED;
    }
    if (nm == 1) return im_launch<NCLS, 1, TS, 0>(b, groups_total, s);
    if (TS == 3) return BTC_ERR_UNSUPPORTED;                // (the 16-bit table exists for the byte-lane words only)
    return im_launch<NCLS, 0, TS == 3 ? 1 : TS, 0>(b, groups_total, s);
}

int launch_gemv_imma(const LinearArgs *problems, int count, cudaStream_t s)
{
    if (count < 1 || count > IM_MAXP) return BTC_ERR_UNSUPPORTED;
    im_encode_fn enc = im_get_encode();
    if (!enc) return BTC_ERR_UNSUPPORTED;
    ImBatch b = {};
    b.count = count;
    int ncls_max = 0, m_max = 0, tab_max = 0, tab16_max = 0, v_max = 0;
    for (int i = 0; i < count; ++i) {
        const LinearArgs &a = problems[i];
        // covered: M <= 8, v a multiple of 4 up to 20, K/v a multiple of 8 (16-byte rows for the bulk copies)
        if (a.M < 1 || a.M > 8 || a.v % 4 != 0 || a.v > 20 || a.Kb % 8 != 0 || a.K > (1 << 20)) return BTC_ERR_UNSUPPORTED;
        if (a.x_dt == BTC_F32 && a.K % 8 != 0) return BTC_ERR_UNSUPPORTED;
        if (a.accumulate && a.y_dt != BTC_F32) return BTC_ERR_UNSUPPORTED;
        if ((a.x_stride && a.x_stride % 8) || (a.idx_stride && (a.idx_stride % 8 || a.idx_bits))) return BTC_ERR_UNSUPPORTED;
        if (a.M > m_max) m_max = a.M;
        if (a.idx_bits != problems[0].idx_bits) return BTC_ERR_UNSUPPORTED;      // one index format per launch
    }
    const int ib = problems[0].idx_bits;
    const int nm = m_max <= 2 ? 1 : 0;                      // integer form up to two rows of x, fp16 form above
    const int pw = nm == 1 ? 256 : 128;
    // the ring is no longer than the longest walk of any CTA needs; the split below assumes the full ring
    int groups_total = 0;
    for (int i = 0; i < count; ++i) {
        const LinearArgs &a = problems[i];
        ImProblem &p = b.p[i];
        p.x = a.x; p.idx = a.idx_bits ? a.idx_packed : static_cast<const void *>(a.idx); p.alpha = a.alpha; p.mu = a.mu; p.y = a.y;
        const int Kc4 = (a.Kc + 3) / 4 * 4;
        p.tab = a.Cp + (nm == 0 ? 1 : 2) * Kc4;      // fp16-layout words (fp16 form) or byte-lane words (integer form)
        p.tab16 = reinterpret_cast<const uint16_t *>(a.Cp + 3 * (size_t)Kc4);
        p.M = a.M; p.N = a.N; p.K = a.K; p.v = a.v; p.Kc = a.Kc; p.Kb = a.Kb;
        p.xs = a.x_stride ? a.x_stride : a.K;
        p.acc = a.accumulate ? 1 : 0;
        p.x_dt = a.x_dt; p.y_dt = a.y_dt;
        p.parts = (a.Kb + pw - 1) / pw;
        p.groups = (a.N + 15) / 16;
        p.ncls = a.v / 4;
        if (!im_tensor_map(enc, p.idx, a.Kb, a.N, ib, ib ? a.idx_pitch : (size_t)(a.idx_stride ? a.idx_stride : a.Kb) * 2, pw * ib / 32, &b.map[i]))
            return BTC_ERR_UNSUPPORTED;                     // shape the tensor map cannot describe: other kernels take it
        // a (tile, part) costs about the same whatever the part's width; rebuilding the activation fragments for a
        // part costs about as much as one and a half of them and is shared by the tiles a CTA walks with that part
        p.cost = p.parts * 16;                               // per tile, in sixteenths of a (tile, part)
        p.fixed = p.parts * 24 * (nm == 0 ? 1 : a.M);        // per CTA (the fp16 form builds all rows of x at once)
        groups_total += p.groups;
        if (p.ncls > ncls_max) ncls_max = p.ncls;
        if (Kc4 * 4 > tab_max) tab_max = Kc4 * 4;
        if ((a.Kc + 7) / 8 * 16 > tab16_max) tab16_max = (a.Kc + 7) / 8 * 16;
        if (a.v > v_max) v_max = a.v;
    }
    // Two CTAs per SM is the aim: 113 KB each.  The table goes to shared memory as 32-bit words when that leaves room
    // for at least six index stages, else (v <= 16) as 16-bit halves, else as much of its head as fits one CTA per SM.
    const uint32_t half_sm = 113u * 1024u, whole_sm = 227u * 1024u;
    int mode = 1;
    b.tab_smem_bytes = tab_max;
    b.tab_head = tab_max / 4;
    uint32_t budget = half_sm;
    if (im_smem_layout(tab_max, nm, 6, ib).total > half_sm) {
        if (nm == 1 && v_max <= 16 && im_smem_layout(tab16_max, nm, 4, ib).total <= half_sm) {
            mode = 3;
            b.tab_smem_bytes = tab16_max;
        } else if (nm == 1 && v_max <= 16 && im_smem_layout(tab16_max, nm, 2, ib).total <= whole_sm) {
            mode = 3;
            b.tab_smem_bytes = tab16_max;
            budget = whole_sm;
        } else if (im_smem_layout(tab_max, nm, 4, ib).total <= whole_sm) {
            budget = whole_sm;
        } else {
            mode = 2;
            budget = whole_sm;
            int head_bytes = tab_max;
            while (head_bytes > 0 && im_smem_layout(head_bytes, nm, 4, ib).total > whole_sm) head_bytes -= 4096;
            if (head_bytes <= 0) { mode = 0; head_bytes = 0; }
            b.tab_smem_bytes = head_bytes;
            b.tab_head = head_bytes / 4;
        }
    }
    b.stages = IM_STAGES;
    while (b.stages > 2 && im_smem_layout(b.tab_smem_bytes, nm, b.stages, ib).total > budget) --b.stages;
    if (ncls_max <= 4) {
        if (mode == 1) return im_launch_nm<4, 1>(b, nm, ib, groups_total, s);
        if (mode == 3) return im_launch_nm<4, 3>(b, nm, ib, groups_total, s);
        if (mode == 2) return im_launch_nm<4, 2>(b, nm, ib, groups_total, s);
        return im_launch_nm<4, 0>(b, nm, ib, groups_total, s);
    }
    if (mode == 1) return im_launch_nm<5, 1>(b, nm, ib, groups_total, s);
    if (mode == 2) return im_launch_nm<5, 2>(b, nm, ib, groups_total, s);
    return im_launch_nm<5, 0>(b, nm, ib, groups_total, s);
}

// Self-test of the bounded wait: one warp waits (with a ~1 ms limit) on a barrier that nothing ever arrives on, which
// must raise the status word and return -- the same code path a lost producer or consumer would take in the kernels.
__global__ void im_selftest_wait_kernel()
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        im_mbar_init(im_smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    (void)im_mbar_wait(im_smem_u32(&bar), 0, &abort_flag, 2000000LL);
}

int imma_selftest_wait(cudaStream_t s)
{
    im_selftest_wait_kernel<<<1, 32, 0, s>>>();
    return cuda_check_launch();
}

int imma_status_reset()
{
    const int zero = 0;
    cudaError_t e = cudaMemcpyToSymbol(g_imma_status, &zero, sizeof(int));
    return e == cudaSuccess ? BTC_OK : cuda_fail(e);
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
