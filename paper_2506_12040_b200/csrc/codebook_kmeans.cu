// Binary codebook construction (paper Section 4.1 "Flash and Accurate Binary Codebook"; loop of the appendix
// Algorithm "Binary Codebook Optimization"): initial centroids = the most frequent distinct vectors, then
//   E-step  z_i = argmin_k d_H(b_i, c_k) = POPCNT(b_i xor c_k)      (||b - c||^2 = 4 d_H; smallest k among equals)
//   M-step  c_k = element-wise majority of the vectors assigned to k  (ties -> +1; an empty cluster keeps its centroid)
// until no assignment changes or max_iter E-steps have run.
//
// Everything is done in the space of the 2^v possible patterns (v <= 20: the paper's range; 65536 of them at v = 16),
// not per vector:
// identical vectors have identical nearest centroids, so one histogram pass over the n vectors (the only pass that
// streams them, besides the final look-up of z) reduces every later step to at most 2^v weighted patterns:
//   histogram       cnt[p]                                     n atomic adds
//   initial order   rank(p) = #{q : (cnt[q], -q) > (cnt[p], -p)}  (frequency descending, packed word ascending);
//                   pattern p becomes centroid rank(p) when rank(p) < c; counted among the patterns at least as
//                   frequent as the c-th most frequent one (threshold by bisection, then a candidate list)
//   E-step          one thread per occurring pattern, centroids broadcast from shared memory;
//                   min over k of (POPCNT << 16 | k) is the nearest centroid with the smallest index among equals
//   M-step          per occurring pattern: add cnt[p] to the vote counters of its cluster; then one thread per centroid
// No step synchronises with the host: the iteration loop is unrolled into max_iter rounds of launches, and every
// kernel of a round returns at once when an earlier round has already found the assignments unchanged.
// Integer arithmetic only; results are bit-exact against the definition.
#include "btc_internal.cuh"

namespace btc {

constexpr int KM_VMAX = 20;                  // longest vector: the steps keep tables of 2^v entries
constexpr int KM_VMAX_SLOTS = 32;            // vote counters per centroid

struct KmState {
    int done;         // 1: assignments unchanged in an E-step (the loop has ended)
    int iters;        // E-steps run
    int kc_eff;       // min(c, number of distinct vectors)
    int n_unique;
    int changed;      // set by the E-step of the current round
    unsigned thr;     // frequency of the c-th most frequent distinct vector (1 when there are fewer than c)
    int n_cand;       // distinct vectors more frequent than that (fewer than c): ranked pairwise; the ones exactly that
                      // frequent follow them in the order of their packed words
};

struct KmWorkspace {
    KmState *st;
    uint32_t *cnt;        // [P]
    uint32_t *label;      // [2][P], E-step i writes half i & 1
    uint32_t *tot;        // [Kc]
    uint32_t *ones;       // [Kc][KM_VMAX_SLOTS]
    uint32_t *cand_p;     // [P] candidate patterns (unordered) ...
    uint32_t *cand_c;     // [P] ... and their frequencies
};

__host__ __device__ inline size_t km_align(size_t x) { return (x + 255) & ~(size_t)255; }

static KmWorkspace km_carve(void *ws, int v, int Kc)
{
    const size_t P = (size_t)1 << v;
    unsigned char *p = reinterpret_cast<unsigned char *>(ws);
    KmWorkspace w;
    w.st = reinterpret_cast<KmState *>(p); p += km_align(sizeof(KmState));
    w.cnt = reinterpret_cast<uint32_t *>(p); p += km_align(P * 4);
    w.label = reinterpret_cast<uint32_t *>(p); p += km_align(2 * P * 4);
    w.tot = reinterpret_cast<uint32_t *>(p); p += km_align((size_t)Kc * 4);
    w.ones = reinterpret_cast<uint32_t *>(p); p += km_align((size_t)Kc * KM_VMAX_SLOTS * 4);
    w.cand_p = reinterpret_cast<uint32_t *>(p); p += km_align(P * 4);
    w.cand_c = reinterpret_cast<uint32_t *>(p);
    return w;
}

static size_t km_workspace_bytes(int v, int Kc)
{
    const size_t P = (size_t)1 << v;
    return km_align(sizeof(KmState)) + km_align(P * 4) + km_align(2 * P * 4) + km_align((size_t)Kc * 4) + km_align((size_t)Kc * KM_VMAX_SLOTS * 4) +
           2 * km_align(P * 4);
}

__global__ void km_hist_kernel(const uint32_t *__restrict__ vecs, size_t n, uint32_t mask, uint32_t *__restrict__ cnt)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (; i < n; i += stride) atomicAdd(cnt + (vecs[i] & mask), 1u);
}

// Initial centroids: occurring pattern p goes to slot rank(p) if that is below c, where rank counts the patterns that
// are more frequent, or as frequent with a smaller packed word.  Only patterns at least as frequent as the c-th most
// frequent one can get a slot.  Those strictly more frequent (fewer than c) are ranked against one another; those
// exactly as frequent (possibly many: frequencies of rare patterns tie) come after them in word order, which is a
// prefix count, not a comparison of pairs.
constexpr int KM_TILE = 2048;

// One CTA: number of distinct vectors, and the largest threshold t with #{p : cnt[p] >= t} >= c (bisection over t).
__global__ void __launch_bounds__(1024)
km_threshold_kernel(const uint32_t *__restrict__ cnt, int P, int Kc, KmState *st)
{
    __shared__ unsigned s_red[32];
    __shared__ unsigned s_val;
    auto block_sum = [&](unsigned v) -> unsigned {
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
        __syncthreads();
        if (threadIdx.x < 32) {
            unsigned w = s_red[threadIdx.x];
            for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
            if (threadIdx.x == 0) s_val = w;
        }
        __syncthreads();
        return s_val;
    };
    // up to 65536 patterns (v <= 16) the thread's 64 frequencies stay in registers over the bisection
    constexpr int KEEP = 64;
    const bool kept = P <= KEEP * 1024;
    uint32_t mine[KEEP];
#pragma unroll
    for (int i = 0; i < KEEP; ++i) {
        const int p = threadIdx.x + i * 1024;
        mine[i] = (kept && p < P) ? cnt[p] : 0u;
    }
    auto count_ge = [&](unsigned t) -> unsigned {
        unsigned c = 0;
        if (kept) {
#pragma unroll
            for (int i = 0; i < KEEP; ++i) c += (mine[i] >= t) ? 1u : 0u;
        } else {
            for (int p = threadIdx.x; p < P; p += blockDim.x) c += (cnt[p] >= t) ? 1u : 0u;
        }
        return block_sum(c);
    };
    unsigned mx = 0;
    for (int p = threadIdx.x; p < P; p += blockDim.x) mx = max(mx, cnt[p]);
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = 0;
    for (int i = 0; i < 32; ++i) mx = max(mx, s_red[i]);
    const unsigned n_unique = count_ge(1u);
    unsigned lo = 1u, hi = max(mx, 1u);                     // invariant: count_ge(lo) >= min(c, n_unique)
    if (n_unique > (unsigned)Kc) {
        while (lo < hi) {
            const unsigned mid = lo + (hi - lo + 1u) / 2u;
            if (count_ge(mid) >= (unsigned)Kc) lo = mid; else hi = mid - 1u;
        }
    }
    if (threadIdx.x == 0) {
        st->n_unique = (int)n_unique;
        st->kc_eff = min(Kc, (int)n_unique);
        st->thr = (n_unique > (unsigned)Kc) ? lo : 1u;
    }
}

__global__ void km_candidates_kernel(const uint32_t *__restrict__ cnt, int P, uint32_t *__restrict__ cand_p, uint32_t *__restrict__ cand_c, KmState *st)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    const uint32_t c = cnt[p];
    if (c > st->thr) {                                      // strictly more frequent than the c-th: fewer than c of them
        const int pos = atomicAdd(&st->n_cand, 1);
        cand_p[pos] = (uint32_t)p;
        cand_c[pos] = c;
    }
}

// (frequency, word) of a candidate as one key: larger key = earlier slot.
__device__ __forceinline__ unsigned long long km_key(uint32_t c, uint32_t p) { return ((unsigned long long)c << 32) | (0xffffffffu - p); }

constexpr int KM_RANK_THREADS = 64;                         // small blocks: a few thousand candidates should still fill the SMs
__global__ void __launch_bounds__(KM_RANK_THREADS)
km_init_rank_kernel(const uint32_t *__restrict__ cand_p, const uint32_t *__restrict__ cand_c, int Kc, uint32_t *__restrict__ C, const KmState *st)
{
    __shared__ __align__(16) unsigned long long s_key[KM_TILE];
    const int L = st->n_cand;
    if ((int)(blockIdx.x * blockDim.x) >= L) return;        // (uniform over the block)
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = i < L;
    const uint32_t p = live ? cand_p[i] : 0u;
    const unsigned long long mine = live ? km_key(cand_c[i], p) : ~0ull;
    int rank = 0;
    for (int q0 = 0; q0 < L; q0 += KM_TILE) {
        __syncthreads();
        for (int j = threadIdx.x; j < KM_TILE; j += blockDim.x)
            s_key[j] = (q0 + j < L) ? km_key(cand_c[q0 + j], cand_p[q0 + j]) : 0ull;     // (key 0 ranks before nothing)
        __syncthreads();
#pragma unroll 8
        for (int j = 0; j < KM_TILE; ++j) rank += (s_key[j] > mine) ? 1 : 0;
    }
    if (live && rank < Kc) C[rank] = p;
}

// The patterns exactly as frequent as the c-th most frequent one follow the strictly more frequent ones in the order
// of their packed words: rank = n_cand + (number of such patterns with a smaller word), a prefix count over p.
__global__ void __launch_bounds__(1024)
km_ties_kernel(const uint32_t *__restrict__ cnt, int P, int Kc, uint32_t *__restrict__ C, const KmState *st)
{
    // each warp takes a contiguous range of patterns and walks it 32 at a time (coalesced); the order inside a step comes
    // from a ballot, the order of the warps from a prefix over their totals
    __shared__ int s_tot[32];
    const unsigned thr = st->thr;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seg = (((P + 31) / 32) + 31) & ~31;           // patterns per warp, a multiple of 32
    const int p_begin = warp * seg;
    int total = 0;
    for (int q = p_begin; q < p_begin + seg; q += 32) {
        const int p = q + lane;
        total += __popc(__ballot_sync(0xffffffffu, p < P && cnt[p] == thr));
    }
    if (lane == 0) s_tot[warp] = total;
    __syncthreads();
    int rank = st->n_cand;
    for (int w = 0; w < warp; ++w) rank += s_tot[w];
    for (int q = p_begin; q < p_begin + seg; q += 32) {
        const int p = q + lane;
        const bool tie = p < P && cnt[p] == thr;
        const unsigned b = __ballot_sync(0xffffffffu, tie);
        if (tie) {
            const int r = rank + __popc(b & ((1u << lane) - 1u));
            if (r < Kc) C[r] = (uint32_t)p;
        }
        rank += __popc(b);
    }
}

__global__ void __launch_bounds__(256)
km_estep_kernel(const uint32_t *__restrict__ cnt, int P, const uint32_t *__restrict__ C, uint32_t *__restrict__ label, KmState *st)
{
    __shared__ __align__(16) uint32_t s_C[KM_TILE];
    if (st->done) return;                                   // (uniform over the grid: set only between launches)
    const int it = st->iters, kc = st->kc_eff;
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = (p < P) && cnt[p] != 0u;
    uint32_t best = 0xffffffffu;
    for (int k0 = 0; k0 < kc; k0 += KM_TILE) {
        __syncthreads();
        for (int i = threadIdx.x; i < KM_TILE; i += blockDim.x) s_C[i] = (k0 + i < kc) ? C[k0 + i] : 0u;
        __syncthreads();
        if (live) {
            const int lim = min(KM_TILE, kc - k0);
            int i = 0;
            for (; i + 4 <= lim; i += 4) {
                const uint4 c = *reinterpret_cast<const uint4 *>(s_C + i);
                best = min(best, ((uint32_t)__popc((uint32_t)p ^ c.x) << 16) | (uint32_t)(k0 + i));
                best = min(best, ((uint32_t)__popc((uint32_t)p ^ c.y) << 16) | (uint32_t)(k0 + i + 1));
                best = min(best, ((uint32_t)__popc((uint32_t)p ^ c.z) << 16) | (uint32_t)(k0 + i + 2));
                best = min(best, ((uint32_t)__popc((uint32_t)p ^ c.w) << 16) | (uint32_t)(k0 + i + 3));
            }
            for (; i < lim; ++i) best = min(best, ((uint32_t)__popc((uint32_t)p ^ s_C[i]) << 16) | (uint32_t)(k0 + i));
        }
    }
    if (live) {
        const uint32_t z = best & 0xffffu;
        uint32_t *cur = label + (size_t)(it & 1) * P, *prev = label + (size_t)((it & 1) ^ 1) * P;
        cur[p] = z;
        if (it == 0 || prev[p] != z) st->changed = 1;       // (benign race: every writer stores 1)
    }
}

// After an E-step: count it; if nothing changed the loop is over (its M-step does not run).
__global__ void km_round_kernel(KmState *st)
{
    if (st->done) return;
    st->iters += 1;
    if (!st->changed) st->done = 1;
    st->changed = 0;
}

__global__ void km_vote_kernel(const uint32_t *__restrict__ cnt, int P, int v, const uint32_t *__restrict__ label,
                               uint32_t *__restrict__ tot, uint32_t *__restrict__ ones, const KmState *st)
{
    if (st->done) return;
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    const uint32_t c = cnt[p];
    if (!c) return;
    const uint32_t k = label[(size_t)((st->iters - 1) & 1) * P + p];     // the E-step just counted wrote half (iters - 1) & 1
    atomicAdd(tot + k, c);
    for (int t = 0; t < v; ++t)
        if ((p >> t) & 1) atomicAdd(ones + (size_t)k * KM_VMAX_SLOTS + t, c);
}

__global__ void km_update_kernel(int v, uint32_t *__restrict__ C, uint32_t *__restrict__ tot, uint32_t *__restrict__ ones, const KmState *st)
{
    if (st->done) return;
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= st->kc_eff) return;
    const uint32_t n = tot[k];
    if (n) {
        uint32_t w = 0;
        for (int t = 0; t < v; ++t) {
            const uint32_t o = ones[(size_t)k * KM_VMAX_SLOTS + t];
            if (o >= n - o) w |= 1u << t;                   // at least as many +1 as -1: sign(0) = +1
            ones[(size_t)k * KM_VMAX_SLOTS + t] = 0;
        }
        C[k] = w;
        tot[k] = 0;
    }
}

__global__ void km_assign_kernel(const uint32_t *__restrict__ vecs, size_t n, uint32_t mask, int P, const uint32_t *__restrict__ label,
                                 uint16_t *__restrict__ z, int *__restrict__ info, const KmState *st)
{
    const uint32_t *fin = label + (size_t)((st->iters - 1) & 1) * P;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) { info[0] = st->iters; info[1] = st->kc_eff; info[2] = st->n_unique; info[3] = st->done; }
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (; i < n; i += stride) z[i] = (uint16_t)fin[vecs[i] & mask];
}

}  // namespace btc

using namespace btc;

extern "C" BTC_API size_t btc_codebook_kmeans_workspace_bytes(int v, int Kc)
{
    if (v < 1 || v > KM_VMAX || Kc < 1 || Kc > 65536) return 0;
    return km_workspace_bytes(v, Kc);
}

extern "C" BTC_API int btc_codebook_kmeans(const uint32_t *vecs, size_t n, int v, int Kc, int max_iter, uint32_t *C_words,
                                           uint16_t *z, int *info, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!vecs || !C_words || !z || !info || !workspace) return BTC_ERR_NULL;
    if (Kc < 1 || Kc > 65536 || n < 1 || n > 0x7fffffffull || max_iter < 1 || max_iter > 4096 || v < 1 || v > 32) return BTC_ERR_SHAPE;
    if (v > KM_VMAX) return BTC_ERR_UNSUPPORTED;             // the pattern-space steps keep 2^v entries
    if (workspace_bytes < km_workspace_bytes(v, Kc)) return BTC_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return BTC_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    const int P = 1 << v;
    const uint32_t mask = (v == 32) ? 0xffffffffu : ((1u << v) - 1u);
    KmWorkspace w = km_carve(workspace, v, Kc);
    cudaError_t e = cudaMemsetAsync(workspace, 0, km_workspace_bytes(v, Kc), s);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaMemsetAsync(C_words, 0, (size_t)Kc * 4, s);
    if (e != cudaSuccess) return cuda_fail(e);
    const unsigned nb = (unsigned)((n + 255) / 256 < 148 * 32 ? (n + 255) / 256 : 148 * 32);
    const unsigned pb = (unsigned)((P + 255) / 256), kb = (unsigned)((Kc + 255) / 256);
    km_hist_kernel<<<nb, 256, 0, s>>>(vecs, n, mask, w.cnt);
    km_threshold_kernel<<<1, 1024, 0, s>>>(w.cnt, P, Kc, w.st);
    km_candidates_kernel<<<pb, 256, 0, s>>>(w.cnt, P, w.cand_p, w.cand_c, w.st);
    km_init_rank_kernel<<<(unsigned)((P + KM_RANK_THREADS - 1) / KM_RANK_THREADS), KM_RANK_THREADS, 0, s>>>(w.cand_p, w.cand_c, Kc, C_words, w.st);
    km_ties_kernel<<<1, 1024, 0, s>>>(w.cnt, P, Kc, C_words, w.st);
    for (int it = 0; it < max_iter; ++it) {
        km_estep_kernel<<<pb, 256, 0, s>>>(w.cnt, P, C_words, w.label, w.st);
        km_round_kernel<<<1, 1, 0, s>>>(w.st);
        km_vote_kernel<<<pb, 256, 0, s>>>(w.cnt, P, v, w.label, w.tot, w.ones, w.st);
        km_update_kernel<<<kb, 256, 0, s>>>(v, C_words, w.tot, w.ones, w.st);
    }
    km_assign_kernel<<<nb, 256, 0, s>>>(vecs, n, mask, P, w.label, z, info, w.st);
    return cuda_check_launch();
}
