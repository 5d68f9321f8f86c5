// Codebook packing, sign-matrix decode and index validation kernels (offline / checking helpers).
#include <cstdlib>
#include "btc_internal.cuh"

namespace btc {

// Kernel-private word of one centroid for the decode path ("MMA layout"): the bit of weight t sits
// at (t & 1) * 16 + P0 + (t >> 1) with P0 = 12 - v/2, so that `word & mask` with one bit kept per
// 16-bit half is a pair of fp16 numbers {0, 2^(pos-24)}.  Defined for v % 4 == 0, v <= 24; 0 otherwise.
__host__ __device__ inline uint32_t mma_layout_word(uint32_t pub, int v)
{
    if (v % 4 != 0 || v > 24) return 0u;
    const int p0 = 12 - v / 2;
    uint32_t w = 0;
    for (int t = 0; t < v; ++t)
        if ((pub >> t) & 1u) w |= 1u << ((t & 1) * 16 + p0 + (t >> 1));
    return w;
}

// Kernel-private word of one centroid for the integer-MMA decode path ("byte-lane layout"): the bit of
// weight t sits at bit (t >> 2) of byte (t & 3), so `word & (0x01010101 << c)` is four unsigned bytes
// {0 or 2^c} for the weights 4c .. 4c+3.
__host__ __device__ inline uint32_t byte_lane_word(uint32_t pub, int v)
{
    uint32_t w = 0;
    for (int t = 0; t < v; ++t)
        if ((pub >> t) & 1u) w |= 1u << (8 * (t & 3) + (t >> 2));
    return w;
}

// The byte-lane word squeezed into 16 bits for codebooks too large to sit in shared memory as 32-bit words
// (v <= 16): nibble q of the result is the low nibble of byte {0, 2, 1, 3}[q] of the byte-lane word, so that
// `h | (h << 12)` has the low nibble of every byte in place (the high nibbles carry leftovers, which the kernel's
// masks never look at).  0 for v > 16.
__host__ __device__ inline uint16_t byte_lane_half(uint32_t pub, int v)
{
    if (v > 16) return 0;
    const uint32_t w = byte_lane_word(pub, v);
    return (uint16_t)((w & 0xFu) | (((w >> 16) & 0xFu) << 4) | (((w >> 8) & 0xFu) << 8) | (((w >> 24) & 0xFu) << 12));
}

// bit t of out[k] = (C[k][t] + 1) / 2, with C >= 0 read as +1; private words at out[Kc4 + k], out[2 Kc4 + k] and, as
// 16-bit halves, from out[3 Kc4].
__global__ void pack_codebook_kernel(const int8_t *__restrict__ C, int Kc, int v, uint32_t *__restrict__ out)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    const int Kc4 = (Kc + 3) / 4 * 4;
    if (k >= Kc4) return;
    uint32_t w = 0;
    if (k < Kc)
        for (int t = 0; t < v; ++t)
            if (C[(size_t)k * v + t] >= 0) w |= 1u << t;
    out[k] = w;
    out[Kc4 + k] = mma_layout_word(w, v);
    out[2 * Kc4 + k] = byte_lane_word(w, v);
    uint16_t *half = reinterpret_cast<uint16_t *>(out + 3 * (size_t)Kc4);   // (Kc + 7) / 8 * 8 entries: a whole number of 16 bytes
    half[k] = byte_lane_half(w, v);
    if (k < (Kc + 7) / 8 * 8 - Kc4) half[Kc4 + k] = 0;
}

// One thread per (row, block): expands the centroid word into v int8 signs.
__global__ void decode_pm1_kernel(const uint16_t *__restrict__ idx, const uint32_t *__restrict__ Cp,
                                  size_t blocks, int Kb, int v, int8_t *__restrict__ B)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= blocks) return;
    const uint32_t w = Cp[idx[i]];
    int8_t *dst = B + i * (size_t)v;   // row n = i / Kb, block j = i % Kb: offset n*K + j*v = i*v
    for (int t = 0; t < v; ++t) dst[t] = ((w >> t) & 1u) ? 1 : -1;
    (void)Kb;
}

__global__ void validate_indices_kernel(const uint16_t *__restrict__ idx, size_t count, int Kc, int *bad)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    int local = 0;
    for (; i < count; i += stride) local += (idx[i] >= Kc) ? 1 : 0;
    for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
    if ((threadIdx.x & 31) == 0 && local) atomicAdd(bad, local);
}

// Dense index packing: row n of the output is the little-endian bit string of its Kb indices, `bits` bits each
// (Section 4.3 counts ceil(log2 c) bits per index).  One thread per 32-bit word of a packed row: it collects the
// fields that overlap its 32 bits.  Words past the bit string (row padding) are written as zeros.
__global__ void index_pack_kernel(const uint16_t *__restrict__ idx, int N, int Kb, int bits, int pitch_words,
                                  uint32_t *__restrict__ out)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)N * pitch_words) return;
    const int n = (int)(i / pitch_words), w = (int)(i % pitch_words);
    const long long b0 = 32ll * w, b1 = b0 + 32;              // this word's bit range of the row
    uint32_t word = 0;
    for (long long j = b0 / bits; j < Kb && j * bits < b1; ++j) {
        const uint32_t val = idx[(size_t)n * Kb + j] & ((1u << bits) - 1u);
        const long long sh = j * bits - b0;                   // position of the field's bit 0 in this word (may be < 0)
        word |= sh >= 0 ? (val << sh) : (val >> (-sh));
    }
    out[i] = word;
}

__global__ void index_unpack_kernel(const uint32_t *__restrict__ in, int N, int Kb, int bits, int pitch_words,
                                    uint16_t *__restrict__ idx)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)N * Kb) return;
    const int n = (int)(i / Kb), j = (int)(i % Kb);
    const long long bit = (long long)j * bits;
    const uint32_t *row = in + (size_t)n * pitch_words;
    const int w = (int)(bit >> 5), sh = (int)(bit & 31);
    uint64_t two = row[w];
    if (sh + bits > 32) two |= (uint64_t)row[w + 1] << 32;   // (only read when the field really crosses the word)
    idx[i] = (uint16_t)((two >> sh) & ((1u << bits) - 1u));
}

// Debug aid (switched on by the environment variable BTC_DEBUG_CHECK_INDICES=1): raises a status word when an index is
// >= Kc.  No trap, no assert: the layer kernels still run (their result is then undefined), the context stays usable and
// btc_device_status reports BTC_ERR_INDEX.
__device__ int g_index_status = 0;

__global__ void flag_bad_indices_kernel(const uint16_t *__restrict__ idx, size_t count, int Kc)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (; i < count; i += stride) bad |= idx[i] >= Kc;
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicExch(&g_index_status, (int)BTC_ERR_INDEX);
}

bool debug_check_indices_enabled()
{
    static int on = -1;
    if (on < 0) {
        const char *e = getenv("BTC_DEBUG_CHECK_INDICES");
        on = (e && e[0] && e[0] != '0') ? 1 : 0;
    }
    return on == 1;
}

int launch_index_check(const uint16_t *idx, size_t count, int Kc, cudaStream_t s)
{
    if (Kc >= 65536 || count == 0) return BTC_OK;             // every 16-bit value is a valid index
    size_t grid = (count + 255) / 256;
    if (grid > 148 * 8) grid = 148 * 8;
    flag_bad_indices_kernel<<<(unsigned)grid, 256, 0, s>>>(idx, count, Kc);
    return cuda_check_launch();
}

int index_status_read(int *out)
{
    int v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, g_index_status, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    *out = v;
    return BTC_OK;
}

int index_status_reset()
{
    const int zero = 0;
    cudaError_t e = cudaMemcpyToSymbol(g_index_status, &zero, sizeof(int));
    return e == cudaSuccess ? BTC_OK : cuda_fail(e);
}

}  // namespace btc

using namespace btc;

extern "C" int btc_codebook_pack(const int8_t *C_pm1, int Kc, int v, uint32_t *C_packed, void *stream)
{
    if (!C_pm1 || !C_packed) return BTC_ERR_NULL;
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536) return BTC_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(C_packed) % 16) return BTC_ERR_ALIGN;
    pack_codebook_kernel<<<(Kc + 3 + 127) / 128, 128, 0, (cudaStream_t)stream>>>(C_pm1, Kc, v, C_packed);
    return cuda_check_launch();
}

extern "C" int btc_codebook_pack_host(const int8_t *C, int Kc, int v, uint32_t *out)
{
    if (!C || !out) return BTC_ERR_NULL;
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536) return BTC_ERR_SHAPE;
    const int Kc4 = (Kc + 3) / 4 * 4;
    for (int k = 0; k < Kc4; ++k) {
        uint32_t w = 0;
        if (k < Kc)
            for (int t = 0; t < v; ++t)
                if (C[(size_t)k * v + t] >= 0) w |= 1u << t;
        out[k] = w;
        out[Kc4 + k] = mma_layout_word(w, v);
        out[2 * Kc4 + k] = byte_lane_word(w, v);
        uint16_t *half = reinterpret_cast<uint16_t *>(out + 3 * (size_t)Kc4);
        half[k] = byte_lane_half(w, v);
        if (k < (Kc + 7) / 8 * 8 - Kc4) half[Kc4 + k] = 0;
    }
    return BTC_OK;
}

extern "C" int btc_decode_pm1(const uint16_t *idx, const uint32_t *C_packed, int N, int K, int v, int Kc,
                              int8_t *B_out, void *stream)
{
    if (!idx || !C_packed || !B_out) return BTC_ERR_NULL;
    if (v < 1 || v > 32 || Kc < 1 || Kc > 65536 || N < 1 || K < 1 || K % v) return BTC_ERR_SHAPE;
    const size_t blocks = (size_t)N * (K / v);
    const size_t grid = (blocks + 255) / 256;
    if (grid > 0x7fffffffull) return BTC_ERR_SHAPE;
    decode_pm1_kernel<<<(unsigned)grid, 256, 0, (cudaStream_t)stream>>>(idx, C_packed, blocks, K / v, v, B_out);
    return cuda_check_launch();
}

extern "C" int btc_validate_indices(const uint16_t *idx, size_t count, int Kc, int *bad_count, void *stream)
{
    if (!idx || !bad_count) return BTC_ERR_NULL;
    if (Kc < 1 || Kc > 65536) return BTC_ERR_SHAPE;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(bad_count, 0, sizeof(int), s);
    if (e != cudaSuccess) return cuda_fail(e);
    if (count == 0) return BTC_OK;
    size_t grid = (count + 255) / 256;
    if (grid > 148 * 16) grid = 148 * 16;
    validate_indices_kernel<<<(unsigned)grid, 256, 0, s>>>(idx, count, Kc, bad_count);
    return cuda_check_launch();
}

extern "C" int btc_index_bits(int Kc)
{
    if (Kc < 1 || Kc > 65536) return 0;
    int b = 1;
    while ((1 << b) < Kc) ++b;
    return b;
}

extern "C" size_t btc_index_packed_row_bytes(int Kb, int Kc)
{
    const int b = btc_index_bits(Kc);
    if (b == 0 || Kb < 1) return 0;
    return (((size_t)Kb * b + 7) / 8 + 15) / 16 * 16;
}

extern "C" int btc_index_pack(const uint16_t *idx, int N, int Kb, int Kc, void *packed, void *stream)
{
    if (!idx || !packed) return BTC_ERR_NULL;
    const int bits = btc_index_bits(Kc);
    if (bits == 0 || N < 1 || Kb < 1) return BTC_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(packed) % 16) return BTC_ERR_ALIGN;
    const int pw = (int)(btc_index_packed_row_bytes(Kb, Kc) / 4);
    const size_t total = (size_t)N * pw, grid = (total + 255) / 256;
    if (grid > 0x7fffffffull) return BTC_ERR_SHAPE;
    index_pack_kernel<<<(unsigned)grid, 256, 0, (cudaStream_t)stream>>>(idx, N, Kb, bits, pw, static_cast<uint32_t *>(packed));
    return cuda_check_launch();
}

extern "C" int btc_index_unpack(const void *packed, int N, int Kb, int Kc, uint16_t *idx, void *stream)
{
    if (!idx || !packed) return BTC_ERR_NULL;
    const int bits = btc_index_bits(Kc);
    if (bits == 0 || N < 1 || Kb < 1) return BTC_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(packed) % 16) return BTC_ERR_ALIGN;
    const int pw = (int)(btc_index_packed_row_bytes(Kb, Kc) / 4);
    const size_t total = (size_t)N * Kb, grid = (total + 255) / 256;
    if (grid > 0x7fffffffull) return BTC_ERR_SHAPE;
    index_unpack_kernel<<<(unsigned)grid, 256, 0, (cudaStream_t)stream>>>(static_cast<const uint32_t *>(packed), N, Kb, bits, pw, idx);
    return cuda_check_launch();
}
