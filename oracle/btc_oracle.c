/*
 * CPU oracle for the codebook-binary linear layer (BTC-LLM inference path).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or
 * constant with the CUDA path and must never be called from the product path;
 * only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Everything is fp64 and follows the paper's definitions literally, with no
 * blocking, fusion or reordering:
 *
 *   storage      W[r, j*v:(j+1)*v] = C[I[r,j]]            (appendix "Binary codebook
 *                                                          LUT-GEMM", first display)
 *   dequantise   W^ = alpha * B^ + mu  (row-wise alpha,mu) (Algorithm "Binary
 *                                                          Transformation and Compression",
 *                                                          step "Dequantize"; Eq. 2)
 *   result       y_r = sum_j <x_j, C[I[r,j]]>              (appendix, second display)
 *   LUT form     Stage-I LUT, Stage-II CBLUT, index gather (appendix, Stage-I/Stage-II)
 *   bit map      b = (B + 1) / 2                           (Algorithm "Efficient Binary
 *                                                          Vector Packing and Unpacking")
 *   distance     ||b - c||^2 = 4 * d_H(b, c)               (Section 4.1, E-step)
 *   storage cost v*c + ceil(log2 c) * m*n / v bits         (Section 4.3)
 *
 * Pinned by tests/test_oracle_*.py against hand-expanded tiny cases, closed
 * forms and textbook special cases.  The optional activation transform
 * (btc_oracle_transform) is pinned only by algebraic identities: the paper
 * prints no worked example, so with respect to the authors' factor-order
 * convention it is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int btc_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* B^[r, j*v + t] = C[I[r,j]][t]  -- the storage rule, one element at a time. */
int btc_oracle_decode_pm1(const uint16_t *idx, const int8_t *C, int N, int K, int v, int Kc,
                          int8_t *B)
{
    if (v <= 0 || K % v) return 2;
    const int Kb = K / v;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int r = 0; r < N; ++r)
        for (int j = 0; j < Kb; ++j) {
            const int k = idx[(size_t)r * Kb + j];
            if (k >= Kc) { bad |= 1; continue; }
            for (int t = 0; t < v; ++t)
                B[(size_t)r * K + (size_t)j * v + t] = C[(size_t)k * v + t] >= 0 ? 1 : -1;
        }
    return bad ? 3 : 0;
}

/* W^[r,k] = alpha_r * B^[r,k] + mu_r   (mu may be NULL = 0). */
void btc_oracle_dense_weight(const int8_t *B, const double *alpha, const double *mu, int N, int K,
                             double *W)
{
#pragma omp parallel for schedule(static)
    for (int r = 0; r < N; ++r)
        for (int k = 0; k < K; ++k)
            W[(size_t)r * K + k] = alpha[r] * (double)B[(size_t)r * K + k] + (mu ? mu[r] : 0.0);
}

/* y[m,n] = sum_k x[m,k] * W[n,k], k ascending: the textbook triple loop. */
void btc_oracle_matmul_nt(const double *x, const double *W, int M, int N, int K, double *y)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            double s = 0.0;
            for (int k = 0; k < K; ++k) s += x[(size_t)m * K + k] * W[(size_t)n * K + k];
            y[(size_t)m * N + n] = s;
        }
}

/* The layer: decode to a dense fp64 matrix, then the naive product.
 * Bout (int8 [N,K]) receives the +-1 matrix when not NULL. */
int btc_oracle_linear(const double *x, const uint16_t *idx, const int8_t *C, const double *alpha,
                      const double *mu, int M, int N, int K, int v, int Kc, double *y, int8_t *Bout)
{
    int8_t *B = Bout ? Bout : (int8_t *)malloc((size_t)N * K);
    double *W = (double *)malloc(sizeof(double) * (size_t)N * K);
    if (!B || !W) { if (!Bout) free(B); free(W); return 1; }
    int rc = btc_oracle_decode_pm1(idx, C, N, K, v, Kc, B);
    if (rc == 0) {
        btc_oracle_dense_weight(B, alpha, mu, N, K, W);
        btc_oracle_matmul_nt(x, W, M, N, K, y);
    }
    if (!Bout) free(B);
    free(W);
    return rc;
}

/*
 * The paper's two-stage lookup scheme restated literally (one activation row
 * at a time).  seg = the segment length (the appendix calls it mu; renamed here
 * because mu is also the row mean); P = v / seg.
 *   Stage-I   LUT[j][p][s]  = sum_t sigma_t(s) * x_{j,p}[t],  sigma_t(s) = +1 if bit t of s is set
 *   Stage-II  key[k][p]     = the seg-bit pattern of C_k[p*seg:(p+1)*seg]  (offline)
 *             CBLUT[j][k]   = sum_p LUT[j][p][key[k][p]]
 *   gather    y_r           = sum_j CBLUT[j][I[r,j]]
 * followed by the row-wise dequantisation  alpha_r * y_r + mu_r * sum_k x_k.
 */
int btc_oracle_lut_linear(const double *x, const uint16_t *idx, const int8_t *C,
                          const double *alpha, const double *mu, int M, int N, int K, int v, int Kc,
                          int seg, double *y)
{
    if (v <= 0 || K % v || seg <= 0 || seg > 16 || v % seg) return 2;
    const int Kb = K / v, P = v / seg, S = 1 << seg;
    uint32_t *key = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)Kc * P);
    double *lut = (double *)malloc(sizeof(double) * (size_t)P * S);
    double *cblut = (double *)malloc(sizeof(double) * (size_t)Kc);
    double *acc = (double *)malloc(sizeof(double) * (size_t)N);
    if (!key || !lut || !cblut || !acc) { free(key); free(lut); free(cblut); free(acc); return 1; }
    for (int k = 0; k < Kc; ++k)
        for (int p = 0; p < P; ++p) {
            uint32_t s = 0;
            for (int t = 0; t < seg; ++t)
                if (C[(size_t)k * v + p * seg + t] >= 0) s |= 1u << t;
            key[(size_t)k * P + p] = s;
        }
    int rc = 0;
    for (int m = 0; m < M && rc == 0; ++m) {
        const double *xm = x + (size_t)m * K;
        double sumx = 0.0;
        for (int k = 0; k < K; ++k) sumx += xm[k];
        for (int r = 0; r < N; ++r) acc[r] = 0.0;
        for (int j = 0; j < Kb; ++j) {
            for (int p = 0; p < P; ++p)
                for (int s = 0; s < S; ++s) {
                    double e = 0.0;
                    for (int t = 0; t < seg; ++t) {
                        const double xv = xm[(size_t)j * v + p * seg + t];
                        e += ((s >> t) & 1) ? xv : -xv;
                    }
                    lut[(size_t)p * S + s] = e;
                }
            for (int k = 0; k < Kc; ++k) {
                double e = 0.0;
                for (int p = 0; p < P; ++p) e += lut[(size_t)p * S + key[(size_t)k * P + p]];
                cblut[k] = e;
            }
            for (int r = 0; r < N; ++r) {
                const int k = idx[(size_t)r * Kb + j];
                if (k >= Kc) { rc = 3; break; }
                acc[r] += cblut[k];
            }
            if (rc) break;
        }
        for (int r = 0; r < N; ++r)
            y[(size_t)m * N + r] = alpha[r] * acc[r] + (mu ? mu[r] * sumx : 0.0);
    }
    free(key); free(lut); free(cblut); free(acc);
    return rc;
}

/* Public packed form: bit t (LSB first) of word k is (C[k][t] + 1) / 2; C >= 0 counts as +1
 * (sign(0) = +1, Section 4.1 M-step). */
void btc_oracle_pack_codebook(const int8_t *C, int Kc, int v, uint32_t *packed)
{
    for (int k = 0; k < Kc; ++k) {
        uint32_t w = 0;
        for (int t = 0; t < v; ++t)
            if (C[(size_t)k * v + t] >= 0) w |= 1u << t;
        packed[k] = w;
    }
}

/* Squared Euclidean distance between two +-1 vectors, summed term by term. */
double btc_oracle_sqdist_pm1(const int8_t *b, const int8_t *c, int v)
{
    double s = 0.0;
    for (int t = 0; t < v; ++t) {
        const double d = (double)(b[t] >= 0 ? 1 : -1) - (double)(c[t] >= 0 ? 1 : -1);
        s += d * d;
    }
    return s;
}

static int ceil_log2(int c)
{
    int b = 0;
    while ((1L << b) < c) ++b;
    return b;
}

/* Storage cost in bits of one layer, Section 4.3: v*c + ceil(log2 c) * m*n / v. */
double btc_oracle_storage_bits(int N, int K, int v, int Kc)
{
    return (double)v * Kc + (double)ceil_log2(Kc) * ((double)N * K / v);
}

/*
 * Dense index packing (Section 4.3 counts ceil(log2 c) bits per index: "v*c + ceil(log2 c) * mn/v").
 * Row n of the packed matrix is the little-endian bit string of its K/v indices, `bits` bits each:
 * bit q of index j is bit j*bits + q of the row, and bit p of the row is bit p % 8 of byte p / 8.
 * Rows start every `pitch` bytes (pitch >= ceil(Kb*bits/8)); bytes between the end of the bit string and
 * the pitch are zero.  Written bit by bit on purpose.
 */
int btc_oracle_pack_indices(const uint16_t *idx, int N, int Kb, int bits, size_t pitch, uint8_t *out)
{
    if (bits < 1 || bits > 16 || pitch * 8 < (size_t)Kb * bits) return 2;
    memset(out, 0, pitch * (size_t)N);
    for (int n = 0; n < N; ++n)
        for (int j = 0; j < Kb; ++j) {
            const unsigned val = idx[(size_t)n * Kb + j];
            if (bits < 16 && (val >> bits)) return 3;
            for (int q = 0; q < bits; ++q) {
                const size_t p = (size_t)j * bits + q;
                if ((val >> q) & 1u) out[(size_t)n * pitch + p / 8] |= (uint8_t)(1u << (p % 8));
            }
        }
    return 0;
}

int btc_oracle_unpack_indices(const uint8_t *in, int N, int Kb, int bits, size_t pitch, uint16_t *idx)
{
    if (bits < 1 || bits > 16 || pitch * 8 < (size_t)Kb * bits) return 2;
    for (int n = 0; n < N; ++n)
        for (int j = 0; j < Kb; ++j) {
            unsigned val = 0;
            for (int q = 0; q < bits; ++q) {
                const size_t p = (size_t)j * bits + q;
                if ((in[(size_t)n * pitch + p / 8] >> (p % 8)) & 1u) val |= 1u << q;
            }
            idx[(size_t)n * Kb + j] = (uint16_t)val;
        }
    return 0;
}

/*
 * Bits per weight.  mode 0 "nominal": log2(Kc)/v; mode 1 "container": ceil(log2 Kc)/v (the paper's
 * accounting); mode 2 "stored": 16/v (uint16 indices as this library keeps them).  Adds the row
 * scales (scale_bits_per_row / K) and, when with_codebook != 0, the codebook v*Kc/(N*K).
 */
double btc_oracle_bits_per_weight(int N, int K, int v, int Kc, int scale_bits_per_row, int mode,
                                  int with_codebook)
{
    double idx_bits;
    if (mode == 0) idx_bits = log2((double)Kc);
    else if (mode == 1) idx_bits = (double)ceil_log2(Kc);
    else idx_bits = 16.0;
    double b = idx_bits / v + (double)scale_bits_per_row / K;
    if (with_codebook) b += (double)v * Kc / ((double)N * K);
    return b;
}

/*
 * Online activation transform  x' = x * T,  T = D * P,  D = diag(sigma) (+-1),  P = P1 (x) P2
 * (Section 4.2, "Transformation Pair"; applied on the fly as X <- X T).  Written as the dense
 * K x K Kronecker matrix: P[(a*k2 + b), (c*k2 + d)] = P1[a,c] * P2[b,d].
 */
int btc_oracle_transform(const double *x, const int8_t *sigma, const double *P1, const double *P2,
                         int M, int k1, int k2, double *xt)
{
    const int K = k1 * k2;
    double *T = (double *)malloc(sizeof(double) * (size_t)K * K);
    if (!T) return 1;
    for (int a = 0; a < k1; ++a)
        for (int b = 0; b < k2; ++b)
            for (int c = 0; c < k1; ++c)
                for (int d = 0; d < k2; ++d) {
                    const int i = a * k2 + b, o = c * k2 + d;
                    T[(size_t)i * K + o] = (sigma[i] >= 0 ? 1.0 : -1.0) * P1[a * k1 + c] * P2[b * k2 + d];
                }
    for (int m = 0; m < M; ++m)
        for (int o = 0; o < K; ++o) {
            double s = 0.0;
            for (int i = 0; i < K; ++i) s += x[(size_t)m * K + i] * T[(size_t)i * K + o];
            xt[(size_t)m * K + o] = s;
        }
    free(T);
    return 0;
}
