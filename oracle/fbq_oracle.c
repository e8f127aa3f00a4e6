/*
 * CPU oracle for the FBQuant inference linear  --  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain definition of what the layer computes, written from
 * the paper, in IEEE double precision, with sequential sums in index order.
 * It exists so that the CUDA library can be checked against something that
 * can be verified by eye.  Nothing in the product path may call it; only the
 * tests, the smoke check and the benchmark's CPU-baseline leg do.  It shares
 * no code with the CUDA sources.
 *
 * What is computed (Algorithm 1, step 6: Z' = Q(W - BA) X^T + B A X^T, with
 * Sigma = B.A from Section 4.2, and W the out x in weight matrix of Section
 * 3.2), written for row-major tokens  y = Z'^T :
 *
 *     y[m][n] =  sum_k x[m][k] * ( s[n][k/group] * ( q[n][k] - z[n][k/group] ) )
 *              + sum_j ( sum_k x[m][k] * A[j][k] ) * B[n][j]
 *
 * q are the 3- or 4-bit codes of the group-wise linear quantiser (Algorithm 1
 * "linear quantizer", Section 5.1 "group size of 128"); s, z are the fp16
 * scale and zero point of each group of `group` consecutive input channels of
 * one output row.  The paper does not fix a storage format for the codes; the
 * packed formats below are this project's (see the comments at each packer).
 *
 * The feedback quantiser of Section 4.1 (oracle_quantize_feedback, below) is
 * pinned by a hand-worked group with ties, exact recovery of weights that lie
 * on a quantiser grid, the s/2 bound of Eq. "diff" in double precision, and
 * numpy's float16 conversion.
 *
 * Pins (tests/test_oracle_*.py): hand-worked 8x8 layer, literal packed words,
 * closed form for x = 1, numpy fp64 matmul special cases (rank 0, codes == zero
 * points), linearity, row permutation, token independence, MAC-count ratio
 * 2r/d of Section 3.2.  Accuracy on trained FBQuant weights: parity unpinned
 * (no checkpoints or calibration data are available to this build).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- exact widening of the 16-bit storage types ------------------------- */
static double half_bits_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int f = h & 0x3FF;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24);              /* subnormal: f * 2^-24            */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(f | 0x400), e - 25); /* (1024+f) * 2^(e-15-10)          */
    return sign ? -v : v;
}

static double bf16_bits_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double act_to_double(uint16_t bits, int act_is_bf16)
{
    return act_is_bf16 ? bf16_bits_to_double(bits) : half_bits_to_double(bits);
}

/* ---- packed formats ------------------------------------------------------
 * INT4: row n owns K/8 consecutive 32-bit words; code k sits in word k/8 at
 *       bits [4*(k%8), 4*(k%8)+3]  (little-endian nibbles).
 * INT3: row n owns 3*K/32 consecutive words; every run of 32 codes c[0..31]
 *       fills three words.  Word i (i = 0,1,2) holds ten codes as 3-bit fields,
 *       five per 16-bit half, and one bit of each of the two remaining codes:
 *          bits  3f .. 3f+2      (f = 0..4) : c[10i + f]
 *          bit   15                         : bit i of c[30]
 *          bits  16+3f .. 16+3f+2 (f = 0..4): c[10i + 5 + f]
 *          bit   31                         : bit i of c[31]
 */
void oracle_pack_int4(const uint8_t *codes, uint32_t *qweight, int N, int K)
{
    for (int n = 0; n < N; ++n)
        for (int w = 0; w < K / 8; ++w) {
            uint32_t word = 0;
            for (int e = 0; e < 8; ++e)
                word |= ((uint32_t)(codes[(size_t)n * K + 8 * w + e] & 0xF)) << (4 * e);
            qweight[(size_t)n * (K / 8) + w] = word;
        }
}

void oracle_pack_int3(const uint8_t *codes, uint32_t *qweight, int N, int K)
{
    const int runs = K / 32;
    for (int n = 0; n < N; ++n)
        for (int r = 0; r < runs; ++r) {
            const uint8_t *c = codes + (size_t)n * K + 32 * r;
            uint32_t *w = qweight + ((size_t)n * runs + r) * 3;
            for (int i = 0; i < 3; ++i) {
                uint32_t word = 0;
                for (int f = 0; f < 5; ++f) {
                    word |= ((uint32_t)(c[10 * i + f] & 7)) << (3 * f);
                    word |= ((uint32_t)(c[10 * i + 5 + f] & 7)) << (16 + 3 * f);
                }
                word |= ((uint32_t)((c[30] >> i) & 1)) << 15;
                word |= ((uint32_t)((c[31] >> i) & 1)) << 31;
                w[i] = word;
            }
        }
}

static int code_at(const uint32_t *qweight, int K, int bits, int n, int k)
{
    if (bits == 4) {
        uint32_t word = qweight[(size_t)n * (K / 8) + k / 8];
        return (int)((word >> (4 * (k % 8))) & 0xF);
    }
    /* bits == 3 */
    const uint32_t *w = qweight + ((size_t)n * (K / 32) + k / 32) * 3;
    int c = k % 32;
    if (c < 30) {
        int i = c / 10, f = c % 10;
        int shift = (f < 5) ? 3 * f : 16 + 3 * (f - 5);
        return (int)((w[i] >> shift) & 7);
    }
    int bitpos = (c == 30) ? 15 : 31;
    return (int)(((w[0] >> bitpos) & 1) | (((w[1] >> bitpos) & 1) << 1) | (((w[2] >> bitpos) & 1) << 2));
}

void oracle_unpack(const uint32_t *qweight, uint8_t *codes, int N, int K, int bits)
{
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k)
            codes[(size_t)n * K + k] = (uint8_t)code_at(qweight, K, bits, n, k);
}

/* w[n][k] = s[n][k/group] * (q[n][k] - z[n][k/group])   (dequantiser of the
 * group-wise linear quantiser; z is taken as any real number, not assumed
 * integral). */
void oracle_dequant(const uint32_t *qweight, const uint16_t *scales, const uint16_t *zeros,
                    double *W, int N, int K, int group, int bits)
{
    const int G = K / group;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            double s = half_bits_to_double(scales[(size_t)n * G + k / group]);
            double z = half_bits_to_double(zeros[(size_t)n * G + k / group]);
            W[(size_t)n * K + k] = s * ((double)code_at(qweight, K, bits, n, k) - z);
        }
}

/* The whole layer.  x: M x K, A: rank x K, B: N x rank (bit patterns of fp16,
 * or of bf16 when act_is_bf16), y: M x n_count doubles.  When n_list is NULL
 * every output row n = 0..N-1 is produced (n_count must equal N); otherwise only
 * the listed rows, in list order.  t_out (may be NULL) receives the unrounded
 * down-projection t = x.A^T, M x rank.  `threads` only spreads independent
 * output rows over cores; every sum is still sequential in index order.
 * Returns 0, or -1 on a malformed request. */
int oracle_linear(const uint16_t *x, const uint32_t *qweight, const uint16_t *scales,
                  const uint16_t *zeros, const uint16_t *A, const uint16_t *B, double *y,
                  double *t_out, int M, int N, int K, int group, int bits, int rank,
                  int act_is_bf16, const int *n_list, int n_count, int threads)
{
    if (M < 0 || N <= 0 || K <= 0 || group <= 0 || K % group || (bits != 3 && bits != 4) || rank < 0)
        return -1;
    if (bits == 4 ? (K % 8) : (K % 32))
        return -1;
    if (rank > 0 && (!A || !B))
        return -1;
    if (!n_list && n_count != N)
        return -1;
    const int G = K / group;
    if (threads < 1)
        threads = 1;

    double *xd = (double *)malloc(sizeof(double) * (size_t)(M > 0 ? M : 1) * K);
    double *t = (double *)calloc((size_t)(M > 0 ? M : 1) * (rank > 0 ? rank : 1), sizeof(double));
    if (!xd || !t) {
        free(xd);
        free(t);
        return -1;
    }
    for (size_t i = 0; i < (size_t)M * K; ++i)
        xd[i] = act_to_double(x[i], act_is_bf16);

    /* down-projection  t[m][j] = sum_k x[m][k] A[j][k]   (not rounded) */
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int j = 0; j < rank; ++j)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k)
                acc += xd[(size_t)m * K + k] * act_to_double(A[(size_t)j * K + k], act_is_bf16);
            t[(size_t)m * rank + j] = acc;
        }
    if (t_out)
        memcpy(t_out, t, sizeof(double) * (size_t)M * rank);

#pragma omp parallel for num_threads(threads) schedule(dynamic, 4)
    for (int i = 0; i < n_count; ++i) {
        const int n = n_list ? n_list[i] : i;
        double *wrow = (double *)malloc(sizeof(double) * (size_t)K);
        for (int k = 0; k < K; ++k) {
            double s = half_bits_to_double(scales[(size_t)n * G + k / group]);
            double z = half_bits_to_double(zeros[(size_t)n * G + k / group]);
            wrow[k] = s * ((double)code_at(qweight, K, bits, n, k) - z);
        }
        for (int m = 0; m < M; ++m) {
            double main_acc = 0.0;
            for (int k = 0; k < K; ++k)
                main_acc += xd[(size_t)m * K + k] * wrow[k];
            double sub = 0.0;
            for (int j = 0; j < rank; ++j)
                sub += t[(size_t)m * rank + j] * act_to_double(B[(size_t)n * rank + j], act_is_bf16);
            y[(size_t)m * n_count + i] = main_acc + sub;
        }
        free(wrow);
    }
    free(xd);
    free(t);
    return 0;
}

/* ---- feedback quantiser (Section 4.1) --------------------------------------
 * The main path of FBQuant stores Q(W - Sigma), Sigma = B.A, so that the
 * reconstructed weight  W_F = Q(W - Sigma) + Sigma  stays within s/2 of W
 * (Eq. "diff" and the bound below it, for a round-to-nearest Q).  The paper
 * says only "linear quantizer", group size 128, round-to-nearest with scaling
 * factor s; the reading taken here (asymmetric min-max per group) is:
 *
 *   r[n][k]   = W[n][k] - sum_j B[n][j]*A[j][k]          (the fed-back residual)
 *   per group g of `group` consecutive k of one row, with maxq = 2^bits - 1:
 *     mn = min r, mx = max r
 *     s  = max((mx - mn)/maxq, 2^-14),  z = rint(-mn/s)                if mx > mn
 *     s  = max(|mn|, 2^-14),            z = 1 if mn < 0 else 0         if mx == mn
 *     s, z are stored as fp16 (round to nearest even); everything below uses
 *     the STORED values, so that dequantisation inverts exactly what was coded
 *   q[n][k]   = clamp(rint(r/s + z), 0, maxq)            (ties to even)
 *   W_F[n][k] = s*(q - z) + Sigma[n][k]
 *
 * A rounding decides every code, so this function works in the arithmetic of
 * the device kernel it checks, IEEE single precision with the operations in
 * exactly this order: Sigma by fused multiply-adds over j ascending from 0,
 * one subtraction for r, one division and one addition before rint, one
 * multiplication and one addition for W_F.  (The bound itself is checked by
 * the tests in double precision from the stored s, z and q.)
 * W: N x K floats.  A: rank x K, B: N x rank: fp16 bit patterns (ab_kind 0), bf16 bit
 * patterns (1) or floats (2, the master copies of the reconstruction loop); may be NULL
 * when rank == 0.  r_out, wf_out: N x K floats, may be NULL.
 * Returns 0, or -1 on a malformed request. */
static uint16_t float_to_half_bits(float f)
{
    /* round to nearest even, with subnormals, overflow to infinity */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    const uint32_t mag = u & 0x7FFFFFFFu;
    if (mag >= 0x7F800000u) return (uint16_t)(sign | (mag > 0x7F800000u ? 0x7E00u : 0x7C00u));
    if (mag >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u);        /* >= 65520 rounds to infinity */
    if (mag < 0x33000001u) return sign;                               /* <= 2^-25 rounds to zero     */
    int e = (int)(mag >> 23) - 127;                                   /* unbiased exponent            */
    uint32_t m = (mag & 0x7FFFFFu) | 0x800000u;                       /* 24-bit significand           */
    int shift = (e < -14) ? (13 + (-14 - e)) : 13;                    /* bits dropped                 */
    uint32_t kept = m >> shift, rem = m & ((1u << shift) - 1u), half = 1u << (shift - 1);
    if (rem > half || (rem == half && (kept & 1u))) ++kept;
    if (e < -14) return (uint16_t)(sign | kept);                      /* subnormal (may carry to the first normal) */
    return (uint16_t)(sign | (uint16_t)(((uint32_t)(e + 15) << 10) + (kept - 0x400u)));
}

/* element i of a sub-branch matrix: fp16 (kind 0) or bf16 (kind 1) bit patterns, or floats (kind 2) */
static float ab_elem(const void *p, size_t i, int kind)
{
    if (kind == 2) return ((const float *)p)[i];
    return (float)act_to_double(((const uint16_t *)p)[i], kind == 1);
}

int oracle_quantize_feedback(const float *W, const void *A, const void *B, uint8_t *codes,
                             uint16_t *scales, uint16_t *zeros, float *r_out, float *wf_out, int N,
                             int K, int group, int bits, int rank, int ab_kind)
{
    if (N < 1 || K < 1 || group < 1 || K % group != 0 || rank < 0 || (bits != 3 && bits != 4)) return -1;
    if (rank > 0 && (!A || !B)) return -1;
    const int G = K / group;
    const float maxq = (float)((1 << bits) - 1);
    const float smin = ldexpf(1.0f, -14);
    float *sig = (float *)malloc(sizeof(float) * (size_t)group);
    float *r = (float *)malloc(sizeof(float) * (size_t)group);
    if (!sig || !r) { free(sig); free(r); return -1; }
    for (int n = 0; n < N; ++n)
        for (int g = 0; g < G; ++g) {
            float mn = INFINITY, mx = -INFINITY;
            for (int i = 0; i < group; ++i) {
                const int k = g * group + i;
                float acc = 0.0f;
                for (int j = 0; j < rank; ++j)
                    acc = fmaf(ab_elem(B, (size_t)n * rank + j, ab_kind), ab_elem(A, (size_t)j * K + k, ab_kind), acc);
                sig[i] = acc;
                r[i] = W[(size_t)n * K + k] - acc;
                if (r[i] < mn) mn = r[i];
                if (r[i] > mx) mx = r[i];
            }
            float s, z;
            if (mx > mn) {
                s = (mx - mn) / maxq;
                if (s < smin) s = smin;
                const float sh = (float)half_bits_to_double(float_to_half_bits(s));
                z = rintf(-mn / sh);
            } else {
                s = fabsf(mn);
                if (s < smin) s = smin;
                z = (mn < 0.0f) ? 1.0f : 0.0f;
            }
            const uint16_t s_bits = float_to_half_bits(s), z_bits = float_to_half_bits(z);
            const float sh = (float)half_bits_to_double(s_bits), zh = (float)half_bits_to_double(z_bits);
            scales[(size_t)n * G + g] = s_bits;
            zeros[(size_t)n * G + g] = z_bits;
            for (int i = 0; i < group; ++i) {
                const size_t idx = (size_t)n * K + (size_t)g * group + i;
                const float t = r[i] / sh;
                float q = rintf(t + zh);
                if (q < 0.0f) q = 0.0f;
                if (q > maxq) q = maxq;
                codes[idx] = (uint8_t)q;
                if (r_out) r_out[idx] = r[i];
                if (wf_out) {
                    const float wq = sh * (q - zh);
                    wf_out[idx] = wq + sig[i];
                }
            }
        }
    free(sig);
    free(r);
    return 0;
}

/* fp16 bit patterns (round to nearest even) of n floats: lets the tests pin the
 * conversion above against numpy's. */
void oracle_float_to_half(const float *in, uint16_t *out, int n)
{
    for (int i = 0; i < n; ++i) out[i] = float_to_half_bits(in[i]);
}

/* Widen n stored 16-bit values to double (lets the tests check the two
 * conversions above against numpy over all 65536 bit patterns). */
void oracle_widen(const uint16_t *bits, double *out, int n, int act_is_bf16)
{
    for (int i = 0; i < n; ++i)
        out[i] = act_to_double(bits[i], act_is_bf16);
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
