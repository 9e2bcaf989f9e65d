/*
 * CPU oracle for the weight-only quantised linear layer -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, obviously-correct C.  It shares no code with the CUDA library
 * and the library never calls it; only the tests, the smoke check and the
 * benchmark's cpu_baseline leg execute it.
 *
 * What it computes (paper Section 4.2: FP16 activations, per-channel int8 for
 * the attention projections, int4 for the feed-forward/embedding weights;
 * Section 3.7: the dequantisation belongs to the linear operator; Section 3.1:
 * weights are O x I, i.e. N x K here).  Group size 32 along K for int4 is the
 * benchmark's choice (the paper's Section 5 calls it sub-channel quantisation).
 *
 *   w[n,k]   = fp16(s[n, k / G]) * q[n,k]                      exact in fp64
 *   y64[m,n] = sum over k ascending of fp16(x[m,k]) * w[n,k]   fp64 accumulate
 *   A[m,n]   = sum over k of | fp16(x[m,k]) * w[n,k] |         tolerance denominator
 *   y16[m,n] = y64[m,n] rounded to nearest-even fp16 (overflow -> inf)
 *
 * The three loops are written out; there is no blocking or reordering.
 * Parity pins (tests/test_oracle_pins.py): hand-computed worked examples,
 * brute force over all byte values, one-hot / zero / all-ones closed forms,
 * power-of-two scaling and negation invariants, agreement with a library fp64
 * matmul, and a double-rounding trap for the fp16 conversion.
 */
#include <stdint.h>
#include <string.h>
#include <stdlib.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Two's-complement nibble pair -> two integers in [-8, 7].
 * Canonical interchange form: byte j of a row = (q[2j] & 0xF) | ((q[2j+1] & 0xF) << 4). */
void oracle_unpack_nibbles(const uint8_t* bytes, int64_t n_bytes, int8_t* q)
{
    for (int64_t j = 0; j < n_bytes; ++j) {
        int lo = bytes[j] & 0xF, hi = (bytes[j] >> 4) & 0xF;
        q[2 * j]     = (int8_t)(lo < 8 ? lo : lo - 16);
        q[2 * j + 1] = (int8_t)(hi < 8 ? hi : hi - 16);
    }
}

/* IEEE binary16 bit pattern -> double (exact). */
double oracle_fp16_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1, e = (h >> 10) & 0x1F, f = h & 0x3FF;
    double v;
    if (e == 0)       v = ldexp((double)f, -24);                 /* zero / subnormal */
    else if (e == 31) v = f ? NAN : INFINITY;
    else              v = ldexp((double)(1024 + f), e - 25);
    return sign ? -v : v;
}

/* double -> IEEE binary16 bit pattern, one rounding, nearest-even, overflow -> inf. */
uint16_t oracle_double_to_fp16(double v)
{
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (isnan(a)) return (uint16_t)(sign | 0x7E00);
    if (a == 0.0) return sign;
    int e;
    frexp(a, &e);                     /* a = m * 2^e, m in [0.5, 1) */
    int ulp_exp = e - 11;             /* 11 significant bits for normals */
    if (ulp_exp < -24) ulp_exp = -24; /* subnormal spacing */
    double scaled = ldexp(a, -ulp_exp);          /* exact: power-of-two scaling */
    double fl = floor(scaled), rem = scaled - fl;
    if (rem > 0.5 || (rem == 0.5 && fmod(fl, 2.0) == 1.0)) fl += 1.0;
    double r = ldexp(fl, ulp_exp);               /* the rounded magnitude, exact */
    if (r >= 65520.0 || isinf(a)) return (uint16_t)(sign | 0x7C00);
    if (r < ldexp(1.0, -14)) return (uint16_t)(sign | (uint16_t)ldexp(r, 24));   /* subnormal */
    int re;
    double rm = frexp(r, &re);                   /* r = rm * 2^re */
    int biased = re - 1 + 15;
    int frac = (int)ldexp(rm, 11) - 1024;
    return (uint16_t)(sign | (biased << 10) | frac);
}

/* w[n,k] = fp16(s[n, k/G]) * q[n,k];  group == 0 means one scale per row (G = K). */
void oracle_dequantize(const int8_t* q, const uint16_t* s, int32_t N, int32_t K, int32_t group, double* w)
{
    int32_t G = group == 0 ? K : group;
    int32_t n_groups = K / G;
    for (int32_t n = 0; n < N; ++n)
        for (int32_t k = 0; k < K; ++k)
            w[(int64_t)n * K + k] = oracle_fp16_to_double(s[(int64_t)n * n_groups + k / G]) * (double)q[(int64_t)n * K + k];
}

/* y = x . w^T with x fp16 [M,K] row-major, w fp64 [N,K] row-major.
 * y64, A: [M,N] fp64; y16: [M,N] fp16 bit patterns.  Any output pointer may be NULL. */
void oracle_linear(const uint16_t* x, const double* w, int32_t M, int32_t N, int32_t K,
                   double* y64, double* A, uint16_t* y16)
{
    double* xd = (double*)malloc(sizeof(double) * (size_t)M * (size_t)K);   /* fp16 -> fp64, exact */
    if (!xd) return;
    for (int64_t i = 0; i < (int64_t)M * K; ++i) xd[i] = oracle_fp16_to_double(x[i]);
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
    for (int32_t n = 0; n < N; ++n) {
        for (int32_t m = 0; m < M; ++m) {
            double acc = 0.0, abs_acc = 0.0;
            for (int32_t k = 0; k < K; ++k) {
                double p = xd[(int64_t)m * K + k] * w[(int64_t)n * K + k];
                acc += p;
                abs_acc += fabs(p);
            }
            int64_t o = (int64_t)m * N + n;
            if (y64) y64[o] = acc;
            if (A)   A[o] = abs_acc;
            if (y16) y16[o] = oracle_double_to_fp16(acc);
        }
    }
    free(xd);
}

/* Threads oracle_linear uses (1 when built without OpenMP). */
int32_t oracle_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int32_t t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}
