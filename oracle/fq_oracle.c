/*
 * CPU oracle for the elastic dequantize-and-matmul path (FlexQuant, arXiv 2501.07139).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  Nothing in the product may call it: only the
 * tests, the smoke check and the "CPU baseline" leg of the benchmark do.  It
 * shares no code, header, table or constant with the CUDA sources.
 *
 * What the paper fixes and what it leaves open
 * --------------------------------------------
 * The paper states only that (a) whatever the stored weight precision, the
 * arithmetic runs in a standard format such as FP16 (Sec. II-A), (b) an elastic
 * model picks, per module, one of a few stored quantised variants (Sec. III-A),
 * and (c) in the AnyPrecision variant lower precisions are obtained by truncating
 * bits of one stored parent, so storage is set by the largest precision
 * (Sec. II-B).  The concrete formats below (uniform asymmetric group
 * quantisation with group size 128, fp16 scale and zero point, the little-endian
 * bitstream, the bit-plane order, the mid-point fill of truncated codes) are
 * this project's reading of that statement; each reading is listed in the
 * design notes of the repository.
 *
 * Every function is a direct transcription of its definition: one loop nest,
 * no blocking, no vectorisation, no threads; sums run in index order in double
 * precision.
 *
 * Pins: every function here is pinned by tests that do not go through this
 * file (numpy's float16 / packbits / matmul, closed forms, hand-worked groups,
 * exhaustive enumeration) -- none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#include <stddef.h>
#include <stdlib.h>

#define FQO_GROUP 128

/* ------------------------------------------------------------------------- */
/* IEEE binary16 / bfloat16 <-> binary64, written out from the format.        */
/* ------------------------------------------------------------------------- */

/* binary16 -> double (exact). */
double fqo_f16_to_f64(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int m = h & 0x3ff;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24);                 /* zero and subnormals: m * 2^-24 */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp((double)(m + 1024), e - 25);     /* (1 + m/1024) * 2^(e-15)        */
    return sign ? -v : v;
}

/* double -> binary16, one rounding, round-to-nearest ties-to-even. */
uint16_t fqo_f64_to_f16(double d)
{
    uint64_t u;
    memcpy(&u, &d, sizeof u);
    uint16_t sign = (uint16_t)((u >> 48) & 0x8000u);
    int e = (int)((u >> 52) & 0x7ff);
    uint64_t m = u & 0xFFFFFFFFFFFFFull;
    if (e == 0x7ff)
        return (uint16_t)(sign | 0x7c00u | (m ? 0x200u : 0u));
    if (e == 0)
        return sign;                               /* below 2^-1022: rounds to zero  */
    int E = e - 1023;
    m |= 1ull << 52;                               /* value = m * 2^(E-52)           */
    int shift = (E >= -14) ? 42 : 42 + (-14 - E);  /* keep 11 bits, fewer if subnormal */
    if (shift > 63)
        return sign;
    uint64_t q = m >> shift;
    uint64_t rem = m & ((1ull << shift) - 1);
    uint64_t half = 1ull << (shift - 1);
    if (rem > half || (rem == half && (q & 1)))
        q++;
    if (E >= -14) {
        uint64_t r = ((uint64_t)(E + 15) << 10) + (q - 1024);  /* a carry bumps the exponent */
        if (r >= 0x7c00u)
            return (uint16_t)(sign | 0x7c00u);
        return (uint16_t)(sign | r);
    }
    return (uint16_t)(sign | q);                   /* subnormal (q == 1024 is the least normal) */
}

/* bfloat16 -> double (exact): bfloat16 is the top half of a binary32. */
double fqo_bf16_to_f64(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------- */
/* Quantiser: min-max asymmetric, b bits, per group of 128 columns.           */
/* Reading: scale is rounded to fp16 first, codes are then computed against   */
/* the rounded scale in double; rint() is round-half-to-even.                 */
/* ------------------------------------------------------------------------- */
void fqo_quantize(const float *w, int64_t n_out, int64_t k_in, int bits,
                  uint8_t *codes, uint16_t *scales, uint16_t *zeros)
{
    const double qmax = (double)((1 << bits) - 1);
    const int64_t groups = k_in / FQO_GROUP;
    for (int64_t n = 0; n < n_out; n++) {
        for (int64_t g = 0; g < groups; g++) {
            const float *wg = w + n * k_in + g * FQO_GROUP;
            double mn = wg[0], mx = wg[0];
            for (int k = 1; k < FQO_GROUP; k++) {
                if (wg[k] < mn) mn = wg[k];
                if (wg[k] > mx) mx = wg[k];
            }
            uint16_t sb = fqo_f64_to_f16((mx - mn) / qmax);
            if ((sb & 0x7fff) == 0)
                sb = 0x0400;                       /* degenerate group: 2^-14 */
            if ((sb & 0x7fff) >= 0x7c00)
                sb = 0x7bff;                       /* largest finite fp16     */
            const double S = fqo_f16_to_f64(sb);
            double z = rint(-mn / S);
            if (!(z > 0)) z = 0.0;                 /* also turns -0 into +0 */
            if (z > qmax) z = qmax;
            for (int k = 0; k < FQO_GROUP; k++) {
                double q = rint((double)wg[k] / S) + z;
                if (q < 0) q = 0;
                if (q > qmax) q = qmax;
                codes[n * k_in + g * FQO_GROUP + k] = (uint8_t)q;
            }
            scales[n * groups + g] = sb;
            zeros[n * groups + g] = fqo_f64_to_f16(z);   /* an integer <= 255: exact */
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Canonical packed format: per row a little-endian bitstream, code k in bits */
/* [k*b, (k+1)*b); stored as little-endian 32-bit words (K*b/32 per row).     */
/* ------------------------------------------------------------------------- */
void fqo_pack_bitstream(const uint8_t *codes, int64_t n_out, int64_t k_in, int bits, uint32_t *out)
{
    const int64_t words = k_in * bits / 32;
    memset(out, 0, (size_t)(n_out * words) * sizeof(uint32_t));
    for (int64_t n = 0; n < n_out; n++)
        for (int64_t k = 0; k < k_in; k++)
            for (int j = 0; j < bits; j++) {
                int64_t pos = k * bits + j;
                uint32_t bit = (codes[n * k_in + k] >> j) & 1u;
                out[n * words + pos / 32] |= bit << (pos % 32);
            }
}

void fqo_unpack_bitstream(const uint32_t *packed, int64_t n_out, int64_t k_in, int bits, uint8_t *codes)
{
    const int64_t words = k_in * bits / 32;
    for (int64_t n = 0; n < n_out; n++)
        for (int64_t k = 0; k < k_in; k++) {
            unsigned q = 0;
            for (int j = 0; j < bits; j++) {
                int64_t pos = k * bits + j;
                q |= ((packed[n * words + pos / 32] >> (pos % 32)) & 1u) << j;
            }
            codes[n * k_in + k] = (uint8_t)q;
        }
}

/* ------------------------------------------------------------------------- */
/* Canonical nested format: the 8-bit parent code as 8 bit-planes, most       */
/* significant plane first.  planes[(7-p)][n][k/32], bit (k%32) = bit p of q8. */
/* A b-bit child is the first b planes (Sec. II-B: truncate / re-append bits). */
/* ------------------------------------------------------------------------- */
void fqo_pack_planes(const uint8_t *q8, int64_t n_out, int64_t k_in, uint32_t *planes)
{
    const int64_t words = k_in / 32;
    memset(planes, 0, (size_t)(8 * n_out * words) * sizeof(uint32_t));
    for (int p = 0; p < 8; p++)
        for (int64_t n = 0; n < n_out; n++)
            for (int64_t k = 0; k < k_in; k++) {
                uint32_t bit = (q8[n * k_in + k] >> p) & 1u;
                planes[((int64_t)(7 - p) * n_out + n) * words + k / 32] |= bit << (k % 32);
            }
}

/* Child codes read from the first `bits` planes only: q_b = q8 >> (8 - b). */
void fqo_child_codes(const uint32_t *planes, int64_t n_out, int64_t k_in, int bits, uint8_t *codes)
{
    const int64_t words = k_in / 32;
    for (int64_t n = 0; n < n_out; n++)
        for (int64_t k = 0; k < k_in; k++) {
            unsigned q = 0;
            for (int t = 0; t < bits; t++) {       /* t-th stored plane holds parent bit 7-t */
                uint32_t bit = (planes[((int64_t)t * n_out + n) * words + k / 32] >> (k % 32)) & 1u;
                q |= bit << (bits - 1 - t);
            }
            codes[n * k_in + k] = (uint8_t)q;
        }
}

/* ------------------------------------------------------------------------- */
/* Dequantisation: w^ = fp16_rne((q - z) * s), one rounding of the exact      */
/* product (Sec. II-A: computation in FP16).                                  */
/* parent_bits == bits : a stored b-bit variant, d = q - z.                   */
/* parent_bits == 8 > bits : a nested child in the parent's code units,       */
/*     d = (q << (8-b)) + 2^(7-b) - z8   (mid-point fill of the dropped bits). */
/* ------------------------------------------------------------------------- */
double fqo_dequant_one(unsigned q, int bits, int parent_bits, uint16_t scale, uint16_t zero)
{
    double d;
    if (parent_bits == bits)
        d = (double)q - fqo_f16_to_f64(zero);
    else
        d = (double)(q << (parent_bits - bits)) + (double)(1 << (parent_bits - bits - 1))
            - fqo_f16_to_f64(zero);
    return fqo_f16_to_f64(fqo_f64_to_f16(d * fqo_f16_to_f64(scale)));
}

/* Dequantised matrix (as doubles holding fp16 values), codes one per byte. */
void fqo_dequant(const uint8_t *codes, const uint16_t *scales, const uint16_t *zeros,
                 int64_t n_out, int64_t k_in, int bits, int parent_bits, double *w_hat)
{
    const int64_t groups = k_in / FQO_GROUP;
    for (int64_t n = 0; n < n_out; n++)
        for (int64_t k = 0; k < k_in; k++) {
            int64_t g = n * groups + k / FQO_GROUP;
            w_hat[n * k_in + k] = fqo_dequant_one(codes[n * k_in + k], bits, parent_bits,
                                                  scales[g], zeros[g]);
        }
}

/* ------------------------------------------------------------------------- */
/* GEMV / GEMM:  Y[m][n] = sum_k X[m][k] * w^[n][k], fp64, k ascending.       */
/* x_is_bf16 == 0: X holds fp16 bit patterns (decode); 1: bf16 (prefill).      */
/* ------------------------------------------------------------------------- */
void fqo_matmul(const uint8_t *codes, const uint16_t *scales, const uint16_t *zeros,
                int64_t n_out, int64_t k_in, int bits, int parent_bits,
                const uint16_t *x, int64_t m_rows, int64_t ldx, int x_is_bf16, double *y)
{
    const int64_t groups = k_in / FQO_GROUP;
    double *w_row = (double *)malloc((size_t)k_in * sizeof(double));   /* w^[n][:] */
    for (int64_t n = 0; n < n_out; n++) {
        for (int64_t k = 0; k < k_in; k++) {
            int64_t g = n * groups + k / FQO_GROUP;
            w_row[k] = fqo_dequant_one(codes[n * k_in + k], bits, parent_bits, scales[g], zeros[g]);
        }
        for (int64_t m = 0; m < m_rows; m++) {
            double acc = 0.0;
            for (int64_t k = 0; k < k_in; k++) {
                double xv = x_is_bf16 ? fqo_bf16_to_f64(x[m * ldx + k]) : fqo_f16_to_f64(x[m * ldx + k]);
                acc += xv * w_row[k];
            }
            y[m * n_out + n] = acc;
        }
    }
    free(w_row);
}

/* ------------------------------------------------------------------------- */
/* Footprint of one configuration: selected code bytes + fp16 scale and zero. */
/* ------------------------------------------------------------------------- */
uint64_t fqo_footprint(const int64_t *n_out, const int64_t *k_in, const uint8_t *bits, int64_t n_layers)
{
    uint64_t total = 0;
    for (int64_t l = 0; l < n_layers; l++) {
        total += (uint64_t)n_out[l] * (uint64_t)k_in[l] * bits[l] / 8;
        total += (uint64_t)n_out[l] * (uint64_t)(k_in[l] / FQO_GROUP) * 4;
    }
    return total;
}
