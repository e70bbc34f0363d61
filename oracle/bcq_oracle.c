/*
 * bcq_oracle.c -- plain CPU oracle for the GPTQT inference path (arxiv 2407.02891).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the binary-coding-quantized (BCQ) linear layer computes.  It is called by the
 * tests, by the smoke check and by the benchmark's CPU-baseline leg, never by the
 * product path.  It shares no source, header, table or helper with the CUDA library.
 *
 * Everything floating point is evaluated in fp64 from the fp16 interface arrays
 * (fp16 -> fp64 is exact).  No blocking, no fusion, no reordering beyond the loops
 * the definitions state.  OpenMP only spreads independent output rows over cores.
 *
 * Passages followed (section "Intermediate Steps Can be Fused in Inference" unless
 * stated otherwise):
 *   Eq. fuse_step1  an n-bit integer is  sum_{i=1..n} 2^(i-2) b_i + (2^n - 1)/2,  b_i = +-1
 *   Eq. fuse_step2  bits that share a plane merge:  m_j = sum_{i in P_j} 2^(i-2)
 *   Eq. round       every W_int is replaced by the nearest value the merged code reaches
 *                   (section "Quantize Weight Twice")
 *   Eq. fuse_step3  S and qbias fold in:  alpha_j = S m_j,  z = S (2^n - 1)/2 + qbias
 *   Eq. gptqt step 1 (section "Quantize Weight Twice") with the scale of section
 *                   "Re-explore Scaling Factor":  S = (Wmax - Wmin)/(2^n - 1), qbias = Wmin,
 *                   W_int = round-to-nearest of the weight on that grid (orc_quantize_rtn)
 *   Eq. bcw         dequantised weight  w = sum_j alpha_j b_j  (+ z after the fusion)
 *
 * Readings taken where the paper is silent:
 *   - W_int is unsigned, 0 .. 2^n - 1 (Eq. fuse_step1 lists 0..7 for n = 3).
 *   - Dequantisation direction is  S * W_int + qbias  with qbias in weight units.
 *   - "Nearest" ties go to the SMALLER reachable value.  The paper fixes no tie rule:
 *     parity unpinned for the tie rule alone (tests assert minimal distance and
 *     determinism, not which of two equidistant values is taken).
 *   - A plane set P is a partition of the n step-1 bits into q non-empty sets.
 *   - Step 1 as printed, round(W/S - qbias), contradicts the dequantisation S W_int + qbias;
 *     the quantiser is the inverse of the dequantisation:  W_int = round((W - qbias)/S),
 *     clamped to 0 .. 2^n - 1, round = nearest, ties to even.  S is the fp16 value that
 *     is stored (the range formula evaluated in fp64, rounded once), so that quantiser and
 *     dequantiser use the same number.  A group whose weights are all equal gets S = 0,
 *     W_int = 0.
 *   - Batch: every column of x is an independent matrix-vector product.
 *
 * Layouts (all row-major, the last index fastest):
 *   w_int, codes  uint8  [N][K]      codes < 2^q, bit j of a code set <=> b_j = +1
 *   S, qbias, z   fp16   [N][G]      G = K / group, or 1 when group == 0 (per row)
 *   alpha         fp16   [q][N][G]
 *   planes        uint8  [q][N][K/8] bit (k mod 8) of byte (k div 8), LSB = lowest k
 *   x             fp16   [B][K]
 *   y             fp64   [B][N]
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_BAD (-1)

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- IEEE binary16 <-> binary64 ------------------------------------------------ */

double orc_half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int frac = h & 0x3ff;
    double v;
    if (expo == 0)
        v = ldexp((double)frac, -24);            /* zero and subnormals */
    else if (expo == 31)
        v = frac ? NAN : INFINITY;
    else
        v = ldexp((double)(frac + 1024), expo - 25);
    return sign ? -v : v;
}

/* round to nearest, ties to even */
uint16_t orc_double_to_half(double v)
{
    uint16_t sign = signbit(v) ? 0x8000u : 0;
    double a = fabs(v);
    if (isnan(v)) return (uint16_t)(sign | 0x7e00u);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u);      /* rounds to infinity */
    if (a < ldexp(1.0, -14)) {
        /* subnormal range: spacing 2^-24; rint() is ties-to-even in the default mode */
        double r = rint(ldexp(a, 24));
        return (uint16_t)(sign | (uint16_t)r);                /* r == 1024 is the least normal */
    }
    int e;
    double f = frexp(a, &e);                                   /* a = f 2^e, f in [0.5,1) */
    double r = rint(ldexp(f, 11));                             /* 11 significant bits */
    if (r == 2048.0) { r = 1024.0; e += 1; }
    int biased = e - 1 + 15;
    if (biased >= 31) return (uint16_t)(sign | 0x7c00u);
    return (uint16_t)(sign | (uint16_t)(biased << 10) | ((uint16_t)r - 1024));
}

/* ---- Eq. fuse_step1 / fuse_step2: what a merged q-plane code can reach --------- */

/*
 * bit_to_plane[i-1] = j says step-1 bit i (weight 2^(i-2), i = 1..n) belongs to plane j.
 * m[j]      <- sum of the weights of the bits in plane j
 * value[c]  <- the integer the sign pattern c reaches (bit j of c set <=> b_j = +1):
 *              (2^n - 1)/2 + sum_j (+-) m_j
 */
int orc_bcchoice(int n_bits, int q, const uint8_t *bit_to_plane, double *m, double *value)
{
    if (n_bits < 1 || n_bits > 8 || q < 1 || q > n_bits || !bit_to_plane) return ORC_BAD;
    for (int j = 0; j < q; ++j) m[j] = 0.0;
    for (int i = 1; i <= n_bits; ++i) {
        int j = bit_to_plane[i - 1];
        if (j >= q) return ORC_BAD;
        m[j] += ldexp(1.0, i - 2);
    }
    for (int j = 0; j < q; ++j)
        if (m[j] == 0.0) return ORC_BAD;          /* every plane needs at least one bit */
    double centre = (ldexp(1.0, n_bits) - 1.0) / 2.0;
    for (int c = 0; c < (1 << q); ++c) {
        double v = centre;
        for (int j = 0; j < q; ++j) v += ((c >> j) & 1) ? m[j] : -m[j];
        value[c] = v;
    }
    return ORC_OK;
}

/* ---- Eq. round: nearest reachable value ---------------------------------------- */

int orc_round_to_bcchoice(const uint8_t *w_int, size_t count, int n_bits, int q,
                          const uint8_t *bit_to_plane, uint8_t *w_q, uint8_t *codes)
{
    double m[8], value[256];
    if (orc_bcchoice(n_bits, q, bit_to_plane, m, value) != ORC_OK) return ORC_BAD;
    for (size_t t = 0; t < count; ++t) {
        if (w_int[t] >= (1u << n_bits)) return ORC_BAD;
        double w = (double)w_int[t];
        int best = 0;
        for (int c = 1; c < (1 << q); ++c) {
            double d = fabs(w - value[c]), db = fabs(w - value[best]);
            if (d < db || (d == db && value[c] < value[best])) best = c;
        }
        if (w_q) w_q[t] = (uint8_t)value[best];
        if (codes) codes[t] = (uint8_t)best;
    }
    return ORC_OK;
}

static int n_groups(int K, int group) { return group == 0 ? 1 : K / group; }
static int group_len(int K, int group) { return group == 0 ? K : group; }

/* ---- Eq. gptqt, step 1: linear quantisation of fp16 weights to n bits ---------- */

/* W fp16 [N][K].  Per (row, group): qbias = Wmin, S = fp16(s_factor (Wmax - Wmin)/(2^n - 1));
 * s_factor = 1 is the step-1 scale, other values are the re-explored scales of Eq. reexplore.
 * w_int = clamp(round((W - qbias)/S), 0, 2^n - 1). */
int orc_quantize_rtn(const uint16_t *W, int N, int K, int group, int n_bits, double s_factor,
                     uint8_t *w_int, uint16_t *S, uint16_t *qbias)
{
    if (N < 1 || K < 1 || group < 0 || (group && K % group) || n_bits < 1 || n_bits > 8) return ORC_BAD;
    if (!(s_factor > 0.0) || !isfinite(s_factor)) return ORC_BAD;
    int G = n_groups(K, group), L = group_len(K, group);
    double top = ldexp(1.0, n_bits) - 1.0;
    for (int n = 0; n < N; ++n)
        for (int g = 0; g < G; ++g) {
            const uint16_t *w = W + (size_t)n * K + (size_t)g * L;
            double lo = orc_half_to_double(w[0]), hi = lo;
            for (int k = 0; k < L; ++k) {
                double v = orc_half_to_double(w[k]);
                if (!isfinite(v)) return ORC_BAD;
                if (v < lo) lo = v;
                if (v > hi) hi = v;
            }
            if (lo == 0.0) lo = 0.0;   /* a zero minimum is stored as +0 whichever zero was met first */
            uint16_t s_h = orc_double_to_half((s_factor * (hi - lo)) / top);
            uint16_t b_h = orc_double_to_half(lo);   /* exact: lo is an fp16 value */
            double s = orc_half_to_double(s_h);
            if (!isfinite(s)) return ORC_BAD;
            S[(size_t)n * G + g] = s_h;
            qbias[(size_t)n * G + g] = b_h;
            for (int k = 0; k < L; ++k) {
                double r = 0.0;
                if (s > 0.0) {
                    r = rint((orc_half_to_double(w[k]) - lo) / s);   /* default rounding mode: ties to even */
                    if (r > top) r = top;
                    if (r < 0.0) r = 0.0;
                }
                w_int[(size_t)n * K + (size_t)g * L + k] = (uint8_t)r;
            }
        }
    return ORC_OK;
}

/* ---- Eq. fuse_step3: fold S and qbias into the code ---------------------------- */

int orc_merge_linear(const uint8_t *w_int, const uint16_t *S, const uint16_t *qbias,
                     int N, int K, int group, int n_bits, int q, const uint8_t *bit_to_plane,
                     uint8_t *codes, uint16_t *alpha, uint16_t *z)
{
    double m[8], value[256];
    if (N < 1 || K < 1 || group < 0 || (group && K % group)) return ORC_BAD;
    if (orc_bcchoice(n_bits, q, bit_to_plane, m, value) != ORC_OK) return ORC_BAD;
    int G = n_groups(K, group);
    if (orc_round_to_bcchoice(w_int, (size_t)N * K, n_bits, q, bit_to_plane, NULL, codes) != ORC_OK)
        return ORC_BAD;
    double centre = (ldexp(1.0, n_bits) - 1.0) / 2.0;
    for (int n = 0; n < N; ++n)
        for (int g = 0; g < G; ++g) {
            double s = orc_half_to_double(S[(size_t)n * G + g]);
            double b = orc_half_to_double(qbias[(size_t)n * G + g]);
            for (int j = 0; j < q; ++j)
                alpha[((size_t)j * N + n) * G + g] = orc_double_to_half(s * m[j]);
            z[(size_t)n * G + g] = orc_double_to_half(s * centre + b);
        }
    return ORC_OK;
}

/* ---- canonical bit-plane packing ----------------------------------------------- */

int orc_pack_canonical(const uint8_t *codes, int N, int K, int q, uint8_t *planes)
{
    if (N < 1 || K < 1 || K % 8 || q < 1 || q > 8) return ORC_BAD;
    size_t row_bytes = (size_t)K / 8;
    memset(planes, 0, (size_t)q * N * row_bytes);
    for (int i = 0; i < q; ++i)
        for (int n = 0; n < N; ++n)
            for (int k = 0; k < K; ++k)
                if ((codes[(size_t)n * K + k] >> i) & 1)
                    planes[((size_t)i * N + n) * row_bytes + k / 8] |= (uint8_t)(1u << (k % 8));
    return ORC_OK;
}

int orc_unpack_canonical(const uint8_t *planes, int N, int K, int q, uint8_t *codes)
{
    if (N < 1 || K < 1 || K % 8 || q < 1 || q > 8) return ORC_BAD;
    size_t row_bytes = (size_t)K / 8;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            unsigned c = 0;
            for (int i = 0; i < q; ++i)
                c |= (unsigned)((planes[((size_t)i * N + n) * row_bytes + k / 8] >> (k % 8)) & 1) << i;
            codes[(size_t)n * K + k] = (uint8_t)c;
        }
    return ORC_OK;
}

/* ---- Eq. bcw (dequant) + fused offset: the matrix the layer multiplies by ------ */

int orc_dequant(const uint8_t *codes, const uint16_t *alpha, const uint16_t *z,
                int N, int K, int q, int group, double *W)
{
    if (N < 1 || K < 1 || group < 0 || (group && K % group)) return ORC_BAD;
    int G = n_groups(K, group), L = group_len(K, group);
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            int g = k / L;
            double w = orc_half_to_double(z[(size_t)n * G + g]);
            for (int i = 0; i < q; ++i) {
                double a = orc_half_to_double(alpha[((size_t)i * N + n) * G + g]);
                w += ((codes[(size_t)n * K + k] >> i) & 1) ? a : -a;
            }
            W[(size_t)n * K + k] = w;
        }
    return ORC_OK;
}

/* ---- forward, form 1: y = W x with W dequantised element by element ------------ */

int orc_forward_dequant(const uint8_t *codes, const uint16_t *alpha, const uint16_t *z,
                        const uint16_t *x, int N, int K, int q, int group, int B, double *y)
{
    if (N < 1 || K < 1 || B < 1 || group < 0 || (group && K % group)) return ORC_BAD;
    int G = n_groups(K, group), L = group_len(K, group);
    double *xd = (double *)malloc(sizeof(double) * (size_t)B * K);
    if (!xd) return ORC_BAD;
    for (size_t t = 0; t < (size_t)B * K; ++t) xd[t] = orc_half_to_double(x[t]);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int b = 0; b < B; ++b) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                int g = k / L;
                double w = orc_half_to_double(z[(size_t)n * G + g]);
                for (int i = 0; i < q; ++i) {
                    double a = orc_half_to_double(alpha[((size_t)i * N + n) * G + g]);
                    w += ((codes[(size_t)n * K + k] >> i) & 1) ? a : -a;
                }
                acc += w * xd[(size_t)b * K + k];
            }
            y[(size_t)b * N + n] = acc;
        }
    free(xd);
    return ORC_OK;
}

/* ---- forward, form 2: y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g ) ------- */

int orc_forward_planes(const uint8_t *planes, const uint16_t *alpha, const uint16_t *z,
                       const uint16_t *x, int N, int K, int q, int group, int B, double *y)
{
    if (N < 1 || K < 1 || K % 8 || B < 1 || group < 0 || (group && K % group)) return ORC_BAD;
    int G = n_groups(K, group), L = group_len(K, group);
    size_t row_bytes = (size_t)K / 8;
    double *xd = (double *)malloc(sizeof(double) * (size_t)B * K);
    if (!xd) return ORC_BAD;
    for (size_t t = 0; t < (size_t)B * K; ++t) xd[t] = orc_half_to_double(x[t]);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int b = 0; b < B; ++b) {
            const double *xb = xd + (size_t)b * K;
            double acc = 0.0;
            for (int g = 0; g < G; ++g) {
                double sum_x = 0.0;
                for (int k = g * L; k < (g + 1) * L; ++k) sum_x += xb[k];
                double part = orc_half_to_double(z[(size_t)n * G + g]) * sum_x;
                for (int i = 0; i < q; ++i) {
                    const uint8_t *row = planes + ((size_t)i * N + n) * row_bytes;
                    double bx = 0.0;
                    for (int k = g * L; k < (g + 1) * L; ++k)
                        bx += ((row[k / 8] >> (k % 8)) & 1) ? xb[k] : -xb[k];
                    part += orc_half_to_double(alpha[((size_t)i * N + n) * G + g]) * bx;
                }
                acc += part;
            }
            y[(size_t)b * N + n] = acc;
        }
    free(xd);
    return ORC_OK;
}
