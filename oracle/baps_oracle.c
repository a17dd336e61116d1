/*
 * BAPS oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision CPU statement of what the BAPS hot path computes
 * (block-aware precision rescaling for softmax in attention).  It exists so that the CUDA
 * library can be checked against something written directly from the paper.  Only the test
 * suite, the smoke check and the CPU-baseline leg of the benchmark may call it; the product
 * path never does, and this file shares no code, table or constant generator with the CUDA
 * sources.
 *
 * What follows the paper and where:
 *   - Eq. (1)            exact attention                       -> exact_attention_tile()
 *   - Eq. (2)            base-2 online softmax iteration       -> the B0 branch below
 *   - Section 3.2        T = S - rowfill(m~), sent in 8 bits   -> step "T8" below
 *   - Section 3.3        integer (ceil) running max            -> ceil() in the max updates
 *   - Algorithm 1        the whole per-query-tile workflow     -> baps_oracle_attention()
 *   - Algorithm 2        2^x with 8-bit input and output       -> baps_oracle_exp2_code()
 *   - Section 4.1        "Exp2 HiF8" setup (Eq. (2), real-valued max, every power of two
 *                        through Algorithm 2)                  -> the exp2_only branch below
 *   - Section 4.2        comparison setups: Exp2 with E4M3 / E5M2 / E4M3 in, E5M2 out as the
 *                        formats of the exponentiation, and "Naive E2E" (scores cast to HiF8
 *                        before the max is subtracted)        -> fmt_in / fmt_out / naive below
 *   - HiF8               the 8-bit format the paper adopts from its reference on the Ascend
 *                        HiFloat8 format (sign, prefix-coded "dot" field, sign-magnitude
 *                        exponent with a hidden leading one, tapered mantissa)
 *
 * Readings of points the paper leaves open (all listed again in the design notes):
 *   R1  conversion to HiF8 rounds to the nearest representable value, ties to the larger
 *       magnitude; values at or beyond the midpoint between the largest finite value and
 *       the next would-be value become infinity; magnitudes below half the smallest
 *       denormal become +0 (the format has no negative zero; code 0x80 is NaN).
 *   R2  the brackets around rowmax in Algorithm 1 are a ceiling.
 *   R3  in the no-restart branch the running max grows by delta = max(0, ceil(rowmax T)),
 *       while P = 2^T is still relative to the previous max; the tile's weights are
 *       therefore multiplied by the exact power of two 2^(-delta) before they enter d and
 *       O~ (this is the only reading under which removing the roundings gives Eq. (1)).
 *   R4  the restart test is taken once per (query tile, key tile): the largest entry of the
 *       8-bit T over the whole tile is compared with lambda.
 *   R5  B0 is the first key tile (Section 4.1), or -- option b0_last, after Section 3.2's remark that
 *       in causal language models the first and the last tile usually hold the large scores --
 *       the first and the last visible key tile (the diagonal tile when causal): the tiles are
 *       then visited in the order 0, last, 1, 2, ..., last - 1, the first two in high precision.
 *       Initial state m = -inf, d = 0, O~ = 0.
 *   R6  a causally masked score is -inf; its 8-bit code is -Inf and its weight 0.
 *   R7  E4M3 / E5M2 (comparison setups only) are the OCP 8-bit formats: E4M3 with bias 7, no
 *       infinity, largest finite 448, subnormals down to 2^-9; E5M2 with bias 15, largest finite
 *       57344, subnormals down to 2^-16.  Conversion rounds to nearest, ties to even, and
 *       saturates at the largest finite value (no NaN or infinity is produced from finite input).
 *   R8  "Naive E2E": the scores are converted to HiF8 as they are, before any maximum is
 *       subtracted, and then go through the Exp2 HiF8 workflow (Eq. (2), real-valued max, 8-bit
 *       exponentials); no integer max, no restart.
 *
 * parity unpinned: (a) agreement of this file's HiF8 code table with the hardware format of
 * the cited HiFloat8 paper cannot be checked here (that paper is not available); the table is
 * pinned to the value set and bit layout recorded in tests/golden/.  (b) the restart rates the
 * paper reports need its models' activations and are not reproduced.
 *
 * Build:  gcc -O2 -fopenmp -shared -fPIC -o libbaps_oracle.so baps_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------------------ */
/* HiF8: value of a code, written out from the field layout.                              */
/* ------------------------------------------------------------------------------------ */

/* Value of code c.  Layout of the low 7 bits b (sign bit s = c >> 7):
 *   11 eeee m   exponent field 4 bits: first bit = exponent sign, rest a -> |E| = 8 + a
 *   10 eee mm   exponent field 3 bits                                    -> |E| = 4 + a
 *   01 ee mmm   exponent field 2 bits                                    -> |E| = 2 + a
 *   001 e mmm   exponent field 1 bit (sign only)                         -> |E| = 1
 *   0001 mmm    no exponent field                                        ->  E  = 0
 *   0000 mmm    denormal: 2^(m - 23), m = 1..7; m = 0: +0 (s = 0) or NaN (s = 1)
 * Normal values are (+/-) 2^E * (1 + m / 2^k), k = number of mantissa bits.  The largest
 * magnitude code (E = +15, m = 1) is infinity. */
double baps_oracle_hif8_value(uint8_t c)
{
    int s = c >> 7;
    int b = c & 0x7F;
    double mag;
    if (b == 0) return s ? NAN : 0.0;
    if ((b >> 5) == 3) {
        int ef = (b >> 1) & 0xF, m = b & 1;
        int E = 8 + (ef & 7);
        if (ef >> 3) E = -E;
        if (E == 15 && m == 1) mag = INFINITY;
        else mag = ldexp(1.0 + m / 2.0, E);
    } else if ((b >> 5) == 2) {
        int ef = (b >> 2) & 7, m = b & 3;
        int E = 4 + (ef & 3);
        if (ef >> 2) E = -E;
        mag = ldexp(1.0 + m / 4.0, E);
    } else if ((b >> 5) == 1) {
        int ef = (b >> 3) & 3, m = b & 7;
        int E = 2 + (ef & 1);
        if (ef >> 1) E = -E;
        mag = ldexp(1.0 + m / 8.0, E);
    } else if ((b >> 4) == 1) {
        int m = b & 7;
        int E = ((b >> 3) & 1) ? -1 : 1;
        mag = ldexp(1.0 + m / 8.0, E);
    } else if ((b >> 3) == 1) {
        mag = 1.0 + (b & 7) / 8.0;
    } else {
        mag = ldexp(1.0, (b & 7) - 23);
    }
    return s ? -mag : mag;
}

/* Ascending list of the non-negative magnitudes the format can hold (0, the denormals, the
 * normals), the code of each with sign bit clear, and one extra slot for the position where
 * infinity sits on the number line (1.5 * 2^15): rounding to it means overflow. */
#define HIF8_NMAG 128
static double g_mag[HIF8_NMAG];
static uint8_t g_mag_code[HIF8_NMAG];
static int g_nmag = 0;

static void hif8_init(void)
{
    if (g_nmag) return;
#pragma omp critical(baps_oracle_init)
    {
        if (!g_nmag) {
            int n = 0;
            for (int c = 0; c < 128; ++c) {
                double v = baps_oracle_hif8_value((uint8_t)c);
                if (isinf(v)) v = ldexp(1.5, 15);
                /* insertion into the ascending list */
                int p = n;
                while (p > 0 && g_mag[p - 1] > v) {
                    g_mag[p] = g_mag[p - 1];
                    g_mag_code[p] = g_mag_code[p - 1];
                    --p;
                }
                g_mag[p] = v;
                g_mag_code[p] = (uint8_t)c;
                ++n;
            }
            g_nmag = n;
        }
    }
}

/* Nearest representable value, ties to the larger magnitude (reading R1).
 * If margin is not NULL it receives the distance from |x| to the nearest rounding boundary
 * (midpoint between adjacent magnitudes) and alt receives the code that the value on the
 * other side of that boundary would get. */
static uint8_t hif8_encode_one(double x, double *margin, uint8_t *alt)
{
    hif8_init();
    if (margin) *margin = INFINITY;
    if (alt) *alt = 0x80;
    if (isnan(x)) return 0x80;
    int neg = signbit(x) ? 1 : 0;
    double a = fabs(x);
    /* largest index lo with g_mag[lo] <= a (g_mag[0] = 0 so lo >= 0) */
    int lo = 0, hi = g_nmag - 1;
    if (a >= g_mag[hi]) lo = hi;
    else {
        while (hi - lo > 1) {
            int mid = (lo + hi) / 2;
            if (g_mag[mid] <= a) lo = mid; else hi = mid;
        }
    }
    int pick = lo;
    if (lo + 1 < g_nmag) {
        double dlo = a - g_mag[lo], dhi = g_mag[lo + 1] - a;
        if (dhi <= dlo) pick = lo + 1;          /* tie -> larger magnitude */
    }
    if (margin) {
        /* boundaries around the picked value */
        double best = INFINITY; int other = pick;
        if (pick + 1 < g_nmag) {
            double mid = 0.5 * (g_mag[pick] + g_mag[pick + 1]);
            if (fabs(a - mid) < best) { best = fabs(a - mid); other = pick + 1; }
        }
        if (pick > 0) {
            double mid = 0.5 * (g_mag[pick] + g_mag[pick - 1]);
            if (fabs(a - mid) < best) { best = fabs(a - mid); other = pick - 1; }
        }
        *margin = best;
        if (alt) {
            uint8_t oc = g_mag_code[other];
            *alt = (other == 0) ? 0x00 : (uint8_t)(oc | (neg << 7));
        }
    }
    uint8_t code = g_mag_code[pick];
    if (pick == 0) return 0x00;                 /* no negative zero */
    return (uint8_t)(code | (neg << 7));
}

void baps_oracle_hif8_encode(const double *x, uint8_t *codes, int64_t n)
{
    hif8_init();
    for (int64_t i = 0; i < n; ++i) codes[i] = hif8_encode_one(x[i], NULL, NULL);
}

void baps_oracle_hif8_decode(const uint8_t *codes, double *x, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) x[i] = baps_oracle_hif8_value(codes[i]);
}

/* Algorithm 2 with the 16-bit detour left out: the real number 2^value(t), rounded once to
 * HiF8.  (For every code the 16-bit intermediate holds 2^value(t) to more bits than the
 * final rounding keeps, and the test suite checks that the detour changes no entry.) */
uint8_t baps_oracle_exp2_code(uint8_t t)
{
    double v = baps_oracle_hif8_value(t);
    if (isnan(v)) return 0x80;
    return hif8_encode_one(exp2(v), NULL, NULL);
}

/* Algorithm 2 taken literally, the 16-bit intermediate supplied by the caller: y16 is
 * fp16(2^value(t)) computed outside (numpy), this returns its HiF8 code. */
uint8_t baps_oracle_encode_scalar(double y)
{
    return hif8_encode_one(y, NULL, NULL);
}

/* ------------------------------------------------------------------------------------ */
/* OCP E4M3 / E5M2 (comparison setups of Section 4.2; reading R7).                         */
/* ------------------------------------------------------------------------------------ */

/* Value of a non-negative code (sign bit clear) of a format with ebits exponent bits, mbits
 * mantissa bits and the usual bias 2^(ebits-1) - 1. */
static double ocp_value(int code, int ebits, int mbits)
{
    int bias = (1 << (ebits - 1)) - 1;
    int e = code >> mbits, m = code & ((1 << mbits) - 1);
    if (e == 0) return ldexp((double)m, 1 - bias - mbits);            /* subnormal */
    return ldexp(1.0 + (double)m / (double)(1 << mbits), e - bias);
}

/* Round x to the format: nearest value, ties to the even code, saturating at the largest finite
 * code max_code (E4M3: 0x7E = 448; E5M2: 0x7B = 57344).  Returns the rounded value. */
static double ocp_round(double x, int ebits, int mbits, int max_code)
{
    if (isnan(x)) return x;
    double a = fabs(x), sgn = signbit(x) ? -1.0 : 1.0;
    if (a >= ocp_value(max_code, ebits, mbits)) return sgn * ocp_value(max_code, ebits, mbits);
    int lo = 0, hi = max_code;                    /* value(lo) <= a < value(hi) */
    while (hi - lo > 1) {
        int mid = (lo + hi) / 2;
        if (ocp_value(mid, ebits, mbits) <= a) lo = mid; else hi = mid;
    }
    double vlo = ocp_value(lo, ebits, mbits), vhi = ocp_value(hi, ebits, mbits);
    double dlo = a - vlo, dhi = vhi - a;
    int pick = (dlo < dhi) ? lo : (dhi < dlo) ? hi : ((lo & 1) ? hi : lo);
    return sgn * ocp_value(pick, ebits, mbits);
}

double baps_oracle_round_e4m3(double x) { return ocp_round(x, 4, 3, 0x7E); }
double baps_oracle_round_e5m2(double x) { return ocp_round(x, 5, 2, 0x7B); }

/* ------------------------------------------------------------------------------------ */
/* Rounding front-ends used by Algorithm 1.  fmt = 0: HiF8; fmt = 1: identity (no          */
/* rounding at all -- used only to check that the workflow then reduces to Eq. (1)).       */
/* ------------------------------------------------------------------------------------ */

static inline double round_T(double u, int fmt, double *margin, double *alt_val)
{
    if (fmt == 1) { if (margin) *margin = INFINITY; if (alt_val) *alt_val = u; return u; }
    if (fmt == 2 || fmt == 3) {                    /* E4M3 / E5M2: comparison setups, no margins */
        double r = (u == -INFINITY) ? u : (fmt == 2 ? baps_oracle_round_e4m3(u) : baps_oracle_round_e5m2(u));
        if (margin) *margin = INFINITY;
        if (alt_val) *alt_val = r;
        return r;
    }
    uint8_t alt;
    uint8_t c = hif8_encode_one(u, margin, &alt);
    if (alt_val) *alt_val = baps_oracle_hif8_value(alt);
    return baps_oracle_hif8_value(c);
}

static inline double exp2_8(double t8, int fmt)
{
    if (fmt == 1) return exp2(t8);
    if (fmt == 2) return baps_oracle_round_e4m3(exp2(t8));
    if (fmt == 3) return baps_oracle_round_e5m2(exp2(t8));
    /* t8 is a HiF8 value: 2^t8 rounded once to HiF8 (Algorithm 2) */
    return baps_oracle_hif8_value(hif8_encode_one(exp2(t8), NULL, NULL));
}

/* ------------------------------------------------------------------------------------ */
/* Algorithm 1 for one query tile.                                                         */
/* ------------------------------------------------------------------------------------ */

typedef struct {
    int S, D, causal, bq, bk, lambda, fmt;
    int exp2_only;     /* 1: "Exp2 HiF8" setup -- Eq. (2) with every 2^x done by Algorithm 2 */
    int b0_last;       /* 1: B0 = {first, last visible key tile}; 0: B0 = {first} */
    int fmt_out;       /* format of the results of 2^x in the Exp2 setup (fmt is the format of its arguments) */
    int naive;         /* 1: "Naive E2E" -- scores converted to HiF8 before the max is subtracted */
    double c;          /* log2(e) * scale */
    double eps_rel;    /* a decision closer than eps_rel * max(1, |s|) to its boundary is "near" */
} tile_cfg;

/* q: [S, D] of this (b, h); k, v: [S, D] of the kv head.  Rows i0 .. i0 + bq - 1.
 * out: [bq, D] (O = O~ / d, not rounded).  row_m, row_d: final max and denominator.
 * row_margin: smallest relative distance of any row-level decision to its boundary.
 * row_allow: bound on the change of any output element if the near-boundary element
 * roundings of this row had gone the other way.  Returns the number of restarted tiles. */
static int baps_tile(const tile_cfg *g, const float *q, const float *k, const float *v,
                     int i0, double *out, double *row_m, double *row_d,
                     double *row_margin, double *row_allow, int *n_tiles)
{
    const int bq = g->bq, bk = g->bk, D = g->D, S = g->S;
    double *Sc = (double *)malloc(sizeof(double) * bq * bk);    /* scores of the tile       */
    double *T8 = (double *)malloc(sizeof(double) * bq * bk);    /* rounded T                */
    double *W = (double *)malloc(sizeof(double) * bq * bk);     /* weights entering d, O~   */
    double *Walt = (double *)malloc(sizeof(double) * bq * bk);  /* |w_alt - w| if near      */
    double *m = (double *)malloc(sizeof(double) * bq);
    double *d = (double *)malloc(sizeof(double) * bq);
    double *O = (double *)calloc((size_t)bq * D, sizeof(double));
    double *marg = (double *)malloc(sizeof(double) * bq);
    double *lg = (double *)calloc((size_t)bq, sizeof(double));   /* log2 of the product of rescale factors */
    /* per element record for the allowance, kept for all tiles: (key index, |dw| / scale) */
    double *amb_dw = (double *)calloc((size_t)bq * S, sizeof(double));
    double *scale_at = (double *)malloc(sizeof(double) * bq * (S / bk)); /* m after tile j */
    int restarts = 0, tiles = 0;
    for (int r = 0; r < bq; ++r) { m[r] = -INFINITY; d[r] = 0.0; marg[r] = INFINITY; }

    int jmax = S / bk;
    if (g->causal) jmax = (i0 + bq - 1) / bk + 1;
    const int nb0 = (g->b0_last && jmax >= 2) ? 2 : 1;      /* number of high-precision tiles */
    for (int step = 0; step < jmax; ++step) {
        /* visiting order: 0, 1, 2, ... or, with b0_last, 0, last, 1, ..., last - 1 */
        const int j = !g->b0_last ? step : (step == 0 ? 0 : (step == 1 ? jmax - 1 : step - 1));
        const int c0 = j * bk;
        /* step 1: S = Q K^T * log2(e) / sqrt(d), masked entries -inf */
        for (int r = 0; r < bq; ++r)
            for (int cc = 0; cc < bk; ++cc) {
                const float *qr = q + (size_t)(i0 + r) * D;
                const float *kc = k + (size_t)(c0 + cc) * D;
                double acc = 0.0;
                for (int t = 0; t < D; ++t) acc += (double)qr[t] * (double)kc[t];
                double s = acc * g->c;
                if (g->causal && c0 + cc > i0 + r) s = -INFINITY;
                Sc[r * bk + cc] = s;
            }
        ++tiles;
        if (g->exp2_only) {
            /* "Exp2 HiF8" (Section 4.1): Eq. (2) as it stands -- real-valued running max -- but the
             * argument of every power of two is converted to HiF8 and the result again
             * (Algorithm 2): P = EXP2_8(HiF8(S - m)), rescale factor EXP2_8(HiF8(m_prev - m)). */
            if (g->naive)      /* reading R8: the scores themselves are sent in 8 bits */
                for (int e = 0; e < bq * bk; ++e)
                    if (Sc[e] != -INFINITY) Sc[e] = round_T(Sc[e], 0, NULL, NULL);
            const int simple = (g->fmt != 0 || g->fmt_out != g->fmt);   /* no margins for the comparison formats */
            for (int r = 0; r < bq; ++r) {
                double rm = -INFINITY;
                for (int cc = 0; cc < bk; ++cc) rm = fmax(rm, Sc[r * bk + cc]);
                double mnew = fmax(m[r], rm);
                double alpha = 0.0;
                if (m[r] != -INFINITY) {
                    double mg, altv;
                    double t8 = round_T(m[r] - mnew, g->fmt, &mg, &altv);
                    alpha = exp2_8(t8, g->fmt_out);
                    if (!simple && exp2_8(altv, 0) != alpha)
                        marg[r] = fmin(marg[r], mg / fmax(1.0, fabs(mnew)));
                }
                double sum = 0.0;
                for (int cc = 0; cc < bk; ++cc) {
                    double s = Sc[r * bk + cc];
                    double w = 0.0, dw = 0.0;
                    if (s != -INFINITY) {
                        double mg, altv;
                        double t8 = round_T(s - mnew, g->fmt, &mg, &altv);
                        w = exp2_8(t8, g->fmt_out);
                        if (!simple && mg < g->eps_rel * fmax(1.0, fabs(s)))
                            dw = fabs(exp2_8(altv, 0) - w);
                    }
                    W[r * bk + cc] = w; Walt[r * bk + cc] = dw;
                    sum += w;
                }
                d[r] = alpha * d[r] + sum;
                for (int t = 0; t < D; ++t) O[r * D + t] *= alpha;
                if (alpha > 0.0) lg[r] += log2(alpha);
                m[r] = mnew;
            }
        } else if (step < nb0) {
            /* B0 tile: Eq. (2) with an integer (ceil) max, everything in high precision */
            for (int r = 0; r < bq; ++r) {
                double rm = -INFINITY;
                for (int cc = 0; cc < bk; ++cc) rm = fmax(rm, Sc[r * bk + cc]);
                double cm = ceil(rm);
                if (isfinite(rm) && cm >= m[r]) {
                    double dist = fmin(cm - rm, rm - (cm - 1.0));
                    marg[r] = fmin(marg[r], dist / fmax(1.0, fabs(rm)));
                }
                double mnew = fmax(m[r], cm);
                double alpha = (m[r] == -INFINITY) ? 0.0 : exp2(m[r] - mnew);
                double sum = 0.0;
                for (int cc = 0; cc < bk; ++cc) {
                    double w = (mnew == -INFINITY) ? 0.0 : exp2(Sc[r * bk + cc] - mnew);
                    W[r * bk + cc] = w; Walt[r * bk + cc] = 0.0;
                    sum += w;
                }
                d[r] = alpha * d[r] + sum;
                for (int t = 0; t < D; ++t) O[r * D + t] *= alpha;
                m[r] = mnew;
            }
        } else {
            /* B1 tile.  m~ = previous max; T = S - m~ in 8 bits. */
            double tile_max = -INFINITY;
            for (int r = 0; r < bq; ++r)
                for (int cc = 0; cc < bk; ++cc) {
                    double s = Sc[r * bk + cc];
                    double t8 = (s == -INFINITY) ? -INFINITY : round_T(s - m[r], g->fmt, NULL, NULL);
                    T8[r * bk + cc] = t8;
                    tile_max = fmax(tile_max, t8);
                }
            int restart = tile_max > (double)g->lambda;
            /* How close was the (tile-wide) restart decision?  Per row: the unrounded row
             * maximum, its rounded value, the distance to the nearest rounding boundary and
             * the value on the other side.  A restart is undone only if every row above
             * lambda falls back; a non-restart is overturned if any row climbs above it.
             * Rows whose own maximum is positive are the ones a changed decision alters. */
            if (g->fmt == 0) {
                double lam = (double)g->lambda;
                double tile_margin = restart ? 0.0 : INFINITY;
                for (int r = 0; r < bq; ++r) {
                    double um = -INFINITY, sm = 0.0;
                    for (int cc = 0; cc < bk; ++cc) {
                        double s = Sc[r * bk + cc];
                        if (s != -INFINITY && s - m[r] > um) { um = s - m[r]; sm = s; }
                    }
                    if (um == -INFINITY) continue;
                    double mg, altv;
                    double t8 = round_T(um, 0, &mg, &altv);
                    double rel = mg / fmax(1.0, fabs(sm));
                    if (restart) {
                        if (t8 > lam) tile_margin = fmax(tile_margin, (altv > lam) ? INFINITY : rel);
                    } else {
                        if (altv > lam) tile_margin = fmin(tile_margin, rel);
                    }
                }
                for (int r = 0; r < bq; ++r) {
                    double um = -INFINITY;
                    for (int cc = 0; cc < bk; ++cc) {
                        double s = Sc[r * bk + cc];
                        if (s != -INFINITY && s - m[r] > um) um = s - m[r];
                    }
                    if (um > 0.0) marg[r] = fmin(marg[r], tile_margin);
                }
            }
            if (restart) {
                ++restarts;
                for (int r = 0; r < bq; ++r) {
                    double rm = -INFINITY;
                    for (int cc = 0; cc < bk; ++cc) rm = fmax(rm, Sc[r * bk + cc]);
                    double cm = ceil(rm);
                    if (isfinite(rm) && cm >= m[r]) {
                        double dist = fmin(cm - rm, rm - (cm - 1.0));
                        marg[r] = fmin(marg[r], dist / fmax(1.0, fabs(rm)));
                    }
                    double mnew = fmax(m[r], cm);
                    double alpha = exp2(m[r] - mnew);
                    double sum = 0.0;
                    for (int cc = 0; cc < bk; ++cc) {
                        double s = Sc[r * bk + cc];
                        double w = 0.0, dw = 0.0;
                        if (s != -INFINITY) {
                            double mg, altv;
                            double t8 = round_T(s - mnew, g->fmt, &mg, &altv);
                            w = exp2_8(t8, g->fmt);
                            if (mg < g->eps_rel * fmax(1.0, fabs(s)))
                                dw = fabs(exp2_8(altv, g->fmt) - w);
                        }
                        W[r * bk + cc] = w; Walt[r * bk + cc] = dw;
                        sum += w;
                    }
                    d[r] = alpha * d[r] + sum;
                    for (int t = 0; t < D; ++t) O[r * D + t] *= alpha;
                    m[r] = mnew;
                }
            } else {
                for (int r = 0; r < bq; ++r) {
                    double rm = -INFINITY;
                    for (int cc = 0; cc < bk; ++cc) rm = fmax(rm, T8[r * bk + cc]);
                    double delta = 0.0;
                    if (rm != -INFINITY) {
                        delta = fmax(0.0, ceil(rm));
                        /* delta changes when the rounded row max crosses 0 or an integer
                         * <= lambda: measure the unrounded distance to those crossings */
                        if (g->fmt == 0) {
                            double um = -INFINITY, sm = 0.0;
                            for (int cc = 0; cc < bk; ++cc) {
                                double s = Sc[r * bk + cc];
                                if (s != -INFINITY && s - m[r] > um) { um = s - m[r]; sm = s; }
                            }
                            double mg, altv;
                            double t8 = round_T(um, 0, &mg, &altv);
                            double dalt = fmax(0.0, ceil(altv));
                            if (dalt != fmax(0.0, ceil(t8)))
                                marg[r] = fmin(marg[r], mg / fmax(1.0, fabs(sm)));
                        }
                    }
                    double mnew = m[r] + delta;
                    double alpha = exp2(m[r] - mnew);       /* = 2^(-delta), exact */
                    double sum = 0.0;
                    for (int cc = 0; cc < bk; ++cc) {
                        double s = Sc[r * bk + cc];
                        double w = 0.0, dw = 0.0;
                        if (s != -INFINITY) {
                            /* reading R3: weights relative to the new max */
                            w = exp2_8(T8[r * bk + cc], g->fmt) * alpha;
                            if (g->fmt == 0) {
                                double mg, altv;
                                (void)round_T(s - m[r], 0, &mg, &altv);
                                if (mg < g->eps_rel * fmax(1.0, fabs(s)))
                                    dw = fabs(exp2_8(altv, 0) * alpha - w);
                            }
                        }
                        W[r * bk + cc] = w; Walt[r * bk + cc] = dw;
                        sum += w;
                    }
                    d[r] = alpha * d[r] + sum;
                    for (int t = 0; t < D; ++t) O[r * D + t] *= alpha;
                    m[r] = mnew;
                }
            }
        }
        /* O~ += W V_j ; remember the ambiguous weight changes at the current scale */
        for (int r = 0; r < bq; ++r) {
            for (int cc = 0; cc < bk; ++cc) {
                double w = W[r * bk + cc];
                if (w != 0.0) {
                    const float *vc = v + (size_t)(c0 + cc) * D;
                    for (int t = 0; t < D; ++t) O[r * D + t] += w * (double)vc[t];
                }
                amb_dw[(size_t)r * S + c0 + cc] = Walt[r * bk + cc];
            }
            /* what later rescales will multiply this tile's weights by is 2^(scale_at - final) */
            scale_at[r * (S / bk) + j] = g->exp2_only ? -lg[r] : m[r];
        }
    }
    /* normalisation O = diag(d)^-1 O~ */
    for (int r = 0; r < bq; ++r) {
        for (int t = 0; t < D; ++t) out[r * D + t] = O[r * D + t] / d[r];
        if (row_m) row_m[r] = m[r];
        if (row_d) row_d[r] = d[r];
        if (row_margin) row_margin[r] = marg[r];
        if (row_allow) {
            /* a weight change dw at key c (scale 2^(m_j - m_final)) moves output element t by
             * at most dw' * |v[c,t] - out[r,t]| / (d - dw'), summed over the near elements */
            double allow = 0.0;
            for (int j = 0; j < jmax; ++j) {
                double sc = exp2(scale_at[r * (S / bk) + j] - (g->exp2_only ? -lg[r] : m[r]));
                for (int cc = 0; cc < bk; ++cc) {
                    double dw = amb_dw[(size_t)r * S + j * bk + cc] * sc;
                    if (dw == 0.0) continue;
                    const float *vc = v + (size_t)(j * bk + cc) * D;
                    double worst = 0.0;
                    for (int t = 0; t < D; ++t)
                        worst = fmax(worst, fabs((double)vc[t] - out[r * D + t]));
                    double den = d[r] - dw; if (den < 0.5 * d[r]) den = 0.5 * d[r];
                    allow += dw * worst / den;
                }
            }
            row_allow[r] = allow;
        }
    }
    if (n_tiles) *n_tiles = tiles;
    free(Sc); free(T8); free(W); free(Walt); free(m); free(d); free(O); free(marg);
    free(amb_dw); free(scale_at); free(lg);
    return restarts;
}

/* Eq. (1) for one query tile, in double: softmax(Q K^T / sqrt(d)) V with the plain
 * max-subtracted exponential. */
static void exact_attention_tile(const tile_cfg *g, double scale, const float *q, const float *k,
                                 const float *v, int i0, double *out)
{
    const int D = g->D, S = g->S;
    double *p = (double *)malloc(sizeof(double) * S);
    for (int r = 0; r < g->bq; ++r) {
        int n = g->causal ? (i0 + r + 1) : S;
        double mx = -INFINITY;
        const float *qr = q + (size_t)(i0 + r) * D;
        for (int cidx = 0; cidx < n; ++cidx) {
            const float *kc = k + (size_t)cidx * D;
            double acc = 0.0;
            for (int t = 0; t < D; ++t) acc += (double)qr[t] * (double)kc[t];
            p[cidx] = acc * scale;
            mx = fmax(mx, p[cidx]);
        }
        double sum = 0.0;
        for (int cidx = 0; cidx < n; ++cidx) { p[cidx] = exp(p[cidx] - mx); sum += p[cidx]; }
        for (int t = 0; t < D; ++t) out[r * D + t] = 0.0;
        for (int cidx = 0; cidx < n; ++cidx) {
            const float *vc = v + (size_t)cidx * D;
            double w = p[cidx] / sum;
            for (int t = 0; t < D; ++t) out[r * D + t] += w * (double)vc[t];
        }
    }
    free(p);
}

/* Attention over a list of query tiles.
 *   q: [B, H, S, D]; k, v: [B, Hkv, S, D]; float32 holding the input values exactly
 *   (bf16 inputs are widened by the caller).  tiles: n_sel triples (b, h, i) selecting query
 *   tile i (rows i*bq ..) of head h of batch b.
 *   mode 0: Algorithm 1 with HiF8 roundings; 1: Eq. (1) exact; 2: the "Exp2 HiF8" setup;
 *   3 / 4: mode 0 / mode 2 with the roundings replaced by the identity (structure checks).
 *   b0_last != 0 (modes 0 and 3): B0 = {first, last visible tile} instead of {first}.
 *   Comparison setups of Section 4.2 (no margins / allowances are produced for them):
 *   5: Exp2 E4M3, 6: Exp2 E5M2, 7: Exp2 with E4M3 arguments and E5M2 results, 8: Naive E2E.
 *   out: [n_sel, bq, D] double.  Optional per selected tile: row_m, row_d, row_margin,
 *   row_allow: [n_sel, bq]; restarts, n_tiles: [n_sel].
 * Returns 0, or -1 on invalid arguments. */
int baps_oracle_attention(const float *q, const float *k, const float *v, double *out,
                          int B, int H, int Hkv, int S, int D, int causal, int bq, int bk,
                          int lambda, int mode, int b0_last, double scale, double eps_rel,
                          const int32_t *tiles, int64_t n_sel,
                          double *row_m, double *row_d, double *row_margin, double *row_allow,
                          int32_t *restarts, int32_t *n_tiles)
{
    if (B <= 0 || H <= 0 || Hkv <= 0 || H % Hkv || S <= 0 || D <= 0 || bq <= 0 || bk <= 0 ||
        S % bq || S % bk)
        return -1;
    hif8_init();
    if (scale == 0.0) scale = 1.0 / sqrt((double)D);
    const int gsz = H / Hkv;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < n_sel; ++t) {
        int b = tiles[3 * t], h = tiles[3 * t + 1], i = tiles[3 * t + 2];
        if (b < 0 || b >= B || h < 0 || h >= H || i < 0 || i >= S / bq) { err = 1; continue; }
        const float *qh = q + ((size_t)b * H + h) * (size_t)S * D;
        const float *kh = k + ((size_t)b * Hkv + h / gsz) * (size_t)S * D;
        const float *vh = v + ((size_t)b * Hkv + h / gsz) * (size_t)S * D;
        tile_cfg g;
        g.S = S; g.D = D; g.causal = causal; g.bq = bq; g.bk = bk; g.lambda = lambda;
        g.fmt = (mode == 3 || mode == 4) ? 1 : (mode == 5 || mode == 7) ? 2 : (mode == 6) ? 3 : 0;
        g.fmt_out = (mode == 6 || mode == 7) ? 3 : g.fmt;
        g.naive = (mode == 8) ? 1 : 0;
        g.exp2_only = (mode == 2 || mode == 4 || (mode >= 5 && mode <= 8)) ? 1 : 0;
        g.b0_last = (b0_last && !g.exp2_only) ? 1 : 0;
        g.c = 1.4426950408889634074 * scale;      /* log2(e) * scale */
        g.eps_rel = eps_rel;
        double *o = out + (size_t)t * bq * D;
        if (mode == 1) {
            exact_attention_tile(&g, scale, qh, kh, vh, i * bq, o);
            if (restarts) restarts[t] = 0;
            if (n_tiles) n_tiles[t] = 0;
        } else {
            int nt = 0;
            int rs = baps_tile(&g, qh, kh, vh, i * bq, o,
                               row_m ? row_m + t * bq : NULL, row_d ? row_d + t * bq : NULL,
                               row_margin ? row_margin + t * bq : NULL,
                               row_allow ? row_allow + t * bq : NULL, &nt);
            if (restarts) restarts[t] = rs;
            if (n_tiles) n_tiles[t] = nt;
        }
    }
    return err ? -1 : 0;
}

/* Row softmax: Algorithm 1 with one query row per "tile" and no V.  logits are natural-log
 * logits held in float32; s = logit * log2(e).  probs[c] = w[c] * 2^(m_block(c) - m_final) / d.
 * allow[c] (optional): |change of probs[c]| bound if near-boundary roundings of the row went
 * the other way (own weight flip plus the induced change of d).
 * row_margin (optional): as for attention. */
int baps_oracle_softmax_rows(const float *logits, double *probs, int64_t rows, int64_t cols,
                             int bk, int lambda, int fmt, double eps_rel,
                             double *row_margin, double *allow)
{
    if (rows < 0 || cols <= 0 || bk <= 0 || cols % bk) return -1;
    hif8_init();
    const double LOG2E = 1.4426950408889634074;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
        const float *x = logits + r * cols;
        double *p = probs + r * cols;
        double *dwv = (double *)calloc((size_t)cols, sizeof(double));
        double m = -INFINITY, d = 0.0, marg = INFINITY;
        int nb = (int)(cols / bk);
        double *mblk = (double *)malloc(sizeof(double) * nb);
        for (int j = 0; j < nb; ++j) {
            const float *xb = x + (int64_t)j * bk;
            double *pb = p + (int64_t)j * bk;
            double *db = dwv + (int64_t)j * bk;
            if (j == 0) {
                double rm = -INFINITY;
                for (int c = 0; c < bk; ++c) rm = fmax(rm, (double)xb[c] * LOG2E);
                double cm = ceil(rm);
                if (isfinite(rm))
                    marg = fmin(marg, fmin(cm - rm, rm - (cm - 1.0)) / fmax(1.0, fabs(rm)));
                double mnew = fmax(m, cm);
                double sum = 0.0;
                for (int c = 0; c < bk; ++c) {
                    double s = (double)xb[c] * LOG2E;
                    pb[c] = (s == -INFINITY) ? 0.0 : exp2(s - mnew);
                    sum += pb[c];
                }
                d = sum; m = mnew;
            } else {
                double tmax = -INFINITY, um = -INFINITY, sm = 0.0;
                for (int c = 0; c < bk; ++c) {
                    double s = (double)xb[c] * LOG2E;
                    if (s == -INFINITY) continue;
                    double t8 = round_T(s - m, fmt, NULL, NULL);
                    tmax = fmax(tmax, t8);
                    if (s - m > um) { um = s - m; sm = s; }
                }
                int restart = tmax > (double)lambda;
                double mnew, alpha;
                if (fmt == 0 && um != -INFINITY) {
                    double mg, altv, lam = (double)lambda;
                    double t8 = round_T(um, 0, &mg, &altv);
                    if ((t8 > lam) != (altv > lam) ||
                        (!restart && fmax(0.0, ceil(t8)) != fmax(0.0, ceil(altv))))
                        marg = fmin(marg, mg / fmax(1.0, fabs(sm)));
                }
                if (restart) {
                    double rm = um + m;          /* row max of S in this block */
                    double cm = ceil(rm);
                    if (cm >= m)
                        marg = fmin(marg, fmin(cm - rm, rm - (cm - 1.0)) / fmax(1.0, fabs(rm)));
                    mnew = fmax(m, cm);
                } else {
                    double delta = (tmax == -INFINITY) ? 0.0 : fmax(0.0, ceil(tmax));
                    mnew = m + delta;
                }
                alpha = exp2(m - mnew);
                double sum = 0.0;
                for (int c = 0; c < bk; ++c) {
                    double s = (double)xb[c] * LOG2E;
                    double w = 0.0, dw = 0.0;
                    if (s != -INFINITY) {
                        double mg, altv;
                        if (restart) {
                            double t8 = round_T(s - mnew, fmt, &mg, &altv);
                            w = exp2_8(t8, fmt);
                            if (fmt == 0 && mg < eps_rel * fmax(1.0, fabs(s)))
                                dw = fabs(exp2_8(altv, fmt) - w);
                        } else {
                            double t8 = round_T(s - m, fmt, &mg, &altv);
                            w = exp2_8(t8, fmt) * alpha;
                            if (fmt == 0 && mg < eps_rel * fmax(1.0, fabs(s)))
                                dw = fabs(exp2_8(altv, fmt) * alpha - w);
                        }
                    }
                    pb[c] = w; db[c] = dw; sum += w;
                }
                d = alpha * d + sum; m = mnew;
            }
            mblk[j] = m;
        }
        double amb_total = 0.0;
        for (int j = 0; j < nb; ++j) {
            double sc = exp2(mblk[j] - m);
            for (int c = 0; c < bk; ++c) {
                int64_t idx = (int64_t)j * bk + c;
                p[idx] = p[idx] * sc / d;
                dwv[idx] = dwv[idx] * sc / d;
                amb_total += dwv[idx];
            }
        }
        if (allow) {
            double *al = allow + r * cols;
            for (int64_t c = 0; c < cols; ++c) {
                double den = 1.0 - amb_total; if (den < 0.5) den = 0.5;
                al[c] = dwv[c] / den + p[c] * amb_total / den;
            }
        }
        if (row_margin) row_margin[r] = marg;
        free(dwv); free(mblk);
    }
    return 0;
}

/* Row softmax with 8-bit output: the weights leave as HiF8 codes with one integer exponent per
 * block and one denominator per row,
 *     probs[r, c] = value(codes[r, c]) * 2^(block_exp[r, c / bk]) / row_d[r],
 * i.e. 1 byte per element instead of 4.  Algorithm 1 per row as in baps_oracle_softmax_rows, with
 * two differences that belong to this variant: (1) block 0 is not kept in high precision -- its
 * weights go through the 8-bit exponential like all others (the output has 8 bits anyway); its
 * maximum still initialises the integer max; (2) because codes are compared bit for bit, T and the
 * max decisions are formed in single precision exactly as the CUDA kernel forms them:
 * T = fl32(x * fl32(log2 e) - mref) with one rounding (a fused multiply-add), block-0 / restart max
 * = ceil(fl32(xmax * fl32(log2 e))).  (The product of two floats is exact in double, and so is the
 * subtraction of the integer max, so "(float)(double expression)" is that single rounding.)
 * block_exp[r, j] = mref_j - m_final <= 0 where mref_j is the max block j's T were taken against. */
int baps_oracle_softmax_rows_codes(const float *logits, uint8_t *codes, int32_t *block_exp, double *row_d,
                                   int64_t rows, int64_t cols, int bk, int lambda)
{
    if (rows < 0 || cols <= 0 || bk <= 0 || cols % bk) return -1;
    hif8_init();
    const double C = (double)(float)1.4426950408889634074;
    const int nb = (int)(cols / bk);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
        const float *x = logits + r * cols;
        double *mref = (double *)malloc(sizeof(double) * nb);
        double m = -INFINITY;
        for (int j = 0; j < nb; ++j) {
            float xmax = -INFINITY;
            for (int c = 0; c < bk; ++c) xmax = fmaxf(xmax, x[(int64_t)j * bk + c]);
            if (j == 0) {
                m = ceil((double)(float)((double)xmax * C));
                mref[j] = m;
            } else {
                double u = (double)(float)((double)xmax * C - m);
                if (u <= 0.0) { mref[j] = m; continue; }
                double t8 = baps_oracle_hif8_value(hif8_encode_one(u, NULL, NULL));
                if (t8 > (double)lambda) {
                    m = fmax(m, ceil((double)(float)((double)xmax * C)));
                    mref[j] = m;                       /* restart: T against the new max */
                } else {
                    mref[j] = m;                       /* T against the old max, then m += delta */
                    m += fmax(0.0, ceil(t8));
                }
            }
        }
        double d = 0.0;
        for (int j = 0; j < nb; ++j) {
            const double sc = exp2(mref[j] - m);
            block_exp[r * nb + j] = (int32_t)(mref[j] - m);
            for (int c = 0; c < bk; ++c) {
                int64_t idx = (int64_t)j * bk + c;
                double t = (double)(float)((double)x[idx] * C - mref[j]);
                uint8_t tc = hif8_encode_one(t, NULL, NULL);
                uint8_t pc = baps_oracle_exp2_code(tc);
                codes[r * cols + idx] = pc;
                d += baps_oracle_hif8_value(pc) * sc;
            }
        }
        row_d[r] = d;
        free(mref);
    }
    return 0;
}

int baps_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
