/*
 * CPU oracle for the QuantPipe activation-quantization path (arXiv 2211.04515, Sec. 3).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, single-threaded C with fp64 accumulation.
 * It is written from the paper, shares no code with the CUDA library, and is used only by
 * the tests, the smoke check and the benchmark's CPU-baseline leg.  Nothing in the product
 * path may call it.
 *
 * What the paper fixes and what it leaves open
 *   - Statistics of the tensor: min / max (Sec. 3 "Naive PTQ and ACIQ"), the Laplace scale
 *     estimated from the data, b_E = sum|X| / N (Sec. 3 "Directed Search").
 *   - ACIQ: clip alpha = F(q) * b under a Laplace model L(mu, b) (Sec. 3).  F(q) is the
 *     minimiser of the Laplace clipping-plus-rounding error model of Banner et al.; it is
 *     solved here from that model, not tabulated.
 *   - Directed search (Eq. 1): t-step numeric search of b* between b_E and
 *     b_R = 1 / (2 max(D_R)), D_R the histogram density of the data, keeping b_E unless a
 *     step has strictly lower MSE.
 *   - Uniform quantizer: equal intervals over the clip range, round to nearest (Sec. 3).
 *   - Bit-width from bandwidth: Eq. 2, and the principle of Sec. 1 that the widest
 *     code that still meets the target rate on the measured link is the one to use.
 *   The packing layout, the rounding mode, the histogram's bin count and the treatment of
 *   non-finite values are not given by the paper; the readings taken are stated at each
 *   function.
 *
 * Parity pins (tests/test_oracle_*.py): every exported function is pinned to something
 * other than itself (closed forms, SciPy, brute force, hand-worked examples, the paper's
 * bandwidth-phase run).  No function here is "parity unpinned".
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#if FLT_EVAL_METHOD != 0
#error "float expressions must be evaluated in float (no excess precision)"
#endif
#if defined(__FAST_MATH__)
#error "build without -ffast-math"
#endif

/* ------------------------------------------------------------------ types */

typedef struct {
    uint64_t n;          /* elements seen, finite or not                     */
    uint64_t nonfinite;  /* NaN and +-Inf; excluded from every other field   */
    double mean;         /* sum x / n_finite                                  */
    double mean_abs;     /* sum |x| / n_finite   (the paper's literal b_E)    */
    double mad;          /* sum |x - mean| / n_finite                         */
    double var;          /* sum (x - mean)^2 / n_finite                       */
    double min, max;     /* over finite elements                              */
} orc_stats_t;

typedef struct {
    float lo, hi;        /* clip range                                        */
    float scale;         /* (hi - lo) / (L - 1)                               */
    float inv_scale;     /* (L - 1) / (hi - lo)                               */
    int32_t bits;
    int32_t flags;       /* bit 0: degenerate range (hi <= lo), all codes 0   */
} orc_qparams_t;

typedef struct {
    double b_e, b_r, b_star, alpha_e, alpha_star, mse_e, mse_star;
    int32_t k_star, steps, hist_bins, bits;
} orc_ds_result_t;

enum { ORC_OK = 0, ORC_ERR_ARG = -1, ORC_ERR_BITS = -2, ORC_WARN_INFEASIBLE = 1, ORC_WARN_DEGENERATE = 2 };

/* ----------------------------------------------- compensated fp64 summation */

typedef struct { double s, c; } ksum_t;
static void ksum_add(ksum_t* k, double v)      /* Neumaier's variant of Kahan summation */
{
    double t = k->s + v;
    if (fabs(k->s) >= fabs(v)) k->c += (k->s - t) + v;
    else                       k->c += (v - t) + k->s;
    k->s = t;
}
static double ksum_get(const ksum_t* k) { return k->s + k->c; }

static int finite_f(float x) { return x == x && x != INFINITY && x != -INFINITY; }

/* ------------------------------------------------------------- statistics */

/* Per-tensor statistics (Sec. 3: min/max range of naive PTQ; mean and Laplace scale of
 * ACIQ; b_E of the directed search).  Non-finite elements are counted and skipped. */
void orc_stats(const float* x, uint64_t n, orc_stats_t* out)
{
    ksum_t sx = {0, 0}, sa = {0, 0};
    uint64_t nf = 0, bad = 0;
    double mn = INFINITY, mx = -INFINITY;
    for (uint64_t i = 0; i < n; ++i) {
        float v = x[i];
        if (!finite_f(v)) { ++bad; continue; }
        ++nf;
        ksum_add(&sx, (double)v);
        ksum_add(&sa, fabs((double)v));
        if ((double)v < mn) mn = (double)v;
        if ((double)v > mx) mx = (double)v;
    }
    memset(out, 0, sizeof *out);
    out->n = n;
    out->nonfinite = bad;
    if (nf == 0) return;
    double mean = ksum_get(&sx) / (double)nf;
    ksum_t sd = {0, 0}, sv = {0, 0};
    for (uint64_t i = 0; i < n; ++i) {
        float v = x[i];
        if (!finite_f(v)) continue;
        double d = (double)v - mean;
        ksum_add(&sd, fabs(d));
        ksum_add(&sv, d * d);
    }
    out->mean = mean;
    out->mean_abs = ksum_get(&sa) / (double)nf;
    out->mad = ksum_get(&sd) / (double)nf;
    out->var = ksum_get(&sv) / (double)nf;
    out->min = mn;
    out->max = mx;
}

/* ---------------------------------------------------------------- ACIQ F(q) */

/* Laplace: clipping noise 2 b^2 exp(-alpha/b), rounding noise alpha^2 / (3 * 4^q).
 * The derivative vanishes where (alpha/b) exp(alpha/b) = 3 * 4^q, so
 * F(q) = W0(3 * 4^q).  Newton's iteration on w exp(w) = z. */
double orc_aciq_F_laplace(int q)
{
    double z = 3.0 * pow(4.0, (double)q);
    double w = log(z) - log(log(z) > 1.0 ? log(z) : 1.0);
    for (int it = 0; it < 100; ++it) {
        double e = exp(w);
        double f = w * e - z;
        double step = f / (e * (w + 1.0));
        w -= step;
        if (fabs(step) <= 1e-15 * fabs(w)) break;
    }
    return w;
}

/* Gaussian N(mu, sigma): clipping noise 2 sigma^2 [(1+a^2)(1-Phi(a)) - a phi(a)] with
 * a = alpha/sigma, plus the same rounding term.  The derivative
 * 4 [a (1-Phi(a)) - phi(a)] + 2a / (3 * 4^q) changes sign once; bisection. */
static double gauss_dmodel(double a, double q4)
{
    double tail = 0.5 * erfc(a / sqrt(2.0));
    double pdf = exp(-0.5 * a * a) / sqrt(2.0 * M_PI);
    return 4.0 * (a * tail - pdf) + 2.0 * a / (3.0 * q4);
}
double orc_aciq_F_gauss(int q)
{
    double q4 = pow(4.0, (double)q);
    double lo = 0.0, hi = 40.0;            /* derivative < 0 at 0, > 0 at 40 */
    for (int it = 0; it < 200; ++it) {
        double mid = 0.5 * (lo + hi);
        if (gauss_dmodel(mid, q4) < 0.0) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

static int bits_ok(int bits) { return (bits >= 1 && bits <= 8) || bits == 16; }

/* ------------------------------------------------------------- quantizer */

/* Uniform quantizer over [lo, hi] with L = 2^bits levels including both ends, i.e. L - 1
 * equal intervals and rounding to the nearest level (Sec. 3, uniform quantization).  The clip range
 * is rounded to fp32 once; scale and its reciprocal are derived in fp64 from the rounded
 * ends and rounded once. */
int orc_make_qparams(double lo, double hi, int bits, orc_qparams_t* qp)
{
    if (!bits_ok(bits)) return ORC_ERR_BITS;
    if (!(lo == lo) || !(hi == hi) || isinf(lo) || isinf(hi)) return ORC_ERR_ARG;
    double levels_m1 = (double)((1u << bits) - 1u);
    float lo_f = (float)lo, hi_f = (float)hi;
    qp->lo = lo_f;
    qp->hi = hi_f;
    qp->bits = bits;
    qp->flags = 0;
    if (!(hi_f > lo_f) || isinf(lo_f) || isinf(hi_f)) {
        qp->scale = 0.0f;
        qp->inv_scale = 0.0f;
        qp->flags = 1;
        return ORC_WARN_DEGENERATE;
    }
    double range = (double)hi_f - (double)lo_f;
    qp->scale = (float)(range / levels_m1);
    qp->inv_scale = (float)(levels_m1 / range);
    return ORC_OK;
}

/* One element: clamp (NaN goes to lo), offset and scale as two separately rounded fp32
 * operations, round half to even, clamp the code to [0, L-1]. */
static uint32_t quantize_one(float x, const orc_qparams_t* qp)
{
    float t = (x > qp->lo) ? x : qp->lo;       /* false for NaN -> lo */
    t = (t < qp->hi) ? t : qp->hi;
    float d = t - qp->lo;                      /* each op rounded to fp32 on its own:  */
    float v = d * qp->inv_scale;               /* no contraction, no excess precision   */
    float r = rintf(v);                        /* default rounding mode: ties to even */
    int32_t top = (int32_t)((1u << qp->bits) - 1u);
    int32_t c = (int32_t)r;
    if (c < 0) c = 0;
    if (c > top) c = top;
    return (uint32_t)c;
}

/* Receiver's inverse map: lo + code * scale, evaluated in extended precision (the product
 * is exact) and rounded to fp32. */
static float dequantize_one(uint32_t code, const orc_qparams_t* qp)
{
    long double v = (long double)qp->lo + (long double)code * (long double)qp->scale;
    return (float)v;
}

void orc_quantize(const float* x, uint64_t n, const orc_qparams_t* qp, uint32_t* codes)
{
    for (uint64_t i = 0; i < n; ++i) codes[i] = quantize_one(x[i], qp);
}

void orc_dequantize(const uint32_t* codes, uint64_t n, const orc_qparams_t* qp, float* y)
{
    for (uint64_t i = 0; i < n; ++i) y[i] = dequantize_one(codes[i], qp);
}

/* Mean squared error between the tensor and its quantize->dequantize image (the paper's
 * quality measure, Sec. 3), over the finite elements. */
double orc_quant_mse(const float* x, uint64_t n, const orc_qparams_t* qp)
{
    ksum_t s = {0, 0};
    uint64_t nf = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (!finite_f(x[i])) continue;
        ++nf;
        double e = (double)dequantize_one(quantize_one(x[i], qp), qp) - (double)x[i];
        ksum_add(&s, e * e);
    }
    return nf ? ksum_get(&s) / (double)nf : 0.0;
}

/* ------------------------------------------------- per-channel quantization */

int orc_clip_range(const orc_stats_t* st, int bits, int method, int flags, int dist, int bmode,
                   double* lo_out, double* hi_out, orc_qparams_t* qp);   /* defined with the ACIQ clip below */

/* Channel-wise variant of the per-tensor method (Sec. 3 applies one clip range to the whole
 * tensor; channel-wise ranges are the alternative the paper's cited PTQ work uses for
 * activations with outlier channels).  The tensor is [rows, channels], row-major, so element
 * i belongs to channel i mod channels; every channel gets the statistics, the clip range and
 * the quantizer that the per-tensor functions give for its column alone, and all channels
 * share the bit-width and the packed layout. */

/* Statistics of each column: out[c] = orc_stats of x[c], x[c + channels], ... */
int orc_stats_channels(const float* x, uint64_t rows, uint64_t channels, orc_stats_t* out)
{
    if (channels < 1) return ORC_ERR_ARG;
    float* col = (float*)malloc((size_t)(rows ? rows : 1) * sizeof(float));
    if (!col) return ORC_ERR_ARG;
    for (uint64_t c = 0; c < channels; ++c) {
        for (uint64_t r = 0; r < rows; ++r) col[r] = x[r * channels + c];
        orc_stats(col, rows, &out[c]);
    }
    free(col);
    return ORC_OK;
}

/* Quantizer of each channel from its statistics (orc_clip_range per channel).  Returns
 * ORC_WARN_DEGENERATE if any channel has an empty range (that channel's codes are all 0). */
int orc_clip_channels(const orc_stats_t* st, uint64_t channels, int bits, int method, int flags, int dist,
                      int bmode, orc_qparams_t* qp)
{
    int worst = ORC_OK;
    for (uint64_t c = 0; c < channels; ++c) {
        int rc = orc_clip_range(&st[c], bits, method, flags, dist, bmode, NULL, NULL, &qp[c]);
        if (rc < 0) return rc;
        if (rc == ORC_WARN_DEGENERATE) worst = rc;
    }
    return worst;
}

void orc_quantize_channels(const float* x, uint64_t rows, uint64_t channels, const orc_qparams_t* qp, uint32_t* codes)
{
    for (uint64_t i = 0; i < rows * channels; ++i) codes[i] = quantize_one(x[i], &qp[i % channels]);
}

void orc_dequantize_channels(const uint32_t* codes, uint64_t rows, uint64_t channels, const orc_qparams_t* qp, float* y)
{
    for (uint64_t i = 0; i < rows * channels; ++i) y[i] = dequantize_one(codes[i], &qp[i % channels]);
}

/* Token-wise variant: the other axis of the same idea.  The tensor is [tokens, channels], row-major,
 * and every token (a row of `channels` contiguous elements, one position of a ViT sequence) gets the
 * statistics, the clip range and the quantizer that the per-tensor functions give for its row alone
 * (Sec. 3's method with the row in place of the tensor; the paper clips per tensor).  Bit-width and
 * packed layout are shared.  The clip ranges come from orc_clip_channels, which only maps an array
 * of statistics to an array of quantizers and does not care what the entries stand for. */

/* Statistics of each row: out[t] = orc_stats of x[t * channels .. (t + 1) * channels). */
int orc_stats_tokens(const float* x, uint64_t tokens, uint64_t channels, orc_stats_t* out)
{
    if (channels < 1) return ORC_ERR_ARG;
    for (uint64_t t = 0; t < tokens; ++t) orc_stats(x + t * channels, channels, &out[t]);
    return ORC_OK;
}

void orc_quantize_tokens(const float* x, uint64_t tokens, uint64_t channels, const orc_qparams_t* qp, uint32_t* codes)
{
    for (uint64_t i = 0; i < tokens * channels; ++i) codes[i] = quantize_one(x[i], &qp[i / channels]);
}

void orc_dequantize_tokens(const uint32_t* codes, uint64_t tokens, uint64_t channels, const orc_qparams_t* qp, float* y)
{
    for (uint64_t i = 0; i < tokens * channels; ++i) y[i] = dequantize_one(codes[i], &qp[i / channels]);
}

/* ----------------------------------------------------------------- packing */

/* Packed length: ceil(n * bits / 8) bytes rounded up to a multiple of 16. */
uint64_t orc_packed_bytes(uint64_t n, int bits)
{
    uint64_t raw = (n * (uint64_t)bits + 7u) / 8u;
    return (raw + 15u) / 16u * 16u;
}

/* Element i owns stream bits [i*bits, (i+1)*bits), least significant code bit first;
 * stream bit j is bit (j mod 8) of byte (j div 8).  Pad bits are zero.  One bit at a time. */
void orc_pack(const uint32_t* codes, uint64_t n, int bits, uint8_t* out)
{
    memset(out, 0, (size_t)orc_packed_bytes(n, bits));
    for (uint64_t i = 0; i < n; ++i)
        for (int b = 0; b < bits; ++b) {
            uint64_t j = i * (uint64_t)bits + (uint64_t)b;
            if ((codes[i] >> b) & 1u) out[j >> 3] |= (uint8_t)(1u << (j & 7u));
        }
}

void orc_unpack(const uint8_t* in, uint64_t n, int bits, uint32_t* codes)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t c = 0;
        for (int b = 0; b < bits; ++b) {
            uint64_t j = i * (uint64_t)bits + (uint64_t)b;
            c |= (uint32_t)((in[j >> 3] >> (j & 7u)) & 1u) << b;
        }
        codes[i] = c;
    }
}

/* ------------------------------------------------------------- ACIQ clip */

/* alpha = F(q) * b, clip range [mean - alpha, mean + alpha] (Sec. 3, ACIQ under L(mu, b)).
 * dist 0: Laplace, b = mean absolute deviation about the mean (bmode 0) or the paper's
 *         literal sum|X|/N (bmode 1).  dist 1: Gaussian, b = standard deviation.
 * b_override > 0 replaces the estimated b (used with the directed search's b*). */
int orc_aciq_alpha(const orc_stats_t* st, int bits, int dist, int bmode, double b_override,
                   double* alpha_out, orc_qparams_t* qp)
{
    if (!bits_ok(bits)) return ORC_ERR_BITS;
    if ((dist != 0 && dist != 1) || (bmode != 0 && bmode != 1)) return ORC_ERR_ARG;
    double b = b_override > 0.0 ? b_override
             : dist == 1        ? sqrt(st->var)
             : bmode == 1       ? st->mean_abs
                                : st->mad;
    double F = dist == 1 ? orc_aciq_F_gauss(bits) : orc_aciq_F_laplace(bits);
    double alpha = F * b;
    if (alpha_out) *alpha_out = alpha;
    if (qp) return orc_make_qparams(st->mean - alpha, st->mean + alpha, bits, qp);
    return ORC_OK;
}

/* Mid-rise grid on a clip range (the other reading of Sec. 3's "divides the data range into
 * equal intervals": 2^q equal bins over [lo, hi], every element reconstructed at the centre of
 * its bin - the grid that the ACIQ noise term alpha^2 / (3 * 4^q) models).  With bin width
 * w = (hi - lo) / 2^q the centres are lo + w/2, lo + 3w/2, ..., hi - w/2: exactly the 2^q levels
 * of the uniform quantizer on [lo + w/2, hi - w/2], whose rounding boundaries are the bin
 * edges.  So the grid is a change of the clip range and nothing else. */
void orc_midrise_range(double lo, double hi, int bits, double* lo_out, double* hi_out)
{
    double half = (hi - lo) / ldexp(1.0, bits + 1);
    *lo_out = lo + half;
    *hi_out = hi - half;
}

/* Clip range by method (Sec. 3, "Naive PTQ and ACIQ").
 *   method 0  ACIQ: [mean - alpha, mean + alpha] with alpha = F(q) b, as orc_aciq_alpha
 *   method 2  naive PTQ: the tensor's own [min, max]
 * flags bit 0 (method 0 only): the ACIQ range cut back to the data's range,
 *   [max(mean - alpha, min), min(mean + alpha, max)].  No element lies outside [min, max], so
 *   the clipping error is unchanged while the step gets smaller whenever alpha reaches past
 *   the data.  This is a variant of this library; the paper clips at mean -/+ alpha only.
 * flags bit 1: mid-rise grid on the resulting range (orc_midrise_range), applied last. */
int orc_clip_range(const orc_stats_t* st, int bits, int method, int flags, int dist, int bmode,
                   double* lo_out, double* hi_out, orc_qparams_t* qp)
{
    if (!bits_ok(bits)) return ORC_ERR_BITS;
    if (method != 0 && method != 2) return ORC_ERR_ARG;
    if (flags < 0 || flags > 3 || (method == 2 && (flags & 1))) return ORC_ERR_ARG;
    double lo, hi;
    if (method == 2) {
        lo = st->min;
        hi = st->max;
    } else {
        double alpha;
        int rc = orc_aciq_alpha(st, bits, dist, bmode, 0.0, &alpha, NULL);
        if (rc < 0) return rc;
        lo = st->mean - alpha;
        hi = st->mean + alpha;
        if (flags & 1) {
            if (st->min > lo) lo = st->min;
            if (st->max < hi) hi = st->max;
        }
    }
    if (flags & 2) orc_midrise_range(lo, hi, bits, &lo, &hi);
    if (lo_out) *lo_out = lo;
    if (hi_out) *hi_out = hi;
    if (qp) return orc_make_qparams(lo, hi, bits, qp);
    return ORC_OK;
}

/* ------------------------------------------------------- histogram of D_R */

/* Density histogram D_R of the data, nb equal bins over [min, max] (Sec. 3, directed
 * search: only its peak is used).  Bin index in fp32:
 * floor((x - min) * inv_w), inv_w = (float)(nb / (max - min)), last bin closed.
 * Returns the peak density max_j count_j / (n_finite * w); counts (nb entries) optional. */
double orc_hist_peak(const float* x, uint64_t n, double mn, double mx, int nb, uint64_t* counts_out)
{
    if (nb < 1 || !(mx > mn)) return 0.0;
    uint64_t* counts = (uint64_t*)calloc((size_t)nb, sizeof(uint64_t));
    float mn_f = (float)mn;
    float inv_w = (float)((double)nb / (mx - mn));
    uint64_t nf = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (!finite_f(x[i])) continue;
        float d = x[i] - mn_f;
        float p = d * inv_w;
        float fl = floorf(p);
        int64_t idx = (int64_t)fl;
        if (idx < 0) idx = 0;
        if (idx > nb - 1) idx = nb - 1;
        ++counts[idx];
        ++nf;
    }
    uint64_t top = 0;
    for (int j = 0; j < nb; ++j) if (counts[j] > top) top = counts[j];
    if (counts_out) memcpy(counts_out, counts, (size_t)nb * sizeof(uint64_t));
    free(counts);
    if (nf == 0) return 0.0;
    double w = (mx - mn) / (double)nb;
    return (double)top / ((double)nf * w);
}

/* --------------------------------------------------------- directed search */

/* DS-ACIQ (Sec. 3 "Directed Search", Eq. 1).
 *   b_E      Laplace scale estimated from the data (bmode as in orc_aciq_alpha)
 *   max(D_E) = 1 / (2 b_E), the peak of the Laplace density with scale b_E
 *   b_R      = 1 / (2 max(D_R)), D_R the histogram density of the data
 *   b_k      = b_E + k (b_R - b_E) / t,  k = 0..t   (towards b_R, whichever side it lies)
 *   mse_k    = quantization MSE of the tensor with clip alpha_k = F(q) b_k about the mean
 *              (bmode | 0x10: on the mid-rise grid, orc_midrise_range)
 *   k*       = smallest k attaining the minimum; k = 0 is b_E itself, so b_E is kept
 *              unless some step is strictly better.
 * bmode | 0x20: the same search under the Gaussian model that ACIQ also offers (a variant of
 *   this library; the paper searches under the Laplace model only).  The scale is the
 *   standard deviation: sigma_E = sqrt(var); the peak of N(mu, sigma) is 1 / (sigma sqrt(2 pi)),
 *   so sigma_R = 1 / (sqrt(2 pi) max(D_R)); sigma_k between them as above, alpha_k = F_G(q) sigma_k.
 *   The result's b_e, b_r, b_star then hold sigma_E, sigma_R, sigma*.
 * mse_curve (t+1 doubles) optional. */
int orc_ds_search(const float* x, uint64_t n, const orc_stats_t* st, int bits, int bmode,
                  int steps, int hist_bins, orc_ds_result_t* res, orc_qparams_t* qp_out,
                  double* mse_curve)
{
    if (!(bits >= 1 && bits <= 8)) return ORC_ERR_BITS;
    int midrise = (bmode & 0x10) != 0;                     /* every candidate on the mid-rise grid */
    int gauss = (bmode & 0x20) != 0;                       /* Gaussian model: scale = standard deviation */
    bmode &= ~0x30;
    if (steps < 1 || hist_bins < 1 || (bmode != 0 && bmode != 1) || (gauss && bmode != 0)) return ORC_ERR_ARG;
    double F = gauss ? orc_aciq_F_gauss(bits) : orc_aciq_F_laplace(bits);
    double b_e = gauss ? sqrt(st->var) : (bmode == 1 ? st->mean_abs : st->mad);
    double peak = orc_hist_peak(x, n, st->min, st->max, hist_bins, NULL);
    int degenerate = !(st->max > st->min) || !(peak > 0.0) || !(b_e > 0.0);
    double peak_factor = gauss ? sqrt(2.0 * 3.14159265358979323846) : 2.0;   /* density peak = 1 / (factor * scale) */
    double b_r = degenerate ? b_e : 1.0 / (peak_factor * peak);
    memset(res, 0, sizeof *res);
    res->b_e = b_e;
    res->b_r = b_r;
    res->steps = steps;
    res->hist_bins = hist_bins;
    res->bits = bits;
    int best_k = 0;
    double best_mse = 0.0;
    orc_qparams_t qp, best_qp;
    for (int k = 0; k <= steps; ++k) {
        double b_k = b_e + (double)k * (b_r - b_e) / (double)steps;
        double mse;
        if (k > 0 && (degenerate || !(b_k > 0.0))) {
            mse = INFINITY;                                  /* not a candidate */
        } else {
            double alpha = F * b_k;
            double lo = st->mean - alpha, hi = st->mean + alpha;
            if (midrise) orc_midrise_range(lo, hi, bits, &lo, &hi);
            orc_make_qparams(lo, hi, bits, &qp);
            mse = orc_quant_mse(x, n, &qp);
        }
        if (mse_curve) mse_curve[k] = mse;
        if (k == 0) { res->mse_e = mse; best_mse = mse; best_qp = qp; }
        else if (mse < best_mse) { best_mse = mse; best_k = k; best_qp = qp; }
    }
    res->k_star = best_k;
    res->b_star = b_e + (double)best_k * (b_r - b_e) / (double)steps;
    res->alpha_e = F * b_e;
    res->alpha_star = F * res->b_star;
    res->mse_star = best_mse;
    if (qp_out) *qp_out = best_qp;
    return degenerate ? ORC_WARN_DEGENERATE : ORC_OK;
}

/* The directed search run for every channel of a [rows, channels] tensor on its column alone
 * (channel-wise variant, see orc_stats_channels): res[c], qp[c] and, if curves is not NULL,
 * curves[c * (steps + 1) + k] are what orc_ds_search gives for column c with statistics st[c].
 * Returns ORC_WARN_DEGENERATE if any channel's search was degenerate. */
int orc_ds_search_channels(const float* x, uint64_t rows, uint64_t channels, const orc_stats_t* st, int bits,
                           int bmode, int steps, int hist_bins, orc_ds_result_t* res, orc_qparams_t* qp,
                           double* curves)
{
    if (channels < 1) return ORC_ERR_ARG;
    float* col = (float*)malloc((size_t)(rows ? rows : 1) * sizeof(float));
    if (!col) return ORC_ERR_ARG;
    int worst = ORC_OK;
    for (uint64_t c = 0; c < channels; ++c) {
        for (uint64_t r = 0; r < rows; ++r) col[r] = x[r * channels + c];
        int rc = orc_ds_search(col, rows, &st[c], bits, bmode, steps, hist_bins, &res[c], &qp[c],
                               curves ? curves + c * (uint64_t)(steps + 1) : NULL);
        if (rc < 0) { free(col); return rc; }
        if (rc == ORC_WARN_DEGENERATE) worst = rc;
    }
    free(col);
    return worst;
}

/* -------------------------------------------------------- bit-width choice */

/* Widest allowed code whose payload fits the link budget (the selection principle of
 * Sec. 1 / Sec. 3 "Adaptive PDA"): 8 * (ceil(n*q/8) + overhead_bytes) <= bandwidth_bps * budget_s.
 * q = 32 stands for the raw fp32 tensor.  Nothing fits: smallest allowed, with a warning. */
int orc_select_bits(double bandwidth_bps, double budget_s, uint64_t n_elems, uint64_t overhead_bytes,
                    const int32_t* allowed, int n_allowed, int32_t* bits_out)
{
    if (n_allowed < 1 || !(bandwidth_bps >= 0.0) || !(budget_s >= 0.0)) return ORC_ERR_ARG;
    double capacity_bits = bandwidth_bps * budget_s;
    int best = -1, smallest = allowed[0];
    for (int i = 0; i < n_allowed; ++i) {
        int q = allowed[i];
        if (q < 1 || q > 32) return ORC_ERR_ARG;
        if (q < smallest) smallest = q;
        double payload_bits = 8.0 * ((double)((n_elems * (uint64_t)q + 7u) / 8u) + (double)overhead_bytes);
        if (payload_bits <= capacity_bits && q > best) best = q;
    }
    if (best < 0) { *bits_out = smallest; return ORC_WARN_INFEASIBLE; }
    *bits_out = best;
    return ORC_OK;
}

/* Eq. 2 as printed:  q' = 32 / 2^ceil(log2( (V * 32 / q) / ((S / R) * B) )).
 * V in bytes at the current bit-width q, B in bit/s, S images per microbatch, R images/s.
 * The logarithm's base is not printed; base 2 makes q' the fp32 width halved until the
 * transfer fits.  Result clamped to [1, 32]. */
int orc_select_bits_eq2(double v_bytes, int q_t, double s_images, double r_images_per_s,
                        double bandwidth_bps, int32_t* bits_out)
{
    if (!(v_bytes > 0.0) || q_t < 1 || q_t > 32 || !(s_images > 0.0) || !(r_images_per_s > 0.0) ||
        !(bandwidth_bps > 0.0))
        return ORC_ERR_ARG;
    double full_bits = v_bytes * 8.0 * 32.0 / (double)q_t;
    double c = full_bits / ((s_images / r_images_per_s) * bandwidth_bps);
    double e = ceil(log2(c));
    double q = 32.0 / pow(2.0, e);
    if (q > 32.0) q = 32.0;
    if (q < 1.0) q = 1.0;
    *bits_out = (int32_t)q;
    return ORC_OK;
}

/* --------------------------------------------------------- adaptive controller */

/* The runtime loop of Sec. 3 "Adaptive PDA" / Sec. 4.2, one microbatch at a time: transfers
 * are averaged over a window of microbatches; when a window closes, the link bandwidth is
 * total bits over total seconds, and if it moved by more than rel_change relative to the
 * bandwidth of the last decision, the width is chosen again for the budget S / R per
 * microbatch (mode 0: widest allowed width that fits; mode 1: Eq. 2 as printed). */
typedef struct {
    int32_t window, count, bits, mode;
    double s_images, r_images_per_s;
    uint64_t n_elems, overhead_bytes;
    double rel_change, sum_bytes, sum_seconds, ref_bw;
    int32_t n_allowed;
    int32_t allowed[8];
} orc_controller_t;

void orc_controller_init(orc_controller_t* c, int window, double s_images, double r_images_per_s, uint64_t n_elems,
                         uint64_t overhead_bytes, const int32_t* allowed, int n_allowed, int mode, double rel_change,
                         int initial_bits)
{
    memset(c, 0, sizeof *c);
    c->window = window;
    c->bits = initial_bits;
    c->mode = mode;
    c->s_images = s_images;
    c->r_images_per_s = r_images_per_s;
    c->n_elems = n_elems;
    c->overhead_bytes = overhead_bytes;
    c->rel_change = rel_change;
    c->n_allowed = n_allowed;
    for (int i = 0; i < n_allowed; ++i) c->allowed[i] = allowed[i];
}

/* returns 1 if this microbatch closed a window and a new decision was taken */
int orc_controller_observe(orc_controller_t* c, double bytes_sent, double seconds, int32_t* bits_out)
{
    c->sum_bytes += bytes_sent;
    c->sum_seconds += seconds;
    c->count += 1;
    *bits_out = c->bits;
    if (c->count < c->window) return 0;
    double bw = c->sum_seconds > 0.0 ? 8.0 * c->sum_bytes / c->sum_seconds : 0.0;
    c->count = 0;
    c->sum_bytes = 0.0;
    c->sum_seconds = 0.0;
    if (!(bw > 0.0)) return 0;
    if (c->ref_bw > 0.0 && fabs(bw - c->ref_bw) <= c->rel_change * c->ref_bw) return 0;
    int32_t q = c->bits;
    if (c->mode == 1) {
        double v = (double)((c->n_elems * (uint64_t)c->bits + 7u) / 8u + c->overhead_bytes);
        if (orc_select_bits_eq2(v, c->bits, c->s_images, c->r_images_per_s, bw, &q) < 0) return 0;
    } else {
        if (orc_select_bits(bw, c->s_images / c->r_images_per_s, c->n_elems, c->overhead_bytes, c->allowed,
                            c->n_allowed, &q) < 0)
            return 0;
    }
    c->ref_bw = bw;
    c->bits = q;
    *bits_out = q;
    return 1;
}
