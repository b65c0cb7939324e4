/*
 * CPU oracle for the residual-VQ KV-cache compressor -- TEST INFRASTRUCTURE.
 *
 * A plain, slow, double-precision restatement of what the paper defines:
 *   - Section 2.2: scale a vector by its standard deviation, split the
 *     channels into groups, quantize every group with the same residual
 *     quantizer, output = sum of the chosen codes times the standard
 *     deviation;
 *   - Algorithm 1: the greedy residual loop (nearest code, subtract, repeat);
 *   - Section 3.1: contiguous groups, or groups of channels d/d^ apart;
 *   - Section 3.2: the standard deviation is kept in half precision;
 *   - Section 3 / Section 2.1: codebooks follow an exponential moving average
 *     (decay 0.99) of per-code counts and sums.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.  It shares no code with the CUDA library and nothing in the CUDA
 * library calls it.  No blocking, fusion or reordering: every loop is the
 * definition written out, so it can be checked against the paper by eye.
 *
 * Readings the paper leaves open (all are this oracle's, not the paper's):
 *   - the standard deviation is over one head vector, population form by
 *     default (ddof = 0), x is not centred;                 [parity unpinned]
 *   - vectors are scaled by the unrounded deviation, the stored value is its
 *     fp16 rounding, decode multiplies by the stored value;
 *   - exact distance ties go to the lowest index;
 *   - the EMA normalisation is the VQ-VAE one with Laplace smoothing,
 *     N^ = (N + eps) * sum(N) / (sum(N) + K * eps), C = M / N^; [parity unpinned]
 *   - a zero or non-finite deviation gives codes 0 and a stored deviation 0.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define RVQ_CONTIGUOUS 0
#define RVQ_STRIDED 1

/* Section 3.1: element i of group g is channel g*gd+i (contiguous) or
 * channel i*G+g, i.e. channels G = d/d^ apart (non-contiguous). */
static inline int chan_of(int layout, int G, int gd, int g, int i)
{
    return layout == RVQ_STRIDED ? i * G + g : g * gd + i;
}

/* Round a double to a binary format with p significand bits (implicit one
 * included), minimum normal exponent emin and maximum exponent emax, nearest
 * even, gradual underflow, overflow to infinity. */
static double round_fmt(double v, int p, int emin, int emax)
{
    if (v == 0.0 || !isfinite(v)) return v;
    int e;
    (void)frexp(v, &e);
    int ex = e - 1;
    if (ex < emin) ex = emin;
    double q = ldexp(1.0, ex - (p - 1));
    double r = nearbyint(v / q) * q;           /* default rounding mode: nearest even */
    double maxfin = (2.0 - ldexp(1.0, 1 - p)) * ldexp(1.0, emax);
    if (fabs(r) > maxfin) r = copysign(INFINITY, v);
    return r;
}

double rvq_oracle_round_scalar(double v, int dtype)
{
    switch (dtype) {
    case 0: return round_fmt(v, 24, -126, 127);   /* fp32 */
    case 1: return round_fmt(v, 8, -126, 127);    /* bf16 */
    case 2: return round_fmt(v, 11, -14, 15);     /* fp16 */
    default: return v;
    }
}

void rvq_oracle_round(const double *in, int64_t count, int dtype, double *out)
{
    for (int64_t i = 0; i < count; ++i) out[i] = rvq_oracle_round_scalar(in[i], dtype);
}

/* IEEE binary16 bit pattern of an fp16-representable double. */
static uint16_t f16_bits(double r)
{
    uint16_t sign = signbit(r) ? 0x8000u : 0u;
    double a = fabs(r);
    if (isnan(r)) return 0x7E00u;
    if (isinf(r)) return (uint16_t)(sign | 0x7C00u);
    if (a == 0.0) return sign;
    int e;
    double m = frexp(a, &e);                    /* a = m * 2^e, 0.5 <= m < 1 */
    int ex = e - 1;
    if (ex < -14) return (uint16_t)(sign | (uint16_t)ldexp(a, 24));  /* subnormal: units of 2^-24 */
    uint16_t frac = (uint16_t)(ldexp(m, 11) - 1024.0);
    return (uint16_t)(sign | ((uint16_t)(ex + 15) << 10) | frac);
}

uint16_t rvq_oracle_f64_to_f16_bits(double v) { return f16_bits(round_fmt(v, 11, -14, 15)); }

double rvq_oracle_f16_bits_to_f64(uint16_t h)
{
    int s = h >> 15, e = (h >> 10) & 31, f = h & 1023;
    double v;
    if (e == 31) v = f ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)f, -24);
    else v = ldexp(1024.0 + f, e - 25);
    return s ? -v : v;
}

/* Section 2.2 (x is scaled by its own standard deviation): mu = mean(x),
 * s = sqrt(sum((x-mu)^2) / (d - ddof)).  x itself is not centred. */
static double vector_std(const double *x, int d, int ddof)
{
    double mu = 0.0;
    for (int c = 0; c < d; ++c) mu += x[c];
    mu /= d;
    double ss = 0.0;
    for (int c = 0; c < d; ++c) ss += (x[c] - mu) * (x[c] - mu);
    return sqrt(ss / (d - ddof));
}

static int degenerate(double s) { return !(s > 0.0) || !isfinite(s); }

/* Algorithm 1, argmin step: squared Euclidean distance to every code of one
 * codebook, direct form, lowest index on ties.  Also returns the runner-up. */
static int nearest(const double *z, const double *cb, int K, int gd, double *d1, double *d2)
{
    int best = 0;
    double b1 = INFINITY, b2 = INFINITY;
    for (int j = 0; j < K; ++j) {
        double acc = 0.0;
        const double *e = cb + (size_t)j * gd;
        for (int i = 0; i < gd; ++i) { double t = z[i] - e[i]; acc += t * t; }
        if (acc < b1) { b2 = b1; b1 = acc; best = j; }
        else if (acc < b2) b2 = acc;
    }
    *d1 = b1; *d2 = b2;
    return best;
}

/*
 * Encode n head vectors.  x[n][dim], cb[R][K][gd] (doubles holding the exact
 * input values).  Outputs: codes[n][G][R]; std16[n] (fp16 bits);
 * std_exact[n]; d1,d2[n][G][R] best and second-best squared distance at every
 * stage (NULL to skip); resid[n][G][gd] the residual left after R stages
 * (NULL to skip).  Returns the number of degenerate vectors.
 */
int64_t rvq_oracle_encode(const double *x, int64_t n, int dim, int gd, int layout, int R, int K,
                          const double *cb, int ddof, int32_t *codes, uint16_t *std16,
                          double *std_exact, double *d1, double *d2, double *resid)
{
    int G = dim / gd;
    int64_t bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (int64_t v = 0; v < n; ++v) {
        const double *xv = x + v * dim;
        double s = vector_std(xv, dim, ddof);
        int deg = degenerate(s);
        if (deg) ++bad;
        if (std_exact) std_exact[v] = s;
        std16[v] = deg ? 0 : rvq_oracle_f64_to_f16_bits(s);
        double z[1024];
        for (int g = 0; g < G; ++g) {
            for (int i = 0; i < gd; ++i) z[i] = deg ? 0.0 : xv[chan_of(layout, G, gd, g, i)] / s;
            for (int r = 0; r < R; ++r) {                       /* Algorithm 1 loop */
                const double *cbr = cb + (size_t)r * K * gd;
                double a, b;
                int j = deg ? 0 : nearest(z, cbr, K, gd, &a, &b);
                if (deg) { a = 0.0; b = INFINITY; }
                size_t pos = ((size_t)v * G + g) * R + r;
                codes[pos] = j;
                if (d1) d1[pos] = a;
                if (d2) d2[pos] = b;
                for (int i = 0; i < gd; ++i) z[i] -= cbr[(size_t)j * gd + i];
            }
            if (resid) memcpy(resid + ((size_t)v * G + g) * gd, z, sizeof(double) * gd);
        }
    }
    return bad;
}

/* Section 2.2, last sentence: output = (sum of the chosen codes) * std, with
 * the std as stored (fp16).  xhat[n][dim] is left unrounded. */
void rvq_oracle_decode(const int32_t *codes, const uint16_t *std16, int64_t n, int dim, int gd,
                       int layout, int R, int K, const double *cb, double *xhat)
{
    int G = dim / gd;
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n; ++v) {
        double s = rvq_oracle_f16_bits_to_f64(std16[v]);
        for (int g = 0; g < G; ++g)
            for (int i = 0; i < gd; ++i) {
                double acc = 0.0;
                for (int r = 0; r < R; ++r) {
                    int j = codes[((size_t)v * G + g) * R + r];
                    acc += cb[((size_t)r * K + j) * gd + i];
                }
                xhat[v * dim + chan_of(layout, G, gd, g, i)] = s * acc;
            }
    }
}

/*
 * EMA statistics of one step: for every stage r and code j, cnt[r][j] = number
 * of group rows whose stage-r code is j and sum[r][j][:] = sum of their
 * stage-r inputs z_r (scaled space, rebuilt from x and the codes with the
 * codebooks the codes were chosen from).
 */
void rvq_oracle_ema_stats(const double *x, int64_t n, int dim, int gd, int layout, int R, int K,
                          const double *cb, int ddof, const int32_t *codes, double *cnt, double *sum)
{
    int G = dim / gd;
    memset(cnt, 0, sizeof(double) * (size_t)R * K);
    memset(sum, 0, sizeof(double) * (size_t)R * K * gd);
    for (int64_t v = 0; v < n; ++v) {
        const double *xv = x + v * dim;
        double s = vector_std(xv, dim, ddof);
        int deg = degenerate(s);
        double z[1024];
        for (int g = 0; g < G; ++g) {
            for (int i = 0; i < gd; ++i) z[i] = deg ? 0.0 : xv[chan_of(layout, G, gd, g, i)] / s;
            for (int r = 0; r < R; ++r) {
                int j = codes[((size_t)v * G + g) * R + r];
                cnt[(size_t)r * K + j] += 1.0;
                double *m = sum + ((size_t)r * K + j) * gd;
                const double *e = cb + ((size_t)r * K + j) * gd;
                for (int i = 0; i < gd; ++i) { m[i] += z[i]; z[i] -= e[i]; }
            }
        }
    }
}

/*
 * EMA update with Laplace smoothing (VQ-VAE appendix form):
 *   N <- g N + (1-g) n ;  M <- g M + (1-g) m ;
 *   N^_j = (N_j + eps) * sum_j N / (sum_j N + K eps) ;  C_j = M_j / N^_j.
 * All arrays are updated in place.
 */
void rvq_oracle_ema_normalise(const double *cnt, const double *sum, int R, int K, int gd,
                              double decay, double eps, double *ema_count, double *ema_sum,
                              double *cb)
{
    for (int r = 0; r < R; ++r) {
        double tot = 0.0;
        for (int j = 0; j < K; ++j) {
            size_t p = (size_t)r * K + j;
            ema_count[p] = decay * ema_count[p] + (1.0 - decay) * cnt[p];
            tot += ema_count[p];
            for (int i = 0; i < gd; ++i)
                ema_sum[p * gd + i] = decay * ema_sum[p * gd + i] + (1.0 - decay) * sum[p * gd + i];
        }
        for (int j = 0; j < K; ++j) {
            size_t p = (size_t)r * K + j;
            double nh = (ema_count[p] + eps) * tot / (tot + K * eps);
            for (int i = 0; i < gd; ++i) cb[p * gd + i] = ema_sum[p * gd + i] / nh;
        }
    }
}

/*
 * Code storage (Section 3.2's compression arithmetic: R*G indices of
 * ceil(log2 K) bits per head vector).  Bit stream per head vector, code
 * number g*R+r at bit offset bits*(g*R+r), least significant bit first,
 * padded to a multiple of 4 bytes.  Returns bytes per head vector.
 */
int64_t rvq_oracle_packed_bytes(int per_vector, int bits)
{
    return ((int64_t)per_vector * bits + 31) / 32 * 4;
}

void rvq_oracle_pack(const int32_t *codes, int64_t n, int per_vector, int bits, uint8_t *out)
{
    int64_t nb = rvq_oracle_packed_bytes(per_vector, bits);
    memset(out, 0, (size_t)(n * nb));
    for (int64_t v = 0; v < n; ++v)
        for (int k = 0; k < per_vector; ++k)
            for (int b = 0; b < bits; ++b)
                if ((codes[v * per_vector + k] >> b) & 1) {
                    int64_t bit = (int64_t)k * bits + b;
                    out[v * nb + bit / 8] |= (uint8_t)(1u << (bit % 8));
                }
}

void rvq_oracle_unpack(const uint8_t *in, int64_t n, int per_vector, int bits, int32_t *codes)
{
    int64_t nb = rvq_oracle_packed_bytes(per_vector, bits);
    for (int64_t v = 0; v < n; ++v)
        for (int k = 0; k < per_vector; ++k) {
            int32_t c = 0;
            for (int b = 0; b < bits; ++b) {
                int64_t bit = (int64_t)k * bits + b;
                if ((in[v * nb + bit / 8] >> (bit % 8)) & 1) c |= 1 << b;
            }
            codes[v * per_vector + k] = c;
        }
}

/*
 * Judge a given code sequence stage by stage, conditioned on its own prefix:
 * the residual entering stage r is rebuilt from the GIVEN codes of stages < r,
 * and the given stage-r code is compared with the exact argmin for that
 * residual.  status[n][G][R]: 0 = it is the argmin (lowest index on ties);
 * 1 = not the argmin but (D_given - D_min) < tol * D_given (a near tie);
 * 2 = a real mismatch; 3 = code out of range.  gap (optional) receives
 * (D_given - D_min) / D_given.
 */
int64_t rvq_oracle_check_codes(const double *x, int64_t n, int dim, int gd, int layout, int R,
                               int K, const double *cb, int ddof, const int32_t *codes,
                               double tol, uint8_t *status, double *gap)
{
    int G = dim / gd;
    int64_t wrong = 0;
#pragma omp parallel for schedule(static) reduction(+ : wrong)
    for (int64_t v = 0; v < n; ++v) {
        const double *xv = x + v * dim;
        double s = vector_std(xv, dim, ddof);
        int deg = degenerate(s);
        double z[1024];
        for (int g = 0; g < G; ++g) {
            for (int i = 0; i < gd; ++i) z[i] = deg ? 0.0 : xv[chan_of(layout, G, gd, g, i)] / s;
            for (int r = 0; r < R; ++r) {
                const double *cbr = cb + (size_t)r * K * gd;
                size_t pos = ((size_t)v * G + g) * R + r;
                int jg = codes[pos];
                if (jg < 0 || jg >= K) { status[pos] = 3; ++wrong; if (gap) gap[pos] = INFINITY; jg = 0; continue; }
                double a, b;
                int j = deg ? 0 : nearest(z, cbr, K, gd, &a, &b);
                double dg = 0.0;
                for (int i = 0; i < gd; ++i) { double t = z[i] - cbr[(size_t)jg * gd + i]; dg += t * t; }
                if (deg) a = dg;
                double rel = dg > 0.0 ? (dg - a) / dg : 0.0;
                if (gap) gap[pos] = rel;
                if (jg == j) status[pos] = 0;
                else if (rel < tol) status[pos] = 1;
                else { status[pos] = 2; ++wrong; }
                for (int i = 0; i < gd; ++i) z[i] -= cbr[(size_t)jg * gd + i];
            }
        }
    }
    return wrong;
}

int rvq_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
