/*
 * speca_oracle.c -- plain CPU statement of the SpeCa feature-cache arithmetic (arXiv 2509.11628).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the yardstick the CUDA library is compared with. It is
 * deliberately slow and literal: double arithmetic on values read back from storage, one loop per
 * equation, no blocking, no fusion. It shares no code, header, table or helper with the CUDA
 * path, and nothing in the product may call it.
 *
 * What each function follows
 *   oracle_update_segment    Eq. 3 (finite differences of the cached feature), kept as difference
 *                            quotients so that reference steps may be unevenly spaced
 *   oracle_forecast_segment  Eq. 2 (TaylorSeer prediction), written as the printed sum
 *   oracle_forecast_history_segment  Eq. 2-3 evaluated from the stored raw features of the last
 *                            references (no rounded intermediate planes)
 *   oracle_rel_l2            Eq. 4 (relative error, epsilon = 1e-8)
 *   oracle_rel_l1/_linf, oracle_cos_dist   the other metrics of the appendix on error metrics
 *                            (named there without formulas: readings, parity unpinned by the paper)
 *   oracle_accept            Section 3.4.2, rule 1/2 (e <= tau accepts)
 *   oracle_tau               Section 3.4.2, tau_t = tau0 * beta^((T-t)/T)
 *   oracle_speedup           Eq. 8, S = 1 / (1 - alpha + alpha*gamma)
 *
 * Pins (tests/test_oracle_pins.py): exact-rational evaluation of Eq. 2-3 from the raw feature
 * history; order 0 == reuse; exactness on polynomials (degree <= 1 Taylor basis, degree <= m
 * Newton basis); closed-form quadratic residual; Eq. 4 special cases and brute force; the
 * paper's worked speed-up number. Unpinned: nothing the paper prints numbers for exists beyond
 * the speed-up example; uneven gaps in the Taylor basis are pinned only through the
 * degree <= 1 exactness and the recursion's definition ("parity unpinned" for that case
 * beyond those two properties).
 *
 * Storage types: 0 = IEEE binary32, 1 = bfloat16 (upper 16 bits of binary32, round to nearest
 * even on store, NaN kept NaN).
 *
 * Precision. Each formula is evaluated in double. The method's stated precision is "fp32
 * accumulation, bf16 storage": the value that is quantised to the storage type is a binary32
 * register. A stored result is therefore rounded double -> binary32 -> storage type, both to
 * nearest even, so that the quantisation decision is taken in the kernel's precision. (Cached
 * features have 8-bit significands and reciprocal gaps like 50 have few bits, so exact bfloat16
 * ties are common in the difference quotients; rounding the double directly would break them by
 * the 1e-16 representation error of the gap instead of by the ties-to-even rule.)
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define ORACLE_MAX_ORDER 8

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_TAYLOR = 0, ORACLE_NEWTON = 1, ORACLE_ADAMS_BASHFORTH = 2 };

/* ---- storage <-> double ------------------------------------------------------------------ */

static double bf16_bits_to_double(uint16_t h) {
    uint32_t w = (uint32_t)h << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Round a double to the nearest bfloat16 (ties to even) and return its bits. bfloat16 has 8
 * significant bits and binary32's exponent range, so: scale the value so that one unit in the
 * last place becomes 1.0, round to an integer with the default rounding mode, scale back. */
uint16_t oracle_double_to_bf16_bits(double v) {
    if (isnan(v)) return 0x7FC0u;
    if (isinf(v)) return v > 0 ? 0x7F80u : 0xFF80u;
    if (v == 0.0) return signbit(v) ? 0x8000u : 0x0000u;
    int e;
    (void)frexp(v, &e); /* |v| = f * 2^e with f in [0.5, 1) -> leading bit has weight 2^(e-1) */
    int lead = e - 1;
    if (lead < -126) lead = -126; /* subnormal range: fixed quantum 2^-133 */
    double q = nearbyint(ldexp(v, 7 - lead)); /* 7 fraction bits below the leading bit */
    double r = ldexp(q, lead - 7);
    if (fabs(r) >= ldexp(1.0, 128)) return r > 0 ? 0x7F80u : 0xFF80u;
    float f = (float)r; /* exact: r has at most 8 significant bits */
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    return (uint16_t)(w >> 16);
}

static double load_elem(const void* p, int dtype, int64_t i) {
    if (dtype == ORACLE_F32) return (double)((const float*)p)[i];
    return bf16_bits_to_double(((const uint16_t*)p)[i]);
}

static void store_elem(void* p, int dtype, int64_t i, double v) {
    float r = (float)v; /* the binary32 register that holds the result */
    if (dtype == ORACLE_F32)
        ((float*)p)[i] = r;
    else
        ((uint16_t*)p)[i] = oracle_double_to_bf16_bits((double)r);
}

/* ---- Eq. 3: table rewrite at a reference step ---------------------------------------------- */
/*
 * One (entry, sample) table of `n` elements, planes[i] at planes + i*plane_stride elements.
 * n_refs  = references folded in so far (0 = empty table).
 * t_hist  = their times, most recent first (t_hist[0] = t_last); min(n_refs, m) are read.
 * The i-th finite difference of Eq. 3 over reference times t, t+N, ..., t+iN obeys
 * Delta^i F(t) = Delta^(i-1) F(t) - Delta^(i-1) F(t+N); the table keeps Delta^i / N^i, so the
 * new quotient of order i+1 is (new order-i quotient - old order-i quotient) / (t_new - t_last).
 * Newton basis: the divisor is t_new - t_hist[i] instead (divided differences).
 * The chain runs on unrounded values; each plane is rounded once when stored.
 * Returns 0, or 1 if a divisor is zero (nothing is written then).
 */
int oracle_update_segment(int dtype, int64_t n, int m, int basis, int n_refs, const double* t_hist,
                          double t_new, const void* feat, void* planes, int64_t plane_stride) {
    int v_new = n_refs < m ? n_refs : m; /* highest order defined after this update */
    double gap[ORACLE_MAX_ORDER];
    for (int i = 0; i < v_new; ++i) {
        gap[i] = t_new - (basis == ORACLE_NEWTON ? t_hist[i] : t_hist[0]);
        if (gap[i] == 0.0) return 1;
    }
    size_t esz = dtype == ORACLE_F32 ? 4 : 2;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        double c[ORACLE_MAX_ORDER + 1];
        c[0] = load_elem(feat, dtype, j);
        for (int i = 0; i < v_new; ++i) {
            double old_i = load_elem((const char*)planes + (size_t)i * plane_stride * esz, dtype, j);
            c[i + 1] = (c[i] - old_i) / gap[i];
        }
        for (int i = 0; i <= v_new; ++i)
            store_elem((char*)planes + (size_t)i * plane_stride * esz, dtype, j, c[i]);
    }
    return 0;
}

/* ---- Eq. 2: forecast ------------------------------------------------------------------------ */
/*
 * v = min(m, n_refs - 1) orders are defined. With x = t_target - t_last (= -k on the paper's
 * integer grid):
 *   Taylor basis:  out = plane_0 + sum_{i=1..v} plane_i * x^i / i!
 *   Newton basis:  out = plane_0 + sum_{i=1..v} plane_i * prod_{j<i} (t_target - t_hist[j])
 * Returns 0, or 1 if the table is empty (n_refs < 1).
 */
int oracle_forecast_segment(int dtype, int64_t n, int m, int basis, int n_refs, const double* t_hist,
                            double t_target, const void* planes, int64_t plane_stride, void* out) {
    if (n_refs < 1) return 1;
    int v = n_refs - 1 < m ? n_refs - 1 : m;
    size_t esz0 = dtype == ORACLE_F32 ? 4 : 2;
    if (basis == ORACLE_ADAMS_BASHFORTH && v >= 1) {
        /*
         * Adams-Bashforth draft model (appendix, ablation of draft models; named there without a
         * formula -- this reading is "parity unpinned" by the paper). The table is kept as in the
         * Taylor basis. With h = t_last - (previous reference time), plane 1 is the latest slope
         * g_0 = (F_0 - F_1)/h and the slope j references back follows from the higher planes by
         * backward differencing, g_j = sum_i C(j,i) (-h)^i plane_{1+i}. The v-step Adams-Bashforth
         * formula with its textbook coefficients b extrapolates over x = t_target - t_last:
         *     out = F_0 + x * sum_{j<v} b_j g_j   (b = row v-1 of the table below).
         */
        static const double b[4][4] = {{1.0, 0, 0, 0},
                                       {3.0 / 2, -1.0 / 2, 0, 0},
                                       {23.0 / 12, -16.0 / 12, 5.0 / 12, 0},
                                       {55.0 / 24, -59.0 / 24, 37.0 / 24, -9.0 / 24}};
        if (v > 4) return 1;
        double x = t_target - t_hist[0];
        double h = v >= 2 ? t_hist[0] - t_hist[1] : 0.0;
#pragma omp parallel for schedule(static)
        for (int64_t j = 0; j < n; ++j) {
            double d[ORACLE_MAX_ORDER + 1];
            for (int i = 0; i <= v; ++i) d[i] = load_elem((const char*)planes + (size_t)i * plane_stride * esz0, dtype, j);
            double sum = 0.0;
            for (int s = 0; s < v; ++s) { /* slope s references back */
                double g = 0.0, binom = 1.0, hp = 1.0;
                for (int i = 0; i <= s; ++i) {
                    g += binom * hp * d[1 + i];
                    binom = binom * (double)(s - i) / (double)(i + 1);
                    hp *= -h;
                }
                sum += b[v - 1][s] * g;
            }
            store_elem(out, dtype, j, d[0] + x * sum);
        }
        return 0;
    }
    double w[ORACLE_MAX_ORDER + 1]; /* weight of plane i */
    w[0] = 1.0;
    if (basis == ORACLE_NEWTON) {
        for (int i = 1; i <= v; ++i) w[i] = w[i - 1] * (t_target - t_hist[i - 1]);
    } else {
        double x = t_target - t_hist[0];
        double fact = 1.0;
        for (int i = 1; i <= v; ++i) {
            fact *= (double)i;
            w[i] = pow(x, (double)i) / fact;
        }
    }
    size_t esz = dtype == ORACLE_F32 ? 4 : 2;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        double s = load_elem(planes, dtype, j);
        for (int i = 1; i <= v; ++i)
            s += load_elem((const char*)planes + (size_t)i * plane_stride * esz, dtype, j) * w[i];
        store_elem(out, dtype, j, s);
    }
    return 0;
}

/* ---- Eq. 2-3 straight from the raw feature history ------------------------------------------------ */
/*
 * The same forecast when the cache keeps the last references' FEATURES instead of their difference
 * quotients: hist[0] is the feature at t_hist[0] (the latest reference), hist[1] the one before, ...;
 * n_hist = min(m + 1, references seen) of them exist. Eq. 3's differences are formed here, in double,
 * by folding the features in one by one from the oldest to the newest exactly as
 * oracle_update_segment would have (same divisors), but without rounding any intermediate plane to
 * the storage type; Eq. 2 (or the Newton / Adams-Bashforth reading) is then applied as in
 * oracle_forecast_segment and the result is rounded once. On a uniform grid this is Eq. 2-3 as
 * printed, evaluated from the raw features.
 * Returns 0, or 1 if there is no reference or a divisor is zero.
 */
static int history_times_ok(int m, int basis, int n_hist, const double* t_hist) {
    if (n_hist < 1 || n_hist > m + 1 || m > ORACLE_MAX_ORDER) return 0;
    int v = n_hist - 1;
    if (basis == ORACLE_ADAMS_BASHFORTH && v > 4) return 0;
    for (int k = v - 1; k >= 0; --k)
        for (int i = 0; i < v - k; ++i)
            if (t_hist[k] - (basis == ORACLE_NEWTON ? t_hist[k + 1 + i] : t_hist[k + 1]) == 0.0) return 0;
    return 1;
}

/* The unrounded forecast of element j from the v + 1 stored features. */
static double history_forecast_elem(int dtype, int basis, int v, const double* t_hist, double t_target,
                                    const void* const* hist, int64_t j) {
    static const double gam[4] = {1.0, 1.0 / 2, 5.0 / 12, 3.0 / 8}; /* Adams-Bashforth, collected by plane */
    double d[ORACLE_MAX_ORDER + 1]; /* the planes a table would hold, unrounded */
    d[0] = load_elem(hist[v], dtype, j);
    for (int k = v - 1; k >= 0; --k) { /* fold in the feature at t_hist[k]; v - k references came before */
        double c[ORACLE_MAX_ORDER + 1];
        c[0] = load_elem(hist[k], dtype, j);
        for (int i = 0; i < v - k; ++i) {
            double gap = t_hist[k] - (basis == ORACLE_NEWTON ? t_hist[k + 1 + i] : t_hist[k + 1]);
            c[i + 1] = (c[i] - d[i]) / gap;
        }
        for (int i = 0; i <= v - k; ++i) d[i] = c[i];
    }
    double s = d[0];
    if (basis == ORACLE_NEWTON) {
        double w = 1.0;
        for (int i = 1; i <= v; ++i) {
            w *= t_target - t_hist[i - 1];
            s += d[i] * w;
        }
    } else if (basis == ORACLE_TAYLOR) {
        double x = t_target - t_hist[0], fact = 1.0;
        for (int i = 1; i <= v; ++i) {
            fact *= (double)i;
            s += d[i] * pow(x, (double)i) / fact;
        }
    } else {
        double x = t_target - t_hist[0], h = v >= 2 ? t_hist[0] - t_hist[1] : 0.0, hp = 1.0;
        for (int i = 1; i <= v; ++i) {
            s += d[i] * x * gam[i - 1] * hp;
            hp *= h;
        }
    }
    return s;
}

int oracle_forecast_history_segment(int dtype, int64_t n, int m, int basis, int n_hist, const double* t_hist,
                                    double t_target, const void* const* hist, void* out) {
    if (!history_times_ok(m, basis, n_hist, t_hist)) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j)
        store_elem(out, dtype, j, history_forecast_elem(dtype, basis, n_hist - 1, t_hist, t_target, hist, j));
    return 0;
}

/* The same forecast added, unrounded, to an accumulator (for the summed forecast below). */
int oracle_forecast_history_accumulate_segment(int dtype, int64_t n, int m, int basis, int n_hist, const double* t_hist,
                                               double t_target, const void* const* hist, double* acc) {
    if (!history_times_ok(m, basis, n_hist, t_hist)) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j) acc[j] += history_forecast_elem(dtype, basis, n_hist - 1, t_hist, t_target, hist, j);
    return 0;
}

/* ---- Eq. 2 summed over several entries ---------------------------------------------------------- */
/*
 * A transformer adds its block outputs to a residual stream, so on a speculative step the forecasts
 * of blocks with equal shapes are only ever consumed as a sum: out = base + sum_e forecast_e. The two
 * functions below state that in the plainest form: each entry's forecast (Eq. 2, any basis) is added
 * UNROUNDED, in double, to an accumulator; the total is rounded once (double -> binary32 -> storage).
 * oracle_forecast_accumulate_segment returns 0, or 1 if the table is empty / the basis unknown.
 */
int oracle_forecast_accumulate_segment(int dtype, int64_t n, int m, int basis, int n_refs, const double* t_hist,
                                       double t_target, const void* planes, int64_t plane_stride, double* acc) {
    if (n_refs < 1) return 1;
    int v = n_refs - 1 < m ? n_refs - 1 : m;
    size_t esz = dtype == ORACLE_F32 ? 4 : 2;
    double w[ORACLE_MAX_ORDER + 1];
    w[0] = 1.0;
    if (basis == ORACLE_NEWTON) {
        for (int i = 1; i <= v; ++i) w[i] = w[i - 1] * (t_target - t_hist[i - 1]);
    } else if (basis == ORACLE_TAYLOR) {
        double x = t_target - t_hist[0], fact = 1.0;
        for (int i = 1; i <= v; ++i) {
            fact *= (double)i;
            w[i] = pow(x, (double)i) / fact;
        }
    } else if (basis == ORACLE_ADAMS_BASHFORTH) {
        /* collected by plane: F + x (D1 + h/2 D2 + 5h^2/12 D3 + 3h^3/8 D4) -- the same polynomial the
         * slope form in oracle_forecast_segment evaluates (tests check the two against each other) */
        static const double gam[4] = {1.0, 1.0 / 2, 5.0 / 12, 3.0 / 8};
        double x = t_target - t_hist[0], h = v >= 2 ? t_hist[0] - t_hist[1] : 0.0, hp = 1.0;
        if (v > 4) return 1;
        for (int i = 1; i <= v; ++i) {
            w[i] = x * gam[i - 1] * hp;
            hp *= h;
        }
    } else {
        return 1;
    }
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        double s = load_elem(planes, dtype, j);
        for (int i = 1; i <= v; ++i)
            s += load_elem((const char*)planes + (size_t)i * plane_stride * esz, dtype, j) * w[i];
        acc[j] += s;
    }
    return 0;
}

void oracle_accumulate_elems(int dtype, int64_t n, const void* src, double* acc) {
    for (int64_t j = 0; j < n; ++j) acc[j] += load_elem(src, dtype, j);
}

void oracle_round_store(int dtype, int64_t n, const double* acc, void* out) {
    for (int64_t j = 0; j < n; ++j) store_elem(out, dtype, j, acc[j]);
}

/* ---- Eq. 4: relative error ------------------------------------------------------------------- */
/* e = ||pred - fresh||_2 / (||fresh||_2 + eps), Euclidean norms over the n elements of a sample. */
double oracle_rel_l2(int dtype, int64_t n, const void* pred, const void* fresh, double eps) {
    double num = 0.0, den = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : num, den)
    for (int64_t j = 0; j < n; ++j) {
        double p = load_elem(pred, dtype, j);
        double f = load_elem(fresh, dtype, j);
        num += (p - f) * (p - f);
        den += f * f;
    }
    return sqrt(num) / (sqrt(den) + eps);
}

/* ---- other error metrics (appendix "Choice of Error Metrics for Verification") ----------------- */
/*
 * The appendix names l1, l-infinity and cosine similarity as alternatives to the l2 norm of Eq. 4
 * and says a relative formulation is used, but prints no formulas: these are readings, pinned in
 * the tests by what the mathematics fixes (zero at p = f, |delta| at p = (1+delta) f, scale
 * invariance, brute force in rationals, the angle between two plane vectors), "parity unpinned" by
 * the paper itself.
 *   l1:     sum |p - f| / (sum |f| + eps)
 *   l-inf:  max |p - f| / (max |f| + eps)
 *   cosine: 1 - <p, f> / (||p||_2 ||f||_2 + eps), a distance so that "accept iff value <= tau" holds
 * A NaN element makes every one of them NaN (rejected).
 */
double oracle_rel_l1(int dtype, int64_t n, const void* pred, const void* fresh, double eps) {
    double num = 0.0, den = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : num, den)
    for (int64_t j = 0; j < n; ++j) {
        double p = load_elem(pred, dtype, j);
        double f = load_elem(fresh, dtype, j);
        num += fabs(p - f);
        den += fabs(f);
    }
    return num / (den + eps);
}

double oracle_rel_linf(int dtype, int64_t n, const void* pred, const void* fresh, double eps) {
    double num = 0.0, den = 0.0;
    int bad = 0;
    for (int64_t j = 0; j < n; ++j) {
        double p = load_elem(pred, dtype, j);
        double f = load_elem(fresh, dtype, j);
        double d = fabs(p - f), a = fabs(f);
        if (isnan(d) || isnan(a)) bad = 1;
        if (d > num) num = d;
        if (a > den) den = a;
    }
    if (bad) return NAN;
    return num / (den + eps);
}

double oracle_cos_dist(int dtype, int64_t n, const void* pred, const void* fresh, double eps) {
    double dot = 0.0, pp = 0.0, ff = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : dot, pp, ff)
    for (int64_t j = 0; j < n; ++j) {
        double p = load_elem(pred, dtype, j);
        double f = load_elem(fresh, dtype, j);
        dot += p * f;
        pp += p * p;
        ff += f * f;
    }
    return 1.0 - dot / (sqrt(pp) * sqrt(ff) + eps);
}

/*
 * The same metrics split in two stages, for a verification entry whose tokens are spread over
 * several caches: the running values of one part (sums, or maxima for l-infinity), and the error
 * from combined values. metric: 0 = l2 (Eq. 4), 1 = l1, 2 = l-infinity, 3 = cosine distance.
 */
void oracle_metric_sums(int metric, int dtype, int64_t n, const void* pred, const void* fresh, double* out3) {
    double a0 = 0.0, a1 = 0.0, a2 = 0.0;
    int bad = 0;
    for (int64_t j = 0; j < n; ++j) {
        double p = load_elem(pred, dtype, j);
        double f = load_elem(fresh, dtype, j);
        if (metric == 0) {
            a0 += (p - f) * (p - f);
            a1 += f * f;
        } else if (metric == 1) {
            a0 += fabs(p - f);
            a1 += fabs(f);
        } else if (metric == 2) {
            double d = fabs(p - f), a = fabs(f);
            if (isnan(d) || isnan(a)) bad = 1;
            if (d > a0) a0 = d;
            if (a > a1) a1 = a;
        } else {
            a0 += p * f;
            a1 += p * p;
            a2 += f * f;
        }
    }
    if (bad) a0 = a1 = NAN;
    out3[0] = a0;
    out3[1] = a1;
    out3[2] = a2;
}

double oracle_metric_from_sums(int metric, const double* s, double eps) {
    if (metric == 0) return sqrt(s[0]) / (sqrt(s[1]) + eps);
    if (metric == 3) return 1.0 - s[0] / (sqrt(s[1]) * sqrt(s[2]) + eps);
    return s[0] / (s[1] + eps);
}

/* Section 3.4.2: accepted iff e <= tau. A NaN error compares false and is rejected. */
int oracle_accept(double err, double tau) { return err <= tau ? 1 : 0; }

/* Section 3.4.2: tau_t = tau0 * beta^((T - t)/T). */
double oracle_tau(double tau0, double beta, double t, double T) { return tau0 * pow(beta, (T - t) / T); }

/* Eq. 8: speed-up for acceptance rate alpha and verification cost ratio gamma. */
double oracle_speedup(double alpha, double gamma) { return 1.0 / (1.0 - alpha + alpha * gamma); }

/* Number of threads the loops above use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int oracle_threads(void) { return omp_get_max_threads(); }
void oracle_set_threads(int n) { omp_set_num_threads(n); }
#else
int oracle_threads(void) { return 1; }
void oracle_set_threads(int n) { (void)n; }
#endif
