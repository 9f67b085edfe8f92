/*
 * CPU oracle for layerwise Query-Key RMSNorm.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the yardstick the CUDA library is measured against.  It is
 * plain C, fp64 throughout, and shares nothing with the CUDA sources: no
 * header, no helper, no table.  Nothing in the product path may call it; only
 * the test-suite, the smoke check and the benchmark's CPU-baseline legs do.
 *
 * What it computes is the definition itself (Eq. 1 of the paper), written out:
 *
 *     y[t][j] = x[t][j] / sqrt( (1/H) * sum_j x[t][j]^2 + eps ) * gamma[j]
 *
 * once for the Q tensor (H = dq, gamma = gamma_q) and once for the K tensor
 * (H = dk, gamma = gamma_k): the callers run it per tensor.  The paper's method
 * (Algorithm 1) reaches exactly this value by a cheaper route (per-shard sums
 * of squares combined as scalars; Section III-A says the semantics are
 * unchanged, and Section IV-C takes "gather everything, then fp64 RMSNorm" as
 * its gold).  So the sharded form below is: put the column slices side by
 * side (slice s = columns [s*w, (s+1)*w), rank order), apply the definition
 * with H = the FULL width (H_total of Algorithm 1), and cut the result back
 * into slices.  It also reports each slice's own sum of squares (Phase A of
 * Algorithm 1) so that tests can check the partials add up to the row total.
 *
 * Storage is bf16 (upper half of an IEEE binary32).  bf16 -> fp64 is exact;
 * fp64 -> bf16 rounds to nearest, ties to even, in ONE step (going through
 * fp32 could round twice).  eps arrives as a float and is widened, so the
 * oracle sees the same eps the GPU kernel does.
 *
 * Every function here is pinned by tests/test_oracle_*.py against closed
 * forms, invariants, hand-computed rows and torch's fp64 rms_norm; no function
 * is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- bf16 <-> fp64 --------------------------------------------------------- */

double qko_bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f; /* exact: every bf16 is a binary32, every binary32 a binary64 */
}

/* Round a double to the nearest bf16 (ties to even), directly.
 * bf16 has 8 significant bits; a normal value in [2^e, 2^(e+1)) is a multiple
 * of 2^(e-7), a subnormal one a multiple of 2^-133.  Divide by that unit (exact,
 * a power of two), round to an integer in the default rounding mode (nearest
 * even), multiply back (exact).  The result is a bf16 value, or 2^128 which
 * becomes infinity when narrowed. */
uint16_t qko_f64_to_bf16(double v) {
    if (isnan(v)) return (uint16_t)(signbit(v) ? 0xFFC0u : 0x7FC0u);
    if (isinf(v)) return (uint16_t)(signbit(v) ? 0xFF80u : 0x7F80u);
    if (v == 0.0) return (uint16_t)(signbit(v) ? 0x8000u : 0x0000u);
    int ex;
    (void)frexp(v, &ex);          /* |v| = m * 2^ex, 0.5 <= m < 1  ->  floor(log2|v|) = ex-1 */
    int e = ex - 1;
    if (e < -126) e = -126;       /* subnormal range shares the smallest normal's unit */
    double unit = ldexp(1.0, e - 7);
    double r = nearbyint(v / unit) * unit;
    float f = (float)r;           /* exact unless |r| = 2^128 -> inf */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(u >> 16);
}

/* ---- one row, one tensor: Eq. 1 -------------------------------------------- */

/* x, gamma: H bf16 values.  y: H bf16 values (may be NULL).  y64: the same
 * result before rounding (may be NULL).  Returns the row's sum of squares in
 * *acc_out and 1/sqrt(mean square + eps) in *rstd_out (either may be NULL). */
static void rmsnorm_row(const uint16_t* x, const uint16_t* gamma, int64_t H, double eps,
                        uint16_t* y, double* y64, double* acc_out, double* rstd_out) {
    double acc = 0.0;
    for (int64_t j = 0; j < H; ++j) {
        double v = qko_bf16_to_f64(x[j]);
        acc += v * v;
    }
    double r = 1.0 / sqrt(acc / (double)H + eps);
    for (int64_t j = 0; j < H; ++j) {
        double o = qko_bf16_to_f64(x[j]) * r * qko_bf16_to_f64(gamma[j]);
        if (y64) y64[j] = o;
        if (y) y[j] = qko_f64_to_bf16(o);
    }
    if (acc_out) *acc_out = acc;
    if (rstd_out) *rstd_out = r;
}

/* ---- unsharded: x[T][H] row-major ------------------------------------------ */

/* Returns 0, or -1 on a bad argument.  y / y64 / acc / rstd may each be NULL.
 * y may be the same buffer as x (each row is read completely before it is
 * written).  nthreads <= 1 runs the plain loop; more only spreads whole rows
 * over OpenMP threads (for the timed baseline). */
int qko_rmsnorm(const uint16_t* x, const uint16_t* gamma, int64_t T, int64_t H, float eps,
                uint16_t* y, double* y64, double* acc, double* rstd, int nthreads) {
    if (T < 0 || H < 0) return -1;
    if (T == 0 || H == 0) return 0;
    if (!x || !gamma) return -1;
    const double e = (double)eps;
#ifdef _OPENMP
    if (nthreads > 1) {
        int failed = 0;
#pragma omp parallel for num_threads(nthreads) schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            uint16_t* row = (uint16_t*)malloc((size_t)H * sizeof(uint16_t));
            if (!row) {
                failed = 1;   /* benign race: every writer stores 1 */
                continue;
            }
            memcpy(row, x + t * H, (size_t)H * sizeof(uint16_t));
            rmsnorm_row(row, gamma, H, e, y ? y + t * H : NULL, y64 ? y64 + t * H : NULL,
                        acc ? acc + t : NULL, rstd ? rstd + t : NULL);
            free(row);
        }
        return failed ? -1 : 0;
    }
#else
    (void)nthreads;
#endif
    uint16_t* row = (uint16_t*)malloc((size_t)H * sizeof(uint16_t));
    if (!row) return -1;
    for (int64_t t = 0; t < T; ++t) {
        memcpy(row, x + t * H, (size_t)H * sizeof(uint16_t)); /* so that y == x is safe */
        rmsnorm_row(row, gamma, H, e, y ? y + t * H : NULL, y64 ? y64 + t * H : NULL,
                    acc ? acc + t : NULL, rstd ? rstd + t : NULL);
    }
    free(row);
    return 0;
}

/* ---- sharded: S buffers x_s[T][w], w = H/S --------------------------------- */

/* x_shards, gamma_shards, y_shards: arrays of S pointers.  H is the FULL width.
 * partials (may be NULL): [S][T], slice s's own sum of squares for token t.
 * acc, rstd (may be NULL): [T], taken from the gathered row, NOT from the
 * partials, so that "partials add up to acc" is a real check.
 * y_shards[s] may equal x_shards[s]. */
int qko_rmsnorm_sharded(const uint16_t* const* x_shards, const uint16_t* const* gamma_shards,
                        int S, int64_t T, int64_t H, float eps, uint16_t* const* y_shards,
                        double* partials, double* acc, double* rstd, int nthreads) {
    if (S < 1 || T < 0 || H < 0 || (H % S) != 0) return -1;
    if (T == 0 || H == 0) return 0;
    if (!x_shards || !gamma_shards) return -1;
    const int64_t w = H / S;
    const double e = (double)eps;
    uint16_t* gfull = (uint16_t*)malloc((size_t)H * sizeof(uint16_t));
    if (!gfull) return -1;
    for (int s = 0; s < S; ++s) memcpy(gfull + s * w, gamma_shards[s], (size_t)w * sizeof(uint16_t));
    int nt = 1;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 1) nt = nthreads;
#pragma omp parallel for num_threads(nt) schedule(static)
#else
    (void)nthreads;
#endif
    for (int64_t t = 0; t < T; ++t) {
        uint16_t* row = (uint16_t*)malloc((size_t)H * sizeof(uint16_t));
        uint16_t* out = (uint16_t*)malloc((size_t)H * sizeof(uint16_t));
        if (!row || !out) {
            free(row);
            free(out);
            failed = 1;
            continue;
        }
        /* gather: slice s goes to columns [s*w, (s+1)*w) */
        for (int s = 0; s < S; ++s) memcpy(row + s * w, x_shards[s] + t * w, (size_t)w * sizeof(uint16_t));
        if (partials) {
            for (int s = 0; s < S; ++s) {
                double p = 0.0;
                for (int64_t j = 0; j < w; ++j) {
                    double v = qko_bf16_to_f64(x_shards[s][t * w + j]);
                    p += v * v;
                }
                partials[(int64_t)s * T + t] = p;
            }
        }
        rmsnorm_row(row, gfull, H, e, out, NULL, acc ? acc + t : NULL, rstd ? rstd + t : NULL);
        if (y_shards) {
            for (int s = 0; s < S; ++s)
                if (y_shards[s]) memcpy(y_shards[s] + t * w, out + s * w, (size_t)w * sizeof(uint16_t));
        }
        free(row);
        free(out);
    }
    free(gfull);
    return failed ? -1 : 0;
}

/* ---- FP8-E4M3 activations (Section IV-C: "BF16 and FP8-E4M3 activations", FP32 accumulation) ----
 *
 * The same definition (Eq. 1) with the activations stored as FP8 E4M3 (1 sign, 4
 * exponent bits with bias 7, 3 mantissa bits; no infinities, S.1111.111 is NaN,
 * largest finite value 448).  gamma stays bf16.  The output is rounded from fp64
 * to E4M3 in ONE step, to nearest even, and values beyond the largest finite
 * value saturate to +-448 (the paper does not say; this is the conversion the
 * hardware offers, cvt.rn.satfinite). */

double qko_e4m3_to_f64(uint8_t b) {
    const int sign = b >> 7, ex = (b >> 3) & 15, man = b & 7;
    double v;
    if (ex == 15 && man == 7) return sign ? -NAN : NAN;
    if (ex == 0) v = ldexp((double)man, -9);              /* subnormal: man/8 * 2^-6 */
    else v = ldexp(1.0 + (double)man / 8.0, ex - 7);
    return sign ? -v : v;
}

uint8_t qko_f64_to_e4m3(double v) {
    const uint8_t sign = signbit(v) ? 0x80u : 0x00u;
    if (isnan(v)) return (uint8_t)(sign | 0x7Fu);
    double a = fabs(v);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint8_t)(sign | 0x7Eu);         /* saturate */
    int ex;
    (void)frexp(a, &ex);
    int e = ex - 1;                                        /* floor(log2 a) */
    if (e < -6) e = -6;                                    /* subnormals share the smallest normal's unit */
    const double unit = ldexp(1.0, e - 3);                 /* 4 significant bits */
    double r = nearbyint(a / unit) * unit;                 /* nearest, ties to even */
    if (r > 448.0) r = 448.0;                              /* saturate to the largest finite value */
    if (r == 0.0) return sign;
    int rex;
    const double m = frexp(r, &rex);                       /* r = m * 2^rex, 0.5 <= m < 1 */
    int re = rex - 1;
    uint8_t bits;
    if (re < -6) {                                         /* subnormal: r = man * 2^-9 */
        bits = (uint8_t)(int)(r * 512.0);
    } else {
        const int man = (int)((m * 2.0 - 1.0) * 8.0);      /* exact: r has at most 4 significant bits */
        bits = (uint8_t)(((re + 7) << 3) | man);
    }
    return (uint8_t)(sign | bits);
}

static void rmsnorm_row_e4m3(const uint8_t* x, const uint16_t* gamma, int64_t H, double eps,
                             uint8_t* y, double* y64, double* acc_out, double* rstd_out) {
    double acc = 0.0;
    for (int64_t j = 0; j < H; ++j) {
        double v = qko_e4m3_to_f64(x[j]);
        acc += v * v;
    }
    double r = 1.0 / sqrt(acc / (double)H + eps);
    for (int64_t j = 0; j < H; ++j) {
        double o = qko_e4m3_to_f64(x[j]) * r * qko_bf16_to_f64(gamma[j]);
        if (y64) y64[j] = o;
        if (y) y[j] = qko_f64_to_e4m3(o);
    }
    if (acc_out) *acc_out = acc;
    if (rstd_out) *rstd_out = r;
}

/* x_shards[s]: [T][H/S] E4M3 bytes; gamma_shards[s]: [H/S] bf16.  S == 1 is the unsharded
 * form.  Same conventions as qko_rmsnorm_sharded (gather, Eq. 1 with the full width, cut back). */
int qko_rmsnorm_sharded_e4m3(const uint8_t* const* x_shards, const uint16_t* const* gamma_shards,
                             int S, int64_t T, int64_t H, float eps, uint8_t* const* y_shards,
                             double* y64, double* partials, double* acc, double* rstd, int nthreads) {
    if (S < 1 || T < 0 || H < 0 || (H % S) != 0) return -1;
    if (T == 0 || H == 0) return 0;
    if (!x_shards || !gamma_shards) return -1;
    const int64_t w = H / S;
    const double e = (double)eps;
    uint16_t* gfull = (uint16_t*)malloc((size_t)H * sizeof(uint16_t));
    if (!gfull) return -1;
    for (int s = 0; s < S; ++s) memcpy(gfull + s * w, gamma_shards[s], (size_t)w * sizeof(uint16_t));
    int nt = 1;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 1) nt = nthreads;
#pragma omp parallel for num_threads(nt) schedule(static)
#else
    (void)nthreads;
#endif
    for (int64_t t = 0; t < T; ++t) {
        uint8_t* row = (uint8_t*)malloc((size_t)H);
        uint8_t* out = (uint8_t*)malloc((size_t)H);
        if (!row || !out) {
            free(row);
            free(out);
            failed = 1;
            continue;
        }
        for (int s = 0; s < S; ++s) memcpy(row + s * w, x_shards[s] + t * w, (size_t)w);
        if (partials) {
            for (int s = 0; s < S; ++s) {
                double p = 0.0;
                for (int64_t j = 0; j < w; ++j) {
                    double v = qko_e4m3_to_f64(x_shards[s][t * w + j]);
                    p += v * v;
                }
                partials[(int64_t)s * T + t] = p;
            }
        }
        rmsnorm_row_e4m3(row, gfull, H, e, out, y64 ? y64 + t * H : NULL, acc ? acc + t : NULL,
                         rstd ? rstd + t : NULL);
        if (y_shards) {
            for (int s = 0; s < S; ++s)
                if (y_shards[s]) memcpy(y_shards[s] + t * w, out + s * w, (size_t)w);
        }
        free(row);
        free(out);
    }
    free(gfull);
    return failed ? -1 : 0;
}

/* ---- headwise granularity (Section II-A) ------------------------------------------------------
 *
 * Headwise granularity gives every attention head a factor of its own: the row is cut
 * into H/head_dim heads of head_dim consecutive elements and Eq. 1 is applied to every head on
 * its own (mean over head_dim), with the gamma entries of those columns.  Heads never straddle
 * a tensor-parallel shard, so the sharded form is the same computation on every shard buffer.
 * fp8 != 0 selects FP8-E4M3 activations (x, y are bytes), else bf16 (x, y are 16-bit words).
 * rstd (may be NULL): [T][H/head_dim]. */
int qko_rmsnorm_headwise(const void* x, const uint16_t* gamma, int64_t T, int64_t H, int64_t head_dim,
                         float eps, int fp8, void* y, double* y64, double* rstd, int nthreads) {
    if (T < 0 || H < 0 || head_dim < 1 || head_dim > 4096 || (H % head_dim) != 0) return -1;
    if (T == 0 || H == 0) return 0;
    if (!x || !gamma) return -1;
    const double e = (double)eps;
    const int64_t nh = H / head_dim;
    int nt = 1;
#ifdef _OPENMP
    if (nthreads > 1) nt = nthreads;
#pragma omp parallel for num_threads(nt) schedule(static)
#else
    (void)nthreads;
#endif
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t h = 0; h < nh; ++h) {
            const int64_t off = t * H + h * head_dim;
            if (fp8) {
                uint8_t head[4096];
                const int64_t n = head_dim <= 4096 ? head_dim : 4096;   /* head_dim is validated by the caller */
                memcpy(head, (const uint8_t*)x + off, (size_t)n);
                rmsnorm_row_e4m3(head, gamma + h * head_dim, n, e, y ? (uint8_t*)y + off : NULL,
                                 y64 ? y64 + off : NULL, NULL, rstd ? rstd + t * nh + h : NULL);
            } else {
                uint16_t head[4096];
                const int64_t n = head_dim <= 4096 ? head_dim : 4096;
                memcpy(head, (const uint16_t*)x + off, (size_t)n * sizeof(uint16_t));
                rmsnorm_row(head, gamma + h * head_dim, n, e, y ? (uint16_t*)y + off : NULL,
                            y64 ? y64 + off : NULL, NULL, rstd ? rstd + t * nh + h : NULL);
            }
        }
    }
    return 0;
}

/* Threads the OpenMP build will actually use when asked for n. */
int qko_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
