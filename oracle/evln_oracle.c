/*
 * fp64 CPU oracle for the "KV-cache reuse with contiguous RoPE" step (paper Sec. 3.2).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition of what one
 * navigation step computes, written out with ordinary loops in double precision:
 *
 *   1. the new frame's tokens get the position ids that continue the cached
 *      sequence, pos_i = L + i                      (Sec. 3.2: ids stay contiguous);
 *   2. the new queries and keys are rotated by RoPE at those positions
 *      (Sec. 3.2: rotation applied when the step runs; 1-D NeoX half-split pairing);
 *   3. rotated keys and the unchanged values are appended to the reused cache
 *      (Sec. 3.2: the cached tensors are joined with the new frame's);
 *   4. only the new frame is prefilled: each new query attends causally to all
 *      cached tokens and to the new tokens up to itself (Sec. 3.2: the transformer
 *      prefill covers the current frame alone).
 *
 * It shares nothing with the CUDA library: no headers, no constants, no helpers.
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call it.
 *
 * Layouts (all token-major, row-major, double):
 *   q_new [n][Hq][D]   k_new,v_new [n][Hkv][D]   k_cache,v_cache [cap][Hkv][D]
 *   out   [n][Hq][D]   lse [n][Hq]               probs (optional) [n][Hq][L+n]
 *
 * Parity pins (tests/test_oracle_pins.py): RoPE closed forms (position 0, D=2, a
 * hand-worked D=4 vector), pair-norm preservation, relative-position invariance,
 * chained steps == brute-force full causal prefill (a separate NumPy program),
 * == the library's scaled-dot-product attention, softmax rows sum to one,
 * Q=0 -> running mean of V, causality, GQA == replicated MHA, split merge == unsplit,
 * bf16 rounding == the library's float->bfloat16 conversion incl. ties.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- storage rounding -------------------------------------------------- */

/* Round a double to the nearest bfloat16 value (8 significant bits, exponent range of
 * binary32), ties to even, directly from the double: no intermediate float rounding. */
double evln_oracle_round_bf16(double x)
{
    if (x == 0.0 || isnan(x) || isinf(x)) return x;
    int e;
    (void)frexp(x, &e);          /* |x| = f * 2^e, f in [0.5, 1)  ->  2^(e-1) <= |x| < 2^e */
    int exp2 = e - 1;            /* exponent of the leading bit                           */
    if (exp2 < -126) exp2 = -126;            /* subnormal range: fixed spacing 2^-133     */
    double ulp = ldexp(1.0, exp2 - 7);       /* 7 fraction bits                           */
    double q = nearbyint(x / ulp) * ulp;     /* default rounding mode = ties to even      */
    /* largest finite bf16 = (2 - 2^-7) * 2^127 ; anything that rounds above it -> inf    */
    double maxv = (2.0 - ldexp(1.0, -7)) * ldexp(1.0, 127);
    if (fabs(q) > maxv) q = (x > 0) ? INFINITY : -INFINITY;
    return q;
}

static double round_storage(double x, int mode)
{
    if (mode == 1) return evln_oracle_round_bf16(x);
    if (mode == 2) return (double)(float)x;   /* binary32, ties to even */
    return x;
}

void evln_oracle_round_array(double* x, long count, int mode)
{
    for (long i = 0; i < count; ++i) x[i] = round_storage(x[i], mode);
}

/* ---- RoPE (Sec. 3.2; half-split pairing (j, j + D/2)) ------------------- */

/* x,y: [n][H][D]; token i is rotated at position pos0 + i.
 * omega_j = theta^(-2j/D); phi = pos * omega_j;
 * y_j       = x_j cos(phi) - x_{j+D/2} sin(phi)
 * y_{j+D/2} = x_{j+D/2} cos(phi) + x_j sin(phi)                                          */
void evln_oracle_rope(const double* x, double* y, int n, int H, int D, long pos0, double theta)
{
    int half = D / 2;
    for (int i = 0; i < n; ++i) {
        double pos = (double)(pos0 + i);
        for (int h = 0; h < H; ++h) {
            const double* xi = x + ((long)i * H + h) * D;
            double* yi = y + ((long)i * H + h) * D;
            for (int j = 0; j < half; ++j) {
                double omega = pow(theta, -2.0 * (double)j / (double)D);
                double phi = pos * omega;
                double c = cos(phi), s = sin(phi);
                double a = xi[j], b = xi[j + half];
                yi[j] = a * c - b * s;
                yi[j + half] = b * c + a * s;
            }
        }
    }
}

/* ---- one step: rotate, append, attend ----------------------------------- */

/* storage_mode: 0 keep doubles, 1 cache is bfloat16, 2 cache is binary32.  The rotated
 * keys are rounded once to the cache type when they are stored; V is stored as given.
 * q_rot_out (optional, [n][Hq][D]) receives the unrounded rotated queries.
 * scale <= 0 selects 1/sqrt(D).  Returns 0, or 1 if L+n exceeds cap.                     */
int evln_oracle_step(const double* q_new, const double* k_new, const double* v_new,
                     double* k_cache, double* v_cache, long cap,
                     int n, int Hq, int Hkv, int D, long L, double theta, double scale,
                     int storage_mode, double* out, double* lse, double* probs,
                     double* q_rot_out)
{
    if (L + n > cap || Hq % Hkv != 0 || D % 2 != 0) return 1;
    int G = Hq / Hkv;
    long T = L + n;
    if (scale <= 0) scale = 1.0 / sqrt((double)D);

    double* q_rot = (double*)malloc(sizeof(double) * (size_t)n * Hq * D);
    double* k_rot = (double*)malloc(sizeof(double) * (size_t)n * Hkv * D);
    evln_oracle_rope(q_new, q_rot, n, Hq, D, L, theta);
    evln_oracle_rope(k_new, k_rot, n, Hkv, D, L, theta);

    /* append at slots L .. L+n-1 */
    for (long i = 0; i < n; ++i)
        for (long e = 0; e < (long)Hkv * D; ++e) {
            k_cache[(L + i) * Hkv * D + e] = round_storage(k_rot[i * Hkv * D + e], storage_mode);
            v_cache[(L + i) * Hkv * D + e] = v_new[i * Hkv * D + e];
        }

    /* attention of new query i (head h, kv head g = h / G) over keys 0 .. L+i */
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
    for (int i = 0; i < n; ++i) {
        for (int h = 0; h < Hq; ++h) {
            int g = h / G;
            long nk = L + i + 1;
            const double* q = q_rot + ((long)i * Hq + h) * D;
            double* s = (double*)malloc(sizeof(double) * (size_t)nk);
            double m = -INFINITY;
            for (long t = 0; t < nk; ++t) {
                const double* k = k_cache + (t * Hkv + g) * D;
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += q[d] * k[d];
                s[t] = acc * scale;
                if (s[t] > m) m = s[t];
            }
            double l = 0.0;
            for (long t = 0; t < nk; ++t) { s[t] = exp(s[t] - m); l += s[t]; }
            double* o = out + ((long)i * Hq + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (long t = 0; t < nk; ++t) {
                double p = s[t] / l;
                const double* v = v_cache + (t * Hkv + g) * D;
                for (int d = 0; d < D; ++d) o[d] += p * v[d];
                if (probs) probs[((long)i * Hq + h) * T + t] = p;
            }
            if (probs) for (long t = nk; t < T; ++t) probs[((long)i * Hq + h) * T + t] = 0.0;
            if (lse) lse[(long)i * Hq + h] = m + log(l);
            free(s);
        }
    }
    if (q_rot_out) memcpy(q_rot_out, q_rot, sizeof(double) * (size_t)n * Hq * D);
    free(q_rot);
    free(k_rot);
    return 0;
}

/* ---- attention restricted to a key range (to test split merging) -------- */

/* Softmax attention of already-rotated queries over cache slots [t0, min(t1, L+i+1)).
 * A row whose range is empty gets out = 0 and lse = -inf.                                */
void evln_oracle_attend_range(const double* q_rot, const double* k_cache, const double* v_cache,
                              int n, int Hq, int Hkv, int D, long L, long t0, long t1,
                              double scale, double* out, double* lse)
{
    int G = Hq / Hkv;
    if (scale <= 0) scale = 1.0 / sqrt((double)D);
    for (int i = 0; i < n; ++i)
        for (int h = 0; h < Hq; ++h) {
            int g = h / G;
            long hi = L + i + 1 < t1 ? L + i + 1 : t1;
            const double* q = q_rot + ((long)i * Hq + h) * D;
            double* o = out + ((long)i * Hq + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (hi <= t0) { lse[(long)i * Hq + h] = -INFINITY; continue; }
            double m = -INFINITY;
            for (long t = t0; t < hi; ++t) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += q[d] * k_cache[(t * Hkv + g) * D + d];
                if (acc * scale > m) m = acc * scale;
            }
            double l = 0.0;
            for (long t = t0; t < hi; ++t) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += q[d] * k_cache[(t * Hkv + g) * D + d];
                double p = exp(acc * scale - m);
                l += p;
                for (int d = 0; d < D; ++d) o[d] += p * v_cache[(t * Hkv + g) * D + d];
            }
            for (int d = 0; d < D; ++d) o[d] /= l;
            lse[(long)i * Hq + h] = m + log(l);
        }
}

/* ---- merge of per-split partial results --------------------------------- */

/* o_parts [S][rows][D] (each normalised within its split), lse_parts [S][rows].
 * M = max_s lse_s;  O = sum_s e^{lse_s-M} O_s / sum_s e^{lse_s-M};  lse = M + log(sum).
 * A split with lse = -inf has weight zero; if every split is empty the row is 0 / -inf.  */
void evln_oracle_combine(const double* o_parts, const double* lse_parts, int S, long rows, int D,
                         double* out, double* lse)
{
    for (long r = 0; r < rows; ++r) {
        double M = -INFINITY;
        for (int s = 0; s < S; ++s)
            if (lse_parts[(long)s * rows + r] > M) M = lse_parts[(long)s * rows + r];
        double* o = out + r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (isinf(M) && M < 0) { if (lse) lse[r] = -INFINITY; continue; }
        double wsum = 0.0;
        for (int s = 0; s < S; ++s) {
            double w = exp(lse_parts[(long)s * rows + r] - M);
            wsum += w;
            for (int d = 0; d < D; ++d) o[d] += w * o_parts[((long)s * rows + r) * D + d];
        }
        for (int d = 0; d < D; ++d) o[d] /= wsum;
        if (lse) lse[r] = M + log(wsum);
    }
}

int evln_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
