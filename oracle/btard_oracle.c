/*
 * Float64 CPU oracle for batched CenteredClip and its verification pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * GPU library must compute.  It shares no code, header, table or helper with the
 * CUDA path; only tests, the smoke check and the benchmark's CPU-baseline leg may
 * load it.  Every function cites the passage of the paper (arXiv 2106.11257,
 * "Secure Distributed Training at Scale") it restates.
 *
 * Parity pins (see tests/test_oracle_*.py): tau = inf gives the mean; one row
 * returns that row; permutation invariance; the clipped-residual sum vanishes at
 * the fixed point; 1-D closed forms; the tau*b/n shift bound; Split sizes;
 * Philox4x32-10 published known answers; z against a libm Box-Muller.
 * parity unpinned (the paper fixes neither): the eps stopping criterion
 * (|| v^{l+1} - v^l ||_2 <= eps, tested after the update) and the rule for
 * non-finite rows (weight 0, row left out of the sum).
 *
 * Arithmetic is double precision throughout, in the order the equations are
 * written: one loop over rows, one loop over coordinates, no blocking or fusion.
 * Inputs are the same fp32 bit patterns the GPU reads, promoted to double.
 * The only single-precision arithmetic is the map from Philox words to the
 * coordinates of z, whose fp32 results are part of the definition of z.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_SPLIT_PAPER 0
#define ORACLE_SPLIT_CEIL_PAD 1

#define ORACLE_INIT_CALLER 0
#define ORACLE_INIT_ZERO 1
#define ORACLE_INIT_MEAN 2
#define ORACLE_INIT_COORD_MEDIAN 3

#define ORACLE_STOP_FIXED 0
#define ORACLE_STOP_EPS 1

#define ORACLE_STATUS_NOT_CONVERGED 1u
#define ORACLE_STATUS_NONFINITE_ROW 2u

/* ------------------------------------------------------------------------- */
/* Split(v, n): App. D.1 "Basic building blocks".                             */
/* mode PAPER: the first d mod P parts have ceil(d/P) entries, the rest        */
/* floor(d/P).  mode CEIL_PAD: every part has ceil(d/P) entries until d runs   */
/* out; the tail part is short (possibly empty) and is zero-padded in memory.  */
/* row_stride = the longest part rounded up to a multiple of align_elems.      */
/* ------------------------------------------------------------------------- */
int btard_oracle_partition_layout(int64_t d, int32_t P, int32_t mode, int32_t align_elems,
                                  int64_t *part_offset, int64_t *part_len, int64_t *row_stride)
{
    if (d < 0 || P < 1 || align_elems < 1) return -1;
    if (mode != ORACLE_SPLIT_PAPER && mode != ORACLE_SPLIT_CEIL_PAD) return -1;
    int64_t fl = d / P, rem = d % P, ce = fl + (rem ? 1 : 0);
    int64_t off = 0, longest = 0;
    for (int32_t j = 0; j < P; ++j) {
        int64_t len;
        if (mode == ORACLE_SPLIT_PAPER) {
            len = (j < rem) ? ce : fl;
        } else {
            len = d - off;
            if (len > ce) len = ce;
        }
        part_offset[j] = off;
        part_len[j] = len;
        off += len;
        if (len > longest) longest = len;
    }
    *row_stride = (longest + align_elems - 1) / align_elems * align_elems;
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), the counter-based        */
/* generator behind GetRandomVector (Alg. 6, "z = GetRandomVector(r)").        */
/* ------------------------------------------------------------------------- */
void btard_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static float u32_as_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static uint32_t f32_as_u32(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

/*
 * Two Philox words -> two standard normals (Box-Muller), in fp32 with a fixed
 * operation order so that the result is a function of the words alone:
 *   u  = ((a >> 8) + 1) / 2^24 in (0, 1],  t = -ln u,
 *   y  = ((b >> 6 & 0xFFFFFF) + 1/2) / 2^24 - 1/2 in (-1/2, 1/2),  phi = (pi/2) y,
 *   (n0, n1) = sqrt(t) (cos phi - sin phi, cos phi + sin phi)
 *            = sqrt(2t) (cos(phi + pi/4), sin(phi + pi/4)),
 * then bit 31 of b flips the sign of n0 and bit 30 that of n1, which spreads the
 * angle over the full circle.  ln, sin and cos are fixed polynomials (absolute
 * error about 3e-7, 6e-7 and 3e-8); every operation is an IEEE single add,
 * multiply, fused multiply-add or square root.  Compile with -ffp-contract=off.
 */
static void normal_pair(uint32_t a, uint32_t b, float *n0, float *n1)
{
    uint32_t i = (a >> 8) + 1u;
    uint32_t bits = f32_as_u32((float)i);
    uint32_t e = (bits - 0x3F3504F3u) >> 23;            /* 2^e * m = i, m in [sqrt(1/2), sqrt 2) */
    float m = u32_as_f32(bits - (e << 23));
    float x = m - 1.0f;
    float q = 0x1.eaf59cp-4f;
    q = fmaf(q, x, -0x1.803d52p-3f);
    q = fmaf(q, x, 0x1.a3b028p-3f);
    q = fmaf(q, x, -0x1.fde802p-3f);
    q = fmaf(q, x, 0x1.5526b4p-2f);
    q = fmaf(q, x, -0x1.0001f2p-1f);
    float x2 = x * x;
    float lnm = fmaf(x2, q, x);                          /* ln m */
    float t = fmaf((float)(24 - (int32_t)e), 0x1.62e43p-1f, -lnm);
    t = fmaxf(t, 0.0f);
    float r = sqrtf(t);

    uint32_t j = (b >> 6) & 0xFFFFFFu;
    float y = fmaf((float)j, 0x1p-24f, -0x1.fffffep-2f); /* (j + 1/2) 2^-24 - 1/2 */
    float z = y * y;
    float s = 0x1.3e202ap-4f;
    s = fmaf(s, z, -0x1.4a9ac4p-1f);
    s = fmaf(s, z, 0x1.921f32p+0f);
    s = s * y;
    float c = -0x1.4e5ed6p-6f;
    c = fmaf(c, z, 0x1.03af5cp-2f);
    c = fmaf(c, z, -0x1.3bd392p+0f);
    c = fmaf(c, z, 1.0f);
    float a0 = r * (c - s);
    float a1 = r * (c + s);
    *n0 = u32_as_f32(f32_as_u32(a0) ^ (b & 0x80000000u));
    *n1 = u32_as_f32(f32_as_u32(a1) ^ ((b << 1) & 0x80000000u));
}

/*
 * GetRandomVector (Alg. 6; App. D.5: z uniform on the unit sphere, i.e. iid
 * normal coordinates, normalised by the caller through ||z||).  Coordinates
 * 4q..4q+3 of vector k of partition p come from one Philox call with
 * counter = (q, p, k, 0x42544152) and key = (seed low word, seed high word):
 * words 0,1 give coordinates 4q, 4q+1 and words 2,3 give 4q+2, 4q+3.
 * Writes the unnormalised fp32 coordinates z[0 .. part_len).
 */
void btard_oracle_random_vector(uint64_t seed, int32_t p, int32_t k, int64_t part_len, float *z)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (int64_t q = 0; 4 * q < part_len; ++q) {
        uint32_t ctr[4] = { (uint32_t)q, (uint32_t)p, (uint32_t)k, 0x42544152u };
        uint32_t w[4];
        float nrm[4];
        btard_oracle_philox4x32_10(ctr, key, w);
        normal_pair(w[0], w[1], &nrm[0], &nrm[1]);
        normal_pair(w[2], w[3], &nrm[2], &nrm[3]);
        for (int t = 0; t < 4; ++t)
            if (4 * q + t < part_len) z[4 * q + t] = nrm[t];
    }
}

/* ------------------------------------------------------------------------- */
/* Coordinate-wise median (named as a baseline aggregator in Sec. 4.1; used    */
/* here only as a starting point v^0).  Values are ordered by the IEEE total   */
/* order of their bit patterns (-NaN < -inf < ... < -0 < +0 < ... < +inf <     */
/* +NaN); for even n the result is the mean of the two middle values.          */
/* ------------------------------------------------------------------------- */
static uint64_t order_key64(double d)
{
    uint64_t u; memcpy(&u, &d, 8);
    return (u & 0x8000000000000000ull) ? ~u : (u | 0x8000000000000000ull);
}
static int cmp_key64(const void *a, const void *b)
{
    uint64_t x = order_key64(*(const double *)a), y = order_key64(*(const double *)b);
    return (x > y) - (x < y);
}
/* Row i as the aggregation sees it: f_i g_i when per-row factors are given (the per-part clipping of
   BTARD-Clipped-SGD, Alg. 9, applied on the fly), g_i otherwise.  A factor of exactly 0 drops the row
   (it reads as zeros whatever it holds); a factor of 1 changes nothing, bit for bit. */
static double row_value(const float *x, int64_t c, double f)
{
    return (f == 0.0) ? 0.0 : f * (double)x[c];
}
static double factor_of(const double *row_scale, int32_t i) { return row_scale ? row_scale[i] : 1.0; }

static void coord_median(const float *g, int32_t n, int64_t stride, int64_t len, const double *row_scale, double *v)
{
    double *col = (double *)malloc(sizeof(double) * (size_t)n);
    for (int64_t c = 0; c < len; ++c) {
        for (int32_t i = 0; i < n; ++i) col[i] = row_value(g + (int64_t)i * stride, c, factor_of(row_scale, i));
        qsort(col, (size_t)n, sizeof(double), cmp_key64);
        if (n & 1) v[c] = col[n / 2];
        else v[c] = (col[n / 2 - 1] + col[n / 2]) / 2.0;
    }
    free(col);
}

/* ------------------------------------------------------------------------- */
/* CenteredClip on one partition (App. D.2, eq. (CenteredClip)):               */
/*   v^{l+1} = v^l + (1/n) sum_i (x_i - v^l) min{1, tau / ||x_i - v^l||}       */
/* rows x_i = g[i*stride .. i*stride+len).  Returns v (double, length len),    */
/* the residual norms ||x_i - v|| at the returned v, the number of updates     */
/* applied, the norm of the last update and a status word.                     */
/* ------------------------------------------------------------------------- */
static double clip_weight(double rho, double tau, uint32_t *status)
{
    if (!isfinite(rho)) { *status |= ORACLE_STATUS_NONFINITE_ROW; return 0.0; }
    if (rho <= tau) return 1.0;          /* covers rho = 0 and tau = inf */
    return tau / rho;
}

static double residual_norm(const float *x, double f, const double *v, int64_t len)
{
    double acc = 0.0;
    for (int64_t c = 0; c < len; ++c) {
        double r = row_value(x, c, f) - v[c];
        acc += r * r;
    }
    return sqrt(acc);
}

#define ORACLE_RULE_CENTERED_CLIP 0
#define ORACLE_RULE_GEOMETRIC_MEDIAN 1   /* Weiszfeld's iteration; the baseline "geometric median" of Sec. 4.1 */
#define ORACLE_RULE_MEAN 2               /* plain averaging (All-Reduce baseline of Sec. 4.1)                   */
#define ORACLE_RULE_COORD_MEDIAN 3       /* coordinate-wise median baseline of Sec. 4.1                          */

int btard_oracle_aggregate_one(int32_t rule, const float *g, int32_t n, int64_t stride, int64_t len,
                               double tau, int32_t init_mode, const float *v0,
                               int32_t stop_mode, int32_t max_iters, double eps,
                               double *v, double *resid_norm, int32_t *iters,
                               double *last_step_norm, uint32_t *status);
int btard_oracle_aggregate_one_ex(int32_t rule, const float *g, int32_t n, int64_t stride, int64_t len,
                                  double tau, const double *tau_sched, const double *row_scale,
                                  int32_t init_mode, const float *v0,
                                  int32_t stop_mode, int32_t max_iters, double eps,
                                  double *v, double *resid_norm, int32_t *iters,
                                  double *last_step_norm, uint32_t *status);

int btard_oracle_centered_clip_one(const float *g, int32_t n, int64_t stride, int64_t len,
                                   double tau, int32_t init_mode, const float *v0,
                                   int32_t stop_mode, int32_t max_iters, double eps,
                                   double *v, double *resid_norm, int32_t *iters,
                                   double *last_step_norm, uint32_t *status)
{
    return btard_oracle_aggregate_one(ORACLE_RULE_CENTERED_CLIP, g, n, stride, len, tau, init_mode, v0,
                                      stop_mode, max_iters, eps, v, resid_norm, iters, last_step_norm,
                                      status);
}

/*
 * One partition under one of the aggregation rules the paper compares (Sec. 4.1).
 *   CENTERED_CLIP:    App. D.2 eq. (CenteredClip), w_i = min{1, tau / rho_i}, v += (1/n) sum_i w_i r_i.
 *   GEOMETRIC_MEDIAN: Weiszfeld, v <- sum_i x_i / rho_i / sum_i 1 / rho_i with rho_i floored at tau,
 *                     written as v += sum_i (1/rho_i) r_i / sum_i (1/rho_i); same stop rules.
 *   MEAN / COORD_MEDIAN: v is the mean / coordinate-wise median of the rows; no update, iters = 0.
 * Two optional inputs:
 *   tau_sched [max_iters]: update l uses the radius tau_sched[l] (the schedule tau_l of App. D.2) instead of
 *     the constant tau;
 *   row_scale [n]: row i enters as row_scale[i] g_i, the per-part clipped gradient of BTARD-Clipped-SGD
 *     (Alg. 9: g~_i(l) = min{1, lambda / ||g_i(l)||} g_i(l)) without rewriting g.
 */
int btard_oracle_aggregate_one(int32_t rule, const float *g, int32_t n, int64_t stride, int64_t len,
                               double tau, int32_t init_mode, const float *v0,
                               int32_t stop_mode, int32_t max_iters, double eps,
                               double *v, double *resid_norm, int32_t *iters,
                               double *last_step_norm, uint32_t *status)
{
    return btard_oracle_aggregate_one_ex(rule, g, n, stride, len, tau, NULL, NULL, init_mode, v0, stop_mode,
                                         max_iters, eps, v, resid_norm, iters, last_step_norm, status);
}

int btard_oracle_aggregate_one_ex(int32_t rule, const float *g, int32_t n, int64_t stride, int64_t len,
                                  double tau, const double *tau_sched, const double *row_scale,
                                  int32_t init_mode, const float *v0,
                                  int32_t stop_mode, int32_t max_iters, double eps,
                                  double *v, double *resid_norm, int32_t *iters,
                                  double *last_step_norm, uint32_t *status)
{
    if (n < 1 || len < 0 || stride < len || max_iters < 1) return -1;
    if (!(tau >= 0.0)) return -1;
    if (rule == ORACLE_RULE_GEOMETRIC_MEDIAN && !(tau > 0.0 && isfinite(tau))) return -1;
    if (rule == ORACLE_RULE_MEAN) { init_mode = ORACLE_INIT_MEAN; max_iters = 0; stop_mode = ORACLE_STOP_FIXED; }
    if (rule == ORACLE_RULE_COORD_MEDIAN) { init_mode = ORACLE_INIT_COORD_MEDIAN; max_iters = 0; stop_mode = ORACLE_STOP_FIXED; }
    uint32_t st = 0;
    /* v^0: the paper leaves the starting point open (App. D.2, "a sequence {v_l}"). */
    if (init_mode == ORACLE_INIT_CALLER) {
        for (int64_t c = 0; c < len; ++c) v[c] = (double)v0[c];
    } else if (init_mode == ORACLE_INIT_ZERO) {
        for (int64_t c = 0; c < len; ++c) v[c] = 0.0;
    } else if (init_mode == ORACLE_INIT_MEAN) {
        for (int64_t c = 0; c < len; ++c) {
            double acc = 0.0;
            for (int32_t i = 0; i < n; ++i) acc += row_value(g + (int64_t)i * stride, c, factor_of(row_scale, i));
            v[c] = acc / n;
        }
    } else if (init_mode == ORACLE_INIT_COORD_MEDIAN) {
        coord_median(g, n, stride, len, row_scale, v);
    } else {
        return -1;
    }

    double *w = (double *)malloc(sizeof(double) * (size_t)n);
    double *u = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
    double step = 0.0;
    int32_t done = 0;
    for (int32_t l = 0; l < max_iters; ++l) {
        if (tau_sched) {                                /* tau_l of App. D.2 */
            tau = tau_sched[l];
            if (!(tau >= 0.0)) { free(w); free(u); return -1; }
        }
        if (rule == ORACLE_RULE_GEOMETRIC_MEDIAN) {
            double total = 0.0;
            for (int32_t i = 0; i < n; ++i) {
                double rho = residual_norm(g + (int64_t)i * stride, factor_of(row_scale, i), v, len);
                if (!isfinite(rho)) { st |= ORACLE_STATUS_NONFINITE_ROW; w[i] = 0.0; }
                else w[i] = 1.0 / (rho > tau ? rho : tau);
                total += w[i];
            }
            /* scaled so that the common update below, (1/n) sum_i w_i r_i, is the Weiszfeld step */
            for (int32_t i = 0; i < n; ++i) w[i] = total > 0.0 ? n * w[i] / total : 0.0;
        } else {
            for (int32_t i = 0; i < n; ++i)
                w[i] = clip_weight(residual_norm(g + (int64_t)i * stride, factor_of(row_scale, i), v, len), tau, &st);
        }
        for (int64_t c = 0; c < len; ++c) u[c] = 0.0;
        for (int32_t i = 0; i < n; ++i) {
            if (w[i] == 0.0) continue;                  /* weight 0: the row is left out */
            const float *x = g + (int64_t)i * stride;
            const double f = factor_of(row_scale, i);
            for (int64_t c = 0; c < len; ++c) u[c] += w[i] * (row_value(x, c, f) - v[c]);
        }
        double s2 = 0.0;
        for (int64_t c = 0; c < len; ++c) {
            u[c] /= n;
            v[c] += u[c];
            s2 += u[c] * u[c];
        }
        step = sqrt(s2);
        done = l + 1;
        if (stop_mode == ORACLE_STOP_EPS && step <= eps) break;
    }
    if (stop_mode == ORACLE_STOP_EPS && !(step <= eps)) st |= ORACLE_STATUS_NOT_CONVERGED;
    for (int32_t i = 0; i < n; ++i) {
        double rho = residual_norm(g + (int64_t)i * stride, factor_of(row_scale, i), v, len);
        if (!isfinite(rho)) st |= ORACLE_STATUS_NONFINITE_ROW;
        resid_norm[i] = rho;
    }
    *iters = done;
    *last_step_norm = step;
    *status = st;
    free(w);
    free(u);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Verification metadata for one partition (Sec. 3.1 eq. (2); Alg. 6):         */
/*   norm_i = ||g_i - v||, w_i = min{1, tau/norm_i},                            */
/*   dot_ik = <g_i - v, z_k> (z_k unnormalised), s_ik = w_i dot_ik / ||z_k||,  */
/*   s_sum_k = sum_i s_ik, resid_sum = sum_i w_i (g_i - v) and its 2-norm.     */
/* v is the fp32 vector a peer would have received.  If norm_in is not NULL    */
/* the weights are taken from those norms (as reported by the aggregation).    */
/* ------------------------------------------------------------------------- */
int btard_oracle_verify_one_ex(const float *g, int32_t n, int64_t stride, int64_t len,
                               const float *v, double tau, const double *row_scale, uint64_t seed, int32_t p, int32_t K,
                               const double *norm_in, double *norm, double *weight, double *dot,
                               double *s, double *s_sum, double *znorm2, double *resid_sum_norm,
                               double *resid_sum /* [len] or NULL */, uint32_t *status);

int btard_oracle_verify_one(const float *g, int32_t n, int64_t stride, int64_t len,
                            const float *v, double tau, uint64_t seed, int32_t p, int32_t K,
                            const double *norm_in, double *norm, double *weight, double *dot,
                            double *s, double *s_sum, double *znorm2, double *resid_sum_norm,
                            double *resid_sum /* [len] or NULL */, uint32_t *status)
{
    return btard_oracle_verify_one_ex(g, n, stride, len, v, tau, NULL, seed, p, K, norm_in, norm, weight, dot, s,
                                      s_sum, znorm2, resid_sum_norm, resid_sum, status);
}

/* row_scale [n] or NULL: row i enters as row_scale[i] g_i (the clipped gradients of Alg. 9), as in the
   aggregation. */
int btard_oracle_verify_one_ex(const float *g, int32_t n, int64_t stride, int64_t len,
                               const float *v, double tau, const double *row_scale, uint64_t seed, int32_t p, int32_t K,
                               const double *norm_in, double *norm, double *weight, double *dot,
                               double *s, double *s_sum, double *znorm2, double *resid_sum_norm,
                               double *resid_sum /* [len] or NULL */, uint32_t *status)
{
    if (n < 1 || len < 0 || stride < len || K < 1 || !(tau >= 0.0)) return -1;
    uint32_t st = 0;
    double *vd = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
    float *z = (float *)malloc(sizeof(float) * (size_t)(len > 0 ? len : 1));
    double *rs = (double *)calloc((size_t)(len > 0 ? len : 1), sizeof(double));
    for (int64_t c = 0; c < len; ++c) vd[c] = (double)v[c];

    for (int32_t i = 0; i < n; ++i) {
        norm[i] = norm_in ? norm_in[i] : residual_norm(g + (int64_t)i * stride, factor_of(row_scale, i), vd, len);
        weight[i] = clip_weight(norm[i], tau, &st);
    }
    for (int32_t k = 0; k < K; ++k) {
        btard_oracle_random_vector(seed, p, k, len, z);
        double zz = 0.0;
        for (int64_t c = 0; c < len; ++c) zz += (double)z[c] * (double)z[c];
        znorm2[k] = zz;
        s_sum[k] = 0.0;
        for (int32_t i = 0; i < n; ++i) {
            const float *x = g + (int64_t)i * stride;
            const double f = factor_of(row_scale, i);
            double acc = 0.0;
            for (int64_t c = 0; c < len; ++c) acc += (row_value(x, c, f) - vd[c]) * (double)z[c];
            dot[(int64_t)i * K + k] = acc;
            /* an empty partition has no coordinates: the inner product is the empty sum, 0 */
            double sik = (weight[i] == 0.0 || zz == 0.0) ? 0.0 : weight[i] * acc / sqrt(zz);
            s[(int64_t)i * K + k] = sik;
            s_sum[k] += sik;
        }
    }
    for (int32_t i = 0; i < n; ++i) {
        if (weight[i] == 0.0) continue;
        const float *x = g + (int64_t)i * stride;
        const double f = factor_of(row_scale, i);
        for (int64_t c = 0; c < len; ++c) rs[c] += weight[i] * (row_value(x, c, f) - vd[c]);
    }
    double acc = 0.0;
    for (int64_t c = 0; c < len; ++c) {
        acc += rs[c] * rs[c];
        if (resid_sum) resid_sum[c] = rs[c];
    }
    *resid_sum_norm = sqrt(acc);
    *status = st;
    free(vd);
    free(z);
    free(rs);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Batched drivers over the [P][n][stride] tensor: the P partitions of          */
/* ButterflyClip (Alg. 2, aggregation) are independent, so they are simply looped;  */
/* OpenMP, when enabled, runs whole partitions on different cores and changes  */
/* no arithmetic.  v is [P][stride] doubles (entries past part_len[p] are 0).  */
/* ------------------------------------------------------------------------- */
int btard_oracle_aggregate(int32_t rule, const float *g, int32_t n, int32_t P, int64_t stride,
                           const int64_t *part_len, const double *tau, int32_t init_mode,
                           const float *v0, int32_t stop_mode, int32_t max_iters, double eps,
                           double *v, double *resid_norm, int32_t *iters, double *last_step_norm,
                           uint32_t *status)
{
    int rc_all = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t p = 0; p < P; ++p) {
        double *vp = v + (int64_t)p * stride;
        for (int64_t c = 0; c < stride; ++c) vp[c] = 0.0;
        int rc = btard_oracle_aggregate_one(
            rule, g + (int64_t)p * n * stride, n, stride, part_len[p], tau[p], init_mode,
            v0 ? v0 + (int64_t)p * stride : NULL, stop_mode, max_iters, eps, vp,
            resid_norm + (int64_t)p * n, iters + p, last_step_norm + p, status + p);
        if (rc) {
#pragma omp atomic write
            rc_all = rc;
        }
    }
    return rc_all;
}

/* The same with the two optional inputs: tau_sched [P][max_iters] and row_scale [P][n] (either may be NULL). */
int btard_oracle_aggregate_ex(int32_t rule, const float *g, int32_t n, int32_t P, int64_t stride,
                              const int64_t *part_len, const double *tau, const double *tau_sched,
                              const double *row_scale, int32_t init_mode, const float *v0, int32_t stop_mode,
                              int32_t max_iters, double eps, double *v, double *resid_norm, int32_t *iters,
                              double *last_step_norm, uint32_t *status)
{
    int rc_all = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t p = 0; p < P; ++p) {
        double *vp = v + (int64_t)p * stride;
        for (int64_t c = 0; c < stride; ++c) vp[c] = 0.0;
        int rc = btard_oracle_aggregate_one_ex(
            rule, g + (int64_t)p * n * stride, n, stride, part_len[p], tau[p],
            tau_sched ? tau_sched + (int64_t)p * max_iters : NULL, row_scale ? row_scale + (int64_t)p * n : NULL,
            init_mode, v0 ? v0 + (int64_t)p * stride : NULL, stop_mode, max_iters, eps, vp,
            resid_norm + (int64_t)p * n, iters + p, last_step_norm + p, status + p);
        if (rc) {
#pragma omp atomic write
            rc_all = rc;
        }
    }
    return rc_all;
}

int btard_oracle_centered_clip(const float *g, int32_t n, int32_t P, int64_t stride,
                               const int64_t *part_len, const double *tau, int32_t init_mode,
                               const float *v0 /* [P][stride] or NULL */, int32_t stop_mode,
                               int32_t max_iters, double eps, double *v, double *resid_norm,
                               int32_t *iters, double *last_step_norm, uint32_t *status)
{
    int rc_all = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t p = 0; p < P; ++p) {
        double *vp = v + (int64_t)p * stride;
        for (int64_t c = 0; c < stride; ++c) vp[c] = 0.0;
        int rc = btard_oracle_centered_clip_one(
            g + (int64_t)p * n * stride, n, stride, part_len[p], tau[p], init_mode,
            v0 ? v0 + (int64_t)p * stride : NULL, stop_mode, max_iters, eps, vp,
            resid_norm + (int64_t)p * n, iters + p, last_step_norm + p, status + p);
        if (rc) {
#pragma omp atomic write
            rc_all = rc;
        }
    }
    return rc_all;
}

int btard_oracle_verify(const float *g, int32_t n, int32_t P, int64_t stride,
                        const int64_t *part_len, const float *v, const double *tau, uint64_t seed,
                        int32_t K, const double *norm_in, double *norm, double *weight,
                        double *dot, double *s, double *s_sum, double *znorm2,
                        double *resid_sum_norm, double *resid_sum /* [P][stride] or NULL */,
                        uint32_t *status)
{
    int rc_all = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t p = 0; p < P; ++p) {
        if (resid_sum)
            for (int64_t c = 0; c < stride; ++c) resid_sum[(int64_t)p * stride + c] = 0.0;
        int rc = btard_oracle_verify_one(
            g + (int64_t)p * n * stride, n, stride, part_len[p], v + (int64_t)p * stride, tau[p],
            seed, p, K, norm_in ? norm_in + (int64_t)p * n : NULL, norm + (int64_t)p * n,
            weight + (int64_t)p * n, dot + (int64_t)p * n * K, s + (int64_t)p * n * K,
            s_sum + (int64_t)p * K, znorm2 + (int64_t)p * K, resid_sum_norm + p,
            resid_sum ? resid_sum + (int64_t)p * stride : NULL, status + p);
        if (rc) {
#pragma omp atomic write
            rc_all = rc;
        }
    }
    return rc_all;
}

/* ------------------------------------------------------------------------- */
/* Verifications 1-3 on the broadcast scalars (Alg. 6, Verifications), for one       */
/* partition.  "differs" is |a - b| > rel_tol max(|a|,|b|) + abs_tol (NaN        */
/* differs); all-zero tolerances give the paper's exact tests.                   */
/* ------------------------------------------------------------------------- */
static int oracle_differs(double x, double y, double rel_tol, double abs_tol)
{
    double scale = fabs(x) > fabs(y) ? fabs(x) : fabs(y);
    return !(fabs(x - y) <= rel_tol * scale + abs_tol);
}

void btard_oracle_checks_one(int32_t n, int32_t K, const double *norm, const double *norm_reported,
                             const double *s, const double *s_reported, double delta_max,
                             double rel_tol, double abs_tol, double sum_tol,
                             uint8_t *norm_mismatch, uint8_t *s_mismatch, uint8_t *sum_violation,
                             uint8_t *check, int32_t *votes, uint8_t *check_averaging)
{
    int32_t v = 0;
    for (int32_t i = 0; i < n; ++i) {
        /* Verification 1: reported norm against the recomputed one */
        norm_mismatch[i] = norm_reported ? (uint8_t)oracle_differs(norm_reported[i], norm[i], rel_tol, abs_tol) : 0;
        /* Verification 3: is the aggregate farther than Delta_max from this peer's part? */
        check[i] = (uint8_t)(norm[i] > delta_max);
        v += check[i];
        /* Verification 2, first test: reported inner products against the recomputed ones */
        for (int32_t k = 0; k < K; ++k)
            s_mismatch[i * K + k] =
                s_reported ? (uint8_t)oracle_differs(s_reported[i * K + k], s[i * K + k], rel_tol, abs_tol) : 0;
    }
    /* Verification 2, second test: the broadcast inner products must sum to zero */
    for (int32_t k = 0; k < K; ++k) {
        const double *sv = s_reported ? s_reported : s;
        double sum = 0.0, mag = 0.0;
        for (int32_t i = 0; i < n; ++i) { sum += sv[i * K + k]; mag += fabs(sv[i * K + k]); }
        sum_violation[k] = (uint8_t)(!(fabs(sum) <= sum_tol * mag));
    }
    *votes = v;
    *check_averaging = (uint8_t)(2 * v > n);      /* more than n/2 peers voted */
}

/* ------------------------------------------------------------------------- */
/* Per-part clipping of BTARD-Clipped-SGD (Alg. 9 and the paragraph after it):  */
/*   g~_i(l) = min{1, lambda / ||g_i(l)||} g_i(l).  One row; a row whose norm is */
/*   not finite is set to zero (factor 0).                                      */
/* ------------------------------------------------------------------------- */
void btard_oracle_preclip_row(const float *x, int64_t len, double lambda, double *out, double *norm,
                              double *factor)
{
    double acc = 0.0;
    for (int64_t c = 0; c < len; ++c) acc += (double)x[c] * (double)x[c];
    double nrm = sqrt(acc), f;
    if (!isfinite(nrm)) f = 0.0;
    else f = (nrm <= lambda) ? 1.0 : lambda / nrm;
    for (int64_t c = 0; c < len; ++c) out[c] = (f == 0.0) ? 0.0 : f * (double)x[c];
    *norm = nrm;
    *factor = f;
}

/* ------------------------------------------------------------------------- */
/* Commitments (Alg. 2, hash broadcasts): SHA-256 (FIPS 180-4), byte oriented, and  */
/* the two-level tree over 4096-byte chunks that the library defines:            */
/*   H(row) = SHA256(SHA256(chunk_0) || ... || SHA256(chunk_m-1) || LE64(bytes)). */
/* ------------------------------------------------------------------------- */
static const uint32_t sha_k[64] = {
    0x428a2f98u, 0x71374491u, 0xb5c0fbcfu, 0xe9b5dba5u, 0x3956c25bu, 0x59f111f1u, 0x923f82a4u, 0xab1c5ed5u,
    0xd807aa98u, 0x12835b01u, 0x243185beu, 0x550c7dc3u, 0x72be5d74u, 0x80deb1feu, 0x9bdc06a7u, 0xc19bf174u,
    0xe49b69c1u, 0xefbe4786u, 0x0fc19dc6u, 0x240ca1ccu, 0x2de92c6fu, 0x4a7484aau, 0x5cb0a9dcu, 0x76f988dau,
    0x983e5152u, 0xa831c66du, 0xb00327c8u, 0xbf597fc7u, 0xc6e00bf3u, 0xd5a79147u, 0x06ca6351u, 0x14292967u,
    0x27b70a85u, 0x2e1b2138u, 0x4d2c6dfcu, 0x53380d13u, 0x650a7354u, 0x766a0abbu, 0x81c2c92eu, 0x92722c85u,
    0xa2bfe8a1u, 0xa81a664bu, 0xc24b8b70u, 0xc76c51a3u, 0xd192e819u, 0xd6990624u, 0xf40e3585u, 0x106aa070u,
    0x19a4c116u, 0x1e376c08u, 0x2748774cu, 0x34b0bcb5u, 0x391c0cb3u, 0x4ed8aa4au, 0x5b9cca4fu, 0x682e6ff3u,
    0x748f82eeu, 0x78a5636fu, 0x84c87814u, 0x8cc70208u, 0x90befffau, 0xa4506cebu, 0xbef9a3f7u, 0xc67178f2u};

static uint32_t ror32(uint32_t x, int n) { return (x >> n) | (x << (32 - n)); }

static void sha256_block(uint32_t h[8], const unsigned char *blk)
{
    uint32_t w[64];
    for (int i = 0; i < 16; ++i)
        w[i] = ((uint32_t)blk[4 * i] << 24) | ((uint32_t)blk[4 * i + 1] << 16) | ((uint32_t)blk[4 * i + 2] << 8) | blk[4 * i + 3];
    for (int i = 16; i < 64; ++i) {
        uint32_t s0 = ror32(w[i - 15], 7) ^ ror32(w[i - 15], 18) ^ (w[i - 15] >> 3);
        uint32_t s1 = ror32(w[i - 2], 17) ^ ror32(w[i - 2], 19) ^ (w[i - 2] >> 10);
        w[i] = w[i - 16] + s0 + w[i - 7] + s1;
    }
    uint32_t a = h[0], b = h[1], c = h[2], d = h[3], e = h[4], f = h[5], g = h[6], hh = h[7];
    for (int i = 0; i < 64; ++i) {
        uint32_t t1 = hh + (ror32(e, 6) ^ ror32(e, 11) ^ ror32(e, 25)) + ((e & f) ^ (~e & g)) + sha_k[i] + w[i];
        uint32_t t2 = (ror32(a, 2) ^ ror32(a, 13) ^ ror32(a, 22)) + ((a & b) ^ (a & c) ^ (b & c));
        hh = g; g = f; f = e; e = d + t1; d = c; c = b; b = a; a = t1 + t2;
    }
    h[0] += a; h[1] += b; h[2] += c; h[3] += d; h[4] += e; h[5] += f; h[6] += g; h[7] += hh;
}

void btard_oracle_sha256(const unsigned char *msg, int64_t len, unsigned char out[32])
{
    uint32_t h[8] = {0x6a09e667u, 0xbb67ae85u, 0x3c6ef372u, 0xa54ff53au,
                     0x510e527fu, 0x9b05688cu, 0x1f83d9abu, 0x5be0cd19u};
    int64_t at = 0;
    for (; at + 64 <= len; at += 64) sha256_block(h, msg + at);
    unsigned char tail[128];
    int64_t rest = len - at;
    memset(tail, 0, sizeof tail);
    memcpy(tail, msg + at, (size_t)rest);
    tail[rest] = 0x80;
    int blocks = (rest + 1 + 8 <= 64) ? 1 : 2;
    uint64_t bits = (uint64_t)len * 8u;
    for (int i = 0; i < 8; ++i) tail[64 * blocks - 1 - i] = (unsigned char)(bits >> (8 * i));
    for (int b = 0; b < blocks; ++b) sha256_block(h, tail + 64 * b);
    for (int i = 0; i < 8; ++i) {
        out[4 * i] = (unsigned char)(h[i] >> 24); out[4 * i + 1] = (unsigned char)(h[i] >> 16);
        out[4 * i + 2] = (unsigned char)(h[i] >> 8); out[4 * i + 3] = (unsigned char)h[i];
    }
}

void btard_oracle_commitment(const float *row, int64_t len, unsigned char out[32])
{
    const int64_t bytes = 4 * len, chunk = 4096;
    const int64_t m = (bytes + chunk - 1) / chunk;
    unsigned char *cat = (unsigned char *)malloc((size_t)(32 * m + 8));
    for (int64_t c = 0; c < m; ++c) {
        int64_t nb = bytes - c * chunk < chunk ? bytes - c * chunk : chunk;
        btard_oracle_sha256((const unsigned char *)row + c * chunk, nb, cat + 32 * c);
    }
    for (int i = 0; i < 8; ++i) cat[32 * m + i] = (unsigned char)((uint64_t)bytes >> (8 * i));
    btard_oracle_sha256(cat, 32 * m + 8, out);
    free(cat);
}

int btard_oracle_max_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
