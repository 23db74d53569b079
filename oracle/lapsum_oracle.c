/*
 * LapSum exact-budget soft top-k: CPU ORACLE.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, single-threaded, fp64, obviously-correct C.
 * It shares no code with the CUDA library and is never linked into it; only
 * tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * What it computes (paper notation; t = |alpha| > 0):
 *   sigma(u) = 1/2 e^u (u<=0), 1 - 1/2 e^{-u} (u>0)            Eq. 3 / App. A
 *   Lap(b)   = sum_i sigma((r_i - b)/t),  solve Lap(b) = k       Eq. 1-2
 *   p_i      = sigma((r_i - b)/t)
 *   VJP      = f .* (g - <g,q>), q = f/sum f,
 *              f_i = e^{-|b-r_i|/t}/(2t)                         Eq. 5
 *   bracketed solve with tail sums S_L, S_R and |R|              Eq. 7, App. B
 *   binomial order-statistic bracket indices j, l                Eq. 8, Alg. 1
 *   validated path: one-sided doubling of a failed bracket,
 *   full sort after max_widen attempts                           Sec. 4, App. C
 *   gradients with respect to k and alpha (implicit differentiation
 *   of sum p = k; the paper learns both, Sec. 6)
 *   alpha > 0 (forward, backward, scalar gradients): Eq. 1 as printed,
 *   p_i = sigma((b - r_i)/alpha), which then decreases in r_i (the k
 *   smallest scores); solved as the alpha < 0 problem on the negated
 *   scores (b -> -b).  The bracket routines take alpha < 0 only.
 *
 * How the threshold is found (App. A: sort, prefix/suffix exponential scans
 * as the affine recurrence x_i = w_i x_{i-1} + 1, node values, interval
 * lookup, closed-form root of the per-interval quadratic):
 *   nodes  x_0 = a_L (if finite), x_1..x_M = sorted middle set, x_{M+1} = a_R
 *   A_j    = sum over elements at or below node j of e^{(r - x_j)/t}
 *            A_0 = S_L,  A_j = A_{j-1} e^{-(x_j - x_{j-1})/t} + 1
 *   B'_j   = sum over elements above node j of e^{-(r - x_j)/t}
 *            Bs_{M+1} = S_R, B'_j = Bs_{j+1} e^{-(x_{j+1}-x_j)/t}, Bs_j = B'_j + 1
 *   F_j    = A_j/2 + N_above(j) - B'_j/2,   N_above(j) = |R| + M - j
 *   j*     = max{ j : F_j >= k }
 *   with c = N_above(j*) - k, lo = x_{j*}, hi = x_{j*+1}, d = hi - lo:
 *     c <= 0:  u = e^{(b-lo)/t} solves  B' u^2 - 2 c u - A = 0,  B' = Bs e^{-d/t}
 *              u = A / (sqrt(c^2 + A B') - c),   b = lo + t ln u
 *     c >  0:  w = e^{(hi-b)/t} solves  A' w^2 + 2 c w - Bs = 0, A' = A e^{-d/t}
 *              w = Bs / (c + sqrt(c^2 + A' Bs)), b = hi - t ln w
 *     c == 0:  b = (lo+hi)/2 + (t/2) ln(A/Bs)    (same root, no underflow)
 *   The unbracketed problem is the case a_L = -inf, a_R = +inf, S_L = S_R = 0.
 *
 * Pins (tests/test_oracle_*.py): full-sum bisection on tiny inputs, closed
 * forms (n = 1, all-equal scores), the symmetric k = n/2 case, the
 * zero-temperature midpoint (Theorem 1), sum p = k, monotonicity, shift and
 * scale invariance, brute-force node values, finite-difference gradients at
 * the paper's shapes (Table "gradcheck"), hand-computed bracket indices,
 * finite differences in k and alpha for the scalar gradients, hand-worked ends
 * and doubling counts for the widening, the validated path's threshold against
 * the full sort; for alpha > 0 bisection on Eq. 1 itself, the n = 1 closed
 * form, the complement identity p(r; k, alpha) = 1 - p(r; n-k, -alpha) and
 * the same finite differences.
 * No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_EARG -1
#define ORACLE_ENOMEM -2
/* bracketed solve outcomes */
#define ORACLE_ROOT_LEFT 1  /* Lap(a_L) < k : root lies left of the bracket  */
#define ORACLE_ROOT_RIGHT 2 /* Lap(a_R) > k : root lies right of the bracket */

/* ------------------------------------------------------------------ */
/* total order on fp32 scores: ascending by the sign-flipped bit pattern;
 * equal patterns keep ascending original index.  -0.0 sorts before +0.0. */
static uint32_t order_key(float x)
{
    uint32_t b;
    memcpy(&b, &x, 4);
    return (b >> 31) ? ~b : (b | 0x80000000u);
}

static float key_to_float(uint32_t u)
{
    uint32_t b = (u >> 31) ? (u & 0x7fffffffu) : ~u;
    float x;
    memcpy(&x, &b, 4);
    return x;
}

/* stable merge sort of 64-bit composites (key << 32 | index) */
static void merge_sort_u64(uint64_t *a, uint64_t *tmp, int64_t n)
{
    if (n <= 24) {
        for (int64_t i = 1; i < n; ++i) {
            uint64_t v = a[i];
            int64_t j = i - 1;
            while (j >= 0 && a[j] > v) {
                a[j + 1] = a[j];
                --j;
            }
            a[j + 1] = v;
        }
        return;
    }
    int64_t h = n / 2;
    merge_sort_u64(a, tmp, h);
    merge_sort_u64(a + h, tmp + h, n - h);
    if (a[h - 1] <= a[h])
        return;
    memcpy(tmp, a, (size_t)h * sizeof(uint64_t));
    int64_t i = 0, j = h, o = 0;
    while (i < h && j < n)
        a[o++] = (a[j] < tmp[i]) ? a[j++] : tmp[i++];
    while (i < h)
        a[o++] = tmp[i++];
}

/* sorted (key, original index) pairs of one row; n < 2^32 */
int oracle_sort_pairs(const float *r, int64_t n, float *keys_out, uint32_t *idx_out)
{
    if (!r || n < 1 || n > 0xffffffffLL)
        return ORACLE_EARG;
    uint64_t *a = (uint64_t *)malloc((size_t)n * 8);
    uint64_t *tmp = (uint64_t *)malloc((size_t)n * 8);
    if (!a || !tmp) {
        free(a);
        free(tmp);
        return ORACLE_ENOMEM;
    }
    for (int64_t i = 0; i < n; ++i)
        a[i] = ((uint64_t)order_key(r[i]) << 32) | (uint64_t)i;
    merge_sort_u64(a, tmp, n);
    for (int64_t i = 0; i < n; ++i) {
        if (keys_out)
            keys_out[i] = key_to_float((uint32_t)(a[i] >> 32));
        if (idx_out)
            idx_out[i] = (uint32_t)(a[i] & 0xffffffffu);
    }
    free(a);
    free(tmp);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ */
static double laplace_cdf(double u)
{
    return (u <= 0.0) ? 0.5 * exp(u) : 1.0 - 0.5 * exp(-u);
}

/* Lap(b) by the plain definition: one full sum */
double oracle_lap_sum(const float *r, int64_t n, double b, double t)
{
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i)
        s += laplace_cdf(((double)r[i] - b) / t);
    return s;
}

/* Eq. 1 as printed, either sign of alpha: G(b) = sum_i sigma((b - r_i)/alpha) */
static double eq1_sum(const float *r, int64_t n, double b, double alpha)
{
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i)
        s += laplace_cdf((b - (double)r[i]) / alpha);
    return s;
}

/* prior-art solver: bisection on the full sum (cross-check on tiny inputs).
 * G decreases in b for alpha < 0 and increases for alpha > 0. */
int oracle_bisect(const float *r, int64_t n, double k, double alpha, double *b_out)
{
    if (!r || n < 1 || !(alpha != 0.0) || !isfinite(alpha) || !(k > 0.0) || !(k < (double)n))
        return ORACLE_EARG;
    double t = fabs(alpha), lo = r[0], hi = r[0];
    int dec = alpha < 0.0;
    for (int64_t i = 1; i < n; ++i) {
        if (r[i] < lo) lo = r[i];
        if (r[i] > hi) hi = r[i];
    }
    /* move lo left until the root is right of it, hi right until it is left of it */
    double w = t;
    while (dec ? eq1_sum(r, n, lo, alpha) < k : eq1_sum(r, n, lo, alpha) > k) { lo -= w; w *= 2.0; }
    w = t;
    while (dec ? eq1_sum(r, n, hi, alpha) > k : eq1_sum(r, n, hi, alpha) < k) { hi += w; w *= 2.0; }
    for (int it = 0; it < 400; ++it) {
        double mid = 0.5 * (lo + hi);
        if (!(mid > lo && mid < hi))
            break;
        double g = eq1_sum(r, n, mid, alpha);
        if (dec ? g >= k : g <= k) lo = mid; else hi = mid;
    }
    *b_out = 0.5 * (lo + hi);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ */
typedef struct {
    double b;        /* threshold */
    int64_t jstar;   /* crossing node index (0..M), see header */
    double c;        /* N_above(j*) - k */
    double A, Bs;    /* A_{j*} (pivot lo) and Bs_{j*+1} (pivot hi) */
    double lo, hi;   /* the interval that holds the root */
    double F_aL, F_aR; /* Lap(a_L), Lap(a_R) when those ends are finite, else +/-inf */
    int status;      /* 0, ORACLE_ROOT_LEFT, ORACLE_ROOT_RIGHT */
} oracle_solve_info;

/*
 * Seeded solve over an ascending-sorted middle set x[0..M) (App. B).
 * a_L = -INFINITY / a_R = +INFINITY mean "no left / right tail".
 * node_F (nullable, M+2 doubles) receives F_0..F_{M+1}.
 */
int oracle_solve_sorted(const double *x, int64_t M, double k, double t,
                        double a_L, double S_L, double a_R, double S_R, int64_t n_R,
                        double *node_F, oracle_solve_info *out)
{
    if (M < 0 || !(t > 0.0) || !out)
        return ORACLE_EARG;
    /* Bs[j] for j = 1..M+1 (pivot node j, self included for j<=M) */
    double *Bs = (double *)malloc((size_t)(M + 2) * sizeof(double));
    if (!Bs)
        return ORACLE_ENOMEM;
    Bs[M + 1] = S_R;
    for (int64_t j = M; j >= 1; --j) {
        double above = (j == M) ? a_R : x[j]; /* node j+1 */
        double Bp = Bs[j + 1] * exp(-(above - x[j - 1]) / t);
        Bs[j] = Bp + 1.0;
    }
    int has_L = isfinite(a_L), has_R = isfinite(a_R);
    int64_t jstar = -1;
    double A_star = 0.0, A = has_L ? S_L : 0.0, prev = a_L;
    double F0 = INFINITY;
    if (has_L) {
        double first = (M > 0) ? x[0] : a_R;
        double Bp0 = Bs[1] * exp(-(first - a_L) / t);
        F0 = 0.5 * A + (double)(n_R + M) - 0.5 * Bp0;
    }
    if (node_F) node_F[0] = F0;
    if (F0 >= k) { jstar = 0; A_star = A; }
    for (int64_t j = 1; j <= M; ++j) {
        double xj = x[j - 1];
        A = (j == 1 && !has_L) ? 1.0 : A * exp(-(xj - prev) / t) + 1.0;
        prev = xj;
        double above = (j == M) ? a_R : x[j];
        double Bp = Bs[j + 1] * exp(-(above - xj) / t);
        double F = 0.5 * A + (double)(n_R + M - j) - 0.5 * Bp;
        if (node_F) node_F[j] = F;
        if (F >= k) { jstar = j; A_star = A; }
    }
    double FR = -INFINITY;
    if (has_R) {
        double A_R = (M == 0 && !has_L) ? 0.0 : A * exp(-(a_R - prev) / t);
        FR = 0.5 * A_R + (double)n_R - 0.5 * S_R;
    }
    if (node_F) node_F[M + 1] = FR;
    out->F_aL = F0;
    out->F_aR = FR;
    out->status = 0;
    out->jstar = jstar;
    if (jstar < 0) { out->status = ORACLE_ROOT_LEFT; out->b = a_L; free(Bs); return ORACLE_OK; }
    if (has_R && FR > k) { out->status = ORACLE_ROOT_RIGHT; out->b = a_R; free(Bs); return ORACLE_OK; }

    double lo = (jstar == 0) ? a_L : x[jstar - 1];
    double hi = (jstar == M) ? a_R : x[jstar];
    double c = (double)(n_R + M - jstar) - k;
    double Bhi = Bs[jstar + 1];
    double b;
    if (c == 0.0) {
        b = 0.5 * (lo + hi) + 0.5 * t * log(A_star / Bhi);
    } else if (c < 0.0) {
        double Bp = isfinite(hi) ? Bhi * exp(-(hi - lo) / t) : 0.0;
        double u = A_star / (sqrt(c * c + A_star * Bp) - c);
        b = lo + t * log(u);
    } else {
        double Ap = isfinite(lo) ? A_star * exp(-(hi - lo) / t) : 0.0;
        double w = Bhi / (c + sqrt(c * c + Ap * Bhi));
        b = hi - t * log(w);
    }
    if (b < lo) b = lo;
    if (b > hi) b = hi;
    out->b = b; out->c = c; out->A = A_star; out->Bs = Bhi; out->lo = lo; out->hi = hi;
    free(Bs);
    return ORACLE_OK;
}

static int sorted_doubles(const float *r, int64_t n, double **out)
{
    float *keys = (float *)malloc((size_t)n * sizeof(float));
    if (!keys) return ORACLE_ENOMEM;
    int rc = oracle_sort_pairs(r, n, keys, NULL);
    if (rc) { free(keys); return rc; }
    double *s = (double *)malloc((size_t)n * sizeof(double));
    if (!s) { free(keys); return ORACLE_ENOMEM; }
    for (int64_t i = 0; i < n; ++i) s[i] = (double)keys[i];
    free(keys);
    *out = s;
    return ORACLE_OK;
}

/*
 * Forward (Eq. 1-3, App. A): per row, sort, scan, look up, solve, map.
 * p (rows*n doubles, nullable), b (rows doubles), jstar (rows, nullable),
 * node_F (rows*(n+2) doubles, nullable; tiny inputs only).
 */
int oracle_forward(const float *r, int64_t rows, int64_t n, double k, double alpha,
                   double *p, double *b, int64_t *jstar, double *node_F)
{
    if (!r || !b || rows < 1 || n < 1 || !(alpha != 0.0) || !isfinite(alpha) ||
        !(k > 0.0) || !(k < (double)n))
        return ORACLE_EARG;
    double t = fabs(alpha);
    if (alpha > 0.0 && node_F)
        return ORACLE_EARG; /* node values are those of the alpha < 0 problem; jstar then counts the negated scores */
    for (int64_t row = 0; row < rows; ++row) {
        const float *rr = r + row * n;
        double *s = NULL;
        int rc = sorted_doubles(rr, n, &s);
        if (rc) return rc;
        if (alpha > 0.0) { /* the negated scores, ascending: sum_i sigma((-r_i - b')/t) = k, b = -b' */
            for (int64_t i = 0; i < n / 2; ++i) {
                double lo_v = s[i];
                s[i] = -s[n - 1 - i];
                s[n - 1 - i] = -lo_v;
            }
            if (n & 1) s[n / 2] = -s[n / 2];
        }
        oracle_solve_info info;
        rc = oracle_solve_sorted(s, n, k, t, -INFINITY, 0.0, INFINITY, 0.0, 0,
                                 node_F ? node_F + row * (n + 2) : NULL, &info);
        free(s);
        if (rc) return rc;
        b[row] = alpha > 0.0 ? -info.b : info.b;
        if (jstar) jstar[row] = info.jstar;
        if (p)
            for (int64_t i = 0; i < n; ++i)
                p[row * n + i] = laplace_cdf((b[row] - (double)rr[i]) / alpha); /* Eq. 1 */
    }
    return ORACLE_OK;
}

/* Backward (Eq. 5): grad = f .* (v - sum(v f)/sum(f)); zero when sum f == 0.
 * For alpha > 0 the Jacobian of Eq. 1 changes sign (p_i then falls as r_i rises, and
 * db/dr_j = f_j/sum f still): grad = -f .* (v - sum(v f)/sum(f)). */
int oracle_backward(const float *v, const float *r, const double *b, int64_t rows, int64_t n,
                    double alpha, double *grad)
{
    if (!v || !r || !b || !grad || rows < 1 || n < 1 || !(alpha != 0.0))
        return ORACLE_EARG;
    double t = fabs(alpha), sgn = alpha < 0.0 ? 1.0 : -1.0;
    for (int64_t row = 0; row < rows; ++row) {
        const float *rr = r + row * n, *vv = v + row * n;
        double sf = 0.0, svf = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double f = exp(-fabs(b[row] - (double)rr[i]) / t) / (2.0 * t);
            sf += f;
            svf += (double)vv[i] * f;
        }
        double mean = (sf > 0.0) ? svf / sf : 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double f = exp(-fabs(b[row] - (double)rr[i]) / t) / (2.0 * t);
            grad[row * n + i] = (sf > 0.0) ? sgn * f * ((double)vv[i] - mean) : 0.0;
        }
    }
    return ORACLE_OK;
}

/*
 * Gradients with respect to the two scalars the paper's applications also learn (Sec. 6: the attack
 * "learns both alpha and k"); the paper prints no formula, these follow from implicit differentiation
 * of sum_i p_i = k with p_i = sigma((r_i - b)/t), t = -alpha, f_i as in Eq. 5:
 *   dp_i/dk     = f_i / sum f                          =>  grad_k     = sum(v f) / sum(f)
 *   dp_i/dt     = -(f_i/t) [ (r_i-b) - sum_j f_j (r_j-b) / sum f ]
 *   grad_alpha  = -grad_t = (1/t) [ sum v f (r-b) - (sum v f / sum f) sum f (r-b) ]
 * Both are 0 when sum f underflows to 0.
 * For alpha > 0 (p_i = sigma((b - r_i)/alpha), t = alpha) the same two expressions hold: dp_i/dk = f_i / sum f
 * again, and dp_i/dalpha = f_i [ (r_i - b) - sum_j f_j (r_j - b)/sum f ] / alpha.
 */
int oracle_backward_scalars(const float *v, const float *r, const double *b, int64_t rows, int64_t n, double alpha,
                            double *grad_k, double *grad_alpha)
{
    if (!v || !r || !b || !grad_k || !grad_alpha || rows < 1 || n < 1 || !(alpha != 0.0))
        return ORACLE_EARG;
    double t = fabs(alpha);
    for (int64_t row = 0; row < rows; ++row) {
        const float *rr = r + row * n, *vv = v + row * n;
        double sf = 0.0, svf = 0.0, sfd = 0.0, svfd = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double d = (double)rr[i] - b[row];
            double f = exp(-fabs(d) / t) / (2.0 * t);
            sf += f;
            svf += (double)vv[i] * f;
            sfd += f * d;
            svfd += (double)vv[i] * f * d;
        }
        if (sf > 0.0) {
            grad_k[row] = svf / sf;
            grad_alpha[row] = (svfd - (svf / sf) * sfd) / t;
        } else {
            grad_k[row] = 0.0;
            grad_alpha[row] = 0.0;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ */
/* Bracket (Eq. 8, Alg. 1) with the systematic sampler.
 *
 * The paper fixes K = ceil(n^{2/3}), q = (n-k)/n, j and l, z = 5.16, and says
 * only that the deployed sampler is a strided view with pre-computed kernel
 * noise.  The sampler specified here (and implemented independently in the
 * CUDA library) is:
 *   K       least integer with K^3 >= n^2
 *   stride  floor(n / K)
 *   i_s     s*stride + hash32(s*0x9E3779B9 + seed_lo) mod stride,  s = 0..K-1
 *   U_s     (hash32(s*0x9E3779B9 + (seed_hi ^ 0x68E31DA4)) + 0.5) / 2^32
 *   e_s     unit Laplace by inverse CDF: ln(2U) for U < 1/2, else -ln(2(1-U)),
 *           evaluated in fp64 and rounded once to fp32
 *   y_s     fmaf((float)t, e_s, r[i_s])          (one fp32 rounding)
 * hash32 is the 32-bit murmur3 finaliser.
 */
static uint32_t hash32(uint32_t h)
{
    h ^= h >> 16; h *= 0x85ebca6bu;
    h ^= h >> 13; h *= 0xc2b2ae35u;
    h ^= h >> 16;
    return h;
}

int64_t oracle_sample_count(int64_t n)
{
    /* least K with K^3 >= n^2 */
    unsigned __int128 n2 = (unsigned __int128)n * (unsigned __int128)n;
    int64_t K = (int64_t)floor(pow((double)n, 2.0 / 3.0));
    while (K > 1 && (unsigned __int128)(K - 1) * (K - 1) * (K - 1) >= n2) --K;
    while ((unsigned __int128)K * K * K < n2) ++K;
    return K;
}

void oracle_bracket_indices(int64_t n, double k, double z, int64_t *K_out, int64_t *j_out, int64_t *l_out)
{
    int64_t K = oracle_sample_count(n);
    double q = ((double)n - k) / (double)n;
    double mu = (double)K * q, sd = sqrt((double)K * q * (1.0 - q));
    *K_out = K;
    *j_out = (int64_t)floor(mu - z * sd);
    *l_out = (int64_t)ceil(mu + z * sd);
}

float oracle_noise(uint64_t seed, int64_t s)
{
    uint32_t seed_hi = (uint32_t)(seed >> 32);
    uint32_t h = hash32((uint32_t)s * 0x9E3779B9u + (seed_hi ^ 0x68E31DA4u));
    double U = ((double)h + 0.5) / 4294967296.0;
    double e = (U < 0.5) ? log(2.0 * U) : -log(2.0 * (1.0 - U));
    return (float)e;
}

int64_t oracle_sample_index(uint64_t seed, int64_t s, int64_t n, int64_t K)
{
    int64_t stride = n / K;
    uint32_t h = hash32((uint32_t)s * 0x9E3779B9u + (uint32_t)(seed & 0xffffffffu));
    return s * stride + (int64_t)(h % (uint32_t)stride);
}

void oracle_noise_table(uint64_t seed, int64_t K, float *out)
{
    for (int64_t s = 0; s < K; ++s) out[s] = oracle_noise(seed, s);
}

void oracle_sample_indices(uint64_t seed, int64_t n, int64_t K, int64_t *out)
{
    for (int64_t s = 0; s < K; ++s) out[s] = oracle_sample_index(seed, s, n, K);
}

typedef struct {
    int64_t K, j, l;      /* Eq. 8 (1-indexed ascending order statistics) */
    float a_L, a_R;       /* -inf when j < 1, +inf when l > K */
    int64_t n_L, n_M, n_R;
    double S_L, S_R;      /* Eq. 7 */
} oracle_bracket_info;

/* y (K floats, nullable) receives the noised sample in draw order */
int oracle_bracket(const float *r, int64_t n, double k, double alpha, double z, uint64_t seed,
                   float *y, oracle_bracket_info *out)
{
    if (!r || !out || n < 8 || !(alpha < 0.0) || !(k > 0.0) || !(k < (double)n))
        return ORACLE_EARG;
    double t = -alpha;
    float tf = (float)t;
    int64_t K, j, l;
    oracle_bracket_indices(n, k, z, &K, &j, &l);
    float *ys = (float *)malloc((size_t)K * sizeof(float));
    float *sorted = (float *)malloc((size_t)K * sizeof(float));
    if (!ys || !sorted) { free(ys); free(sorted); return ORACLE_ENOMEM; }
    for (int64_t s = 0; s < K; ++s)
        ys[s] = fmaf(tf, oracle_noise(seed, s), r[oracle_sample_index(seed, s, n, K)]);
    if (y) memcpy(y, ys, (size_t)K * sizeof(float));
    int rc = oracle_sort_pairs(ys, K, sorted, NULL);
    if (rc) { free(ys); free(sorted); return rc; }
    out->K = K; out->j = j; out->l = l;
    out->a_L = (j >= 1) ? sorted[j - 1] : -INFINITY;
    out->a_R = (l <= K) ? sorted[l - 1] : INFINITY;
    free(ys);
    free(sorted);
    /* one streaming pass (Alg. 1, App. B): L = {r < a_L}, M = {a_L <= r < a_R}, R = {r >= a_R} */
    int64_t nL = 0, nM = 0, nR = 0;
    double SL = 0.0, SR = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        float x = r[i];
        if (x < out->a_L) { ++nL; SL += exp(((double)x - (double)out->a_L) / t); }
        else if (x >= out->a_R) { ++nR; SR += exp(-((double)x - (double)out->a_R) / t); }
        else ++nM;
    }
    out->n_L = nL; out->n_M = nM; out->n_R = nR; out->S_L = SL; out->S_R = SR;
    return ORACLE_OK;
}

/*
 * Exact solve inside a given bracket [a_L, a_R) (App. B): stream once for the
 * tails, gather and sort the middle set, run the seeded solve.  status reports
 * a failed certificate Lap(a_R) <= k <= Lap(a_L) (Alg. 1).  band_keys
 * (nullable, capacity band_cap) receives the sorted middle set.
 */
int oracle_forward_bracketed(const float *r, int64_t n, double k, double alpha, float a_L, float a_R,
                             double *p, double *b, int *status, int64_t *counts /* nL,nM,nR */,
                             double *tails /* S_L,S_R */, float *band_keys, int64_t band_cap)
{
    if (!r || !b || !status || n < 1 || !(alpha < 0.0) || !(k > 0.0) || !(k < (double)n))
        return ORACLE_EARG;
    double t = -alpha;
    int64_t nL = 0, nM = 0, nR = 0;
    double SL = 0.0, SR = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        float x = r[i];
        if (x < a_L) { ++nL; SL += exp(((double)x - (double)a_L) / t); }
        else if (x >= a_R) { ++nR; SR += exp(-((double)x - (double)a_R) / t); }
        else ++nM;
    }
    float *mid = (float *)malloc((size_t)(nM > 0 ? nM : 1) * sizeof(float));
    if (!mid) return ORACLE_ENOMEM;
    int64_t w = 0;
    for (int64_t i = 0; i < n; ++i)
        if (!(r[i] < a_L) && !(r[i] >= a_R)) mid[w++] = r[i];
    double *x = NULL;
    if (nM > 0) {
        int rc = sorted_doubles(mid, nM, &x);
        if (rc) { free(mid); return rc; }
    }
    if (band_keys)
        for (int64_t i = 0; i < nM && i < band_cap; ++i) band_keys[i] = (float)x[i];
    free(mid);
    oracle_solve_info info;
    int rc = oracle_solve_sorted(x, nM, k, t, (double)a_L, SL, (double)a_R, SR, nR, NULL, &info);
    free(x);
    if (rc) return rc;
    *status = info.status;
    *b = info.b;
    if (counts) { counts[0] = nL; counts[1] = nM; counts[2] = nR; }
    if (tails) { tails[0] = SL; tails[1] = SR; }
    if (p && info.status == 0)
        for (int64_t i = 0; i < n; ++i) p[i] = laplace_cdf(((double)r[i] - info.b) / t);
    return ORACLE_OK;
}

/*
 * One-sided doubling of a bracket whose certificate failed (App. C, "Expected
 * linear time": the missed side moves to [a_R, a_R + 2(a_R - a_L)], mirrored
 * on the left).  The ends are fp32 values, so the step is taken in fp32.
 * Reading where the paper is silent: a bracket that is empty or open on the
 * other side has no width to double; the temperature t stands in for it.  Returns 0, or 1 when no finite widened bracket exists.
 */
int oracle_widen(float a_L, float a_R, double t, int status, float *new_L, float *new_R)
{
    int both = a_L > -INFINITY && a_R < INFINITY;
    float w = both ? a_R - a_L : 0.0f;
    if (!(w > 0.0f)) w = (float)t;
    float two_w = 2.0f * w;
    if (status == ORACLE_ROOT_RIGHT) {
        if (!(a_R < INFINITY)) return 1;
        *new_L = a_R;
        *new_R = a_R + two_w;
    } else {
        if (!(a_L > -INFINITY)) return 1;
        *new_R = a_L;
        *new_L = a_L - two_w;
    }
    return (*new_L < *new_R) ? 0 : 1;
}

/*
 * The validated bracket path as a whole (Sec. 4 "validated path", App. C):
 * solve inside [a_L, a_R); when the certificate fails, widen on the failing
 * side and stream again, at most max_widen times; after that the trivial
 * global bounds, that is the full sort, give the threshold.
 * info[0] = widenings done, info[1] = 1 if the full sort was needed;
 * ends[0..1] = the last bracket tried; counts/tails as oracle_forward_bracketed
 * for that last bracket.
 */
int oracle_forward_validated(const float *r, int64_t n, double k, double alpha, float a_L, float a_R,
                             int max_widen, double *p, double *b, int64_t *info, float *ends,
                             int64_t *counts, double *tails)
{
    if (!info || !ends || max_widen < 0) return ORACLE_EARG;
    int status = 0;
    info[0] = 0;
    info[1] = 0;
    for (int attempt = 0;; ++attempt) {
        ends[0] = a_L;
        ends[1] = a_R;
        int rc = oracle_forward_bracketed(r, n, k, alpha, a_L, a_R, p, b, &status, counts, tails, NULL, 0);
        if (rc) return rc;
        if (status == 0) return ORACLE_OK;
        float nl, nr;
        if (attempt >= max_widen || oracle_widen(a_L, a_R, -alpha, status, &nl, &nr)) break;
        a_L = nl;
        a_R = nr;
        info[0] += 1;
    }
    info[1] = 1;
    return oracle_forward(r, 1, n, k, alpha, p, b, NULL, NULL);
}
