/*
 * attention_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of "standard attention" as the paper defines
 * it in Section 5.1 (the naive chain of matrix operations
 * Softmax(Q K^T / sqrt(d)) V, with no operator fusion and no online softmax),
 * with the lower-triangular attention_mask of Section 4.1 and the decode-stage
 * form of Appendix C (one query row per sequence over the cached K and V).
 * The fused, tiled method of Section 4.1 / Appendix A is stated there to keep
 * the same output, so this definition is what the CUDA library is compared to.
 *
 * Only tests/, the smoke check and the benchmark's cpu_baseline leg may call
 * this file. It shares no code, header, table or helper with the CUDA path.
 *
 * Every function is pinned by tests that do not go through this file's own
 * formulas (closed forms, brute force in another arithmetic, invariants,
 * library special cases): nothing here is "parity unpinned".
 *
 * Conventions (all buffers are HOST memory, owned by the caller):
 *   q            element (b, i, h, t) at  b*q_sb + i*q_ss + h*q_sh + t
 *   k, v         element (b, j, hk, t) at b*k_sb + j*k_ss + hk*k_sh + t
 *   strides are in ELEMENTS; the head dimension d is contiguous.
 *   dtype        0 = IEEE binary16 bits, 1 = bfloat16 bits, 2 = float, 3 = double
 *   kv head of query head h is  h / (Hq / Hkv)   (consecutive grouping)
 *   causal       row i sees key j  iff  j <= i + (Skv - Sq)   (bottom-right
 *                aligned; equals the lower-triangular mask when Sq == Skv)
 *   a row that sees no key gives O = 0 and LSE = -inf
 *   LSE          natural log of the sum of exp(scaled scores) over visible keys
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { DT_F16 = 0, DT_BF16 = 1, DT_F32 = 2, DT_F64 = 3 };

/* Exact widening of one stored element to double. */
static double half_bits_to_double(uint16_t hbits)
{
    int sign = (hbits >> 15) & 1;
    int e = (hbits >> 10) & 0x1f;
    int frac = hbits & 0x3ff;
    double val;
    if (e == 0)
        val = ldexp((double)frac, -24); /* subnormal: frac * 2^-10 * 2^-14 */
    else if (e == 31)
        val = frac ? NAN : INFINITY;
    else
        val = ldexp(1.0 + (double)frac / 1024.0, e - 15);
    return sign ? -val : val;
}

static double bf16_bits_to_double(uint16_t bbits)
{
    uint32_t w = (uint32_t)bbits << 16; /* bfloat16 is the top half of a float */
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

static double load_elem(const void *base, int64_t idx, int dtype)
{
    switch (dtype) {
    case DT_F16: return half_bits_to_double(((const uint16_t *)base)[idx]);
    case DT_BF16: return bf16_bits_to_double(((const uint16_t *)base)[idx]);
    case DT_F32: return (double)((const float *)base)[idx];
    default: return ((const double *)base)[idx];
    }
}

typedef struct {
    const void *q, *k, *v;
    int dtype;
    int B, Hq, Hkv, Sq, Skv, d;
    int causal;
    double scale;
    int64_t q_sb, q_ss, q_sh;
    int64_t k_sb, k_ss, k_sh;
    int64_t v_sb, v_ss, v_sh;
} problem_t;

/* Number of keys row i may see out of the first skv keys (Section 4.1: the
 * attention_mask is lower triangular; aligned to the last key when Sq != Skv). */
static int64_t visible_keys(int causal, int64_t i, int64_t sq, int64_t skv)
{
    if (!causal) return skv;
    int64_t n = i + (skv - sq) + 1;
    if (n < 0) n = 0;
    if (n > skv) n = skv;
    return n;
}

/* One row of standard attention over the first skv_b keys of batch b.
 * s_row and p_row are scratch of length >= skv_b: the full row of scores S and
 * of probabilities P is written out, then P is multiplied into V. */
static void attention_row(const problem_t *pb, int b, int h, int64_t i, int64_t sq_b,
                          int64_t skv_b, double *s_row, double *p_row, double *o_row,
                          double *lse)
{
    const int d = pb->d;
    const int hk = h / (pb->Hq / pb->Hkv);
    const int64_t qoff = (int64_t)b * pb->q_sb + i * pb->q_ss + (int64_t)h * pb->q_sh;
    const int64_t nvis = visible_keys(pb->causal, i, sq_b, skv_b);

    for (int t = 0; t < d; ++t) o_row[t] = 0.0;
    if (nvis == 0) {
        *lse = -INFINITY;
        return;
    }
    /* S = scale * q . k_j for every key; masked entries are -inf */
    for (int64_t j = 0; j < skv_b; ++j) {
        if (j >= nvis) {
            s_row[j] = -INFINITY;
            continue;
        }
        const int64_t koff = (int64_t)b * pb->k_sb + j * pb->k_ss + (int64_t)hk * pb->k_sh;
        double acc = 0.0;
        for (int t = 0; t < d; ++t)
            acc += load_elem(pb->q, qoff + t, pb->dtype) * load_elem(pb->k, koff + t, pb->dtype);
        s_row[j] = pb->scale * acc;
    }
    /* softmax over the row */
    double m = -INFINITY;
    for (int64_t j = 0; j < skv_b; ++j)
        if (s_row[j] > m) m = s_row[j];
    double l = 0.0;
    for (int64_t j = 0; j < skv_b; ++j) {
        p_row[j] = exp(s_row[j] - m); /* exp(-inf) = 0 for masked keys */
        l += p_row[j];
    }
    for (int64_t j = 0; j < skv_b; ++j) p_row[j] /= l;
    /* O = P V */
    for (int64_t j = 0; j < nvis; ++j) {
        const int64_t voff = (int64_t)b * pb->v_sb + j * pb->v_ss + (int64_t)hk * pb->v_sh;
        const double p = p_row[j];
        for (int t = 0; t < d; ++t) o_row[t] += p * load_elem(pb->v, voff + t, pb->dtype);
    }
    *lse = m + log(l);
}

static int check_problem(const problem_t *pb)
{
    if (!pb->q || !pb->k || !pb->v) return -1;
    if (pb->B < 0 || pb->Hq <= 0 || pb->Hkv <= 0 || pb->Sq < 0 || pb->Skv < 0 || pb->d <= 0)
        return -2;
    if (pb->Hq % pb->Hkv) return -2;
    if (pb->dtype < 0 || pb->dtype > 3) return -3;
    return 0;
}

/*
 * Full problem. O is [B, Sq, Hq, d] doubles, LSE is [B, Hq, Sq] doubles.
 * For each (b, h) the whole Sq x Skv score matrix S and probability matrix P
 * exist in memory at once (Section 5.1: no fusion, no online softmax).
 */
int oracle_attention_full(const void *q, const void *k, const void *v, int dtype, int B,
                          int Hq, int Hkv, int Sq, int Skv, int d, int causal, double scale,
                          const int64_t *strides9, double *O, double *LSE, int nthreads)
{
    problem_t pb = {q, k, v, dtype, B, Hq, Hkv, Sq, Skv, d, causal, scale,
                    strides9[0], strides9[1], strides9[2], strides9[3], strides9[4],
                    strides9[5], strides9[6], strides9[7], strides9[8]};
    int rc = check_problem(&pb);
    if (rc) return rc;
    if (!O || !LSE) return -1;
    if (B == 0 || Sq == 0) return 0;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq;
        const size_t n = (size_t)Sq * (size_t)(Skv > 0 ? Skv : 1);
        double *S = (double *)malloc(n * sizeof(double));
        double *P = (double *)malloc(n * sizeof(double));
        if (!S || !P) {
            failed = 1;
            free(S);
            free(P);
            continue;
        }
        for (int64_t i = 0; i < Sq; ++i) {
            double *o_row = O + (((int64_t)b * Sq + i) * Hq + h) * d;
            attention_row(&pb, b, h, i, Sq, Skv, S + i * (int64_t)Skv, P + i * (int64_t)Skv,
                          o_row, &LSE[((int64_t)b * Hq + h) * Sq + i]);
        }
        free(S);
        free(P);
    }
    return failed ? -4 : 0;
}

/*
 * Row-sampled mode: the same per-row computation for n chosen rows.
 * rows is [n, 3] int32 = (b, h, i). O is [n, d], LSE is [n].
 */
int oracle_attention_rows(const void *q, const void *k, const void *v, int dtype, int B,
                          int Hq, int Hkv, int Sq, int Skv, int d, int causal, double scale,
                          const int64_t *strides9, const int32_t *rows, int n, double *O,
                          double *LSE, int nthreads)
{
    problem_t pb = {q, k, v, dtype, B, Hq, Hkv, Sq, Skv, d, causal, scale,
                    strides9[0], strides9[1], strides9[2], strides9[3], strides9[4],
                    strides9[5], strides9[6], strides9[7], strides9[8]};
    int rc = check_problem(&pb);
    if (rc) return rc;
    if (n < 0 || (n > 0 && (!rows || !O || !LSE))) return -1;
    for (int r = 0; r < n; ++r) {
        const int32_t *t = rows + 3 * (int64_t)r;
        if (t[0] < 0 || t[0] >= B || t[1] < 0 || t[1] >= Hq || t[2] < 0 || t[2] >= Sq) return -2;
    }
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
#pragma omp parallel
    {
        const size_t len = (size_t)(Skv > 0 ? Skv : 1);
        double *s_row = (double *)malloc(len * sizeof(double));
        double *p_row = (double *)malloc(len * sizeof(double));
        if (!s_row || !p_row) failed = 1;
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n; ++r) {
            if (!s_row || !p_row) continue;
            const int32_t *t = rows + 3 * (int64_t)r;
            attention_row(&pb, t[0], t[1], t[2], Sq, Skv, s_row, p_row, O + (int64_t)r * d,
                          &LSE[r]);
        }
        free(s_row);
        free(p_row);
    }
    return failed ? -4 : 0;
}

/*
 * Decode stage (Appendix C): one query row per sequence, attending to the first
 * seqlens[b] rows of that sequence's K/V cache, no mask inside that prefix.
 * q is [B, 1, Hq, d] (q_ss unused), caches are [B, Smax, Hkv, d] through the strides.
 * O is [B, Hq, d], LSE is [B, Hq]. A sequence of length 0 gives O = 0, LSE = -inf.
 */
int oracle_decode(const void *q, const void *k_cache, const void *v_cache, int dtype,
                  const int32_t *seqlens, int B, int Hq, int Hkv, int Smax, int d,
                  double scale, const int64_t *strides9, double *O, double *LSE, int nthreads)
{
    problem_t pb = {q, k_cache, v_cache, dtype, B, Hq, Hkv, 1, Smax, d, 0, scale,
                    strides9[0], strides9[1], strides9[2], strides9[3], strides9[4],
                    strides9[5], strides9[6], strides9[7], strides9[8]};
    int rc = check_problem(&pb);
    if (rc) return rc;
    if (!seqlens || !O || !LSE) return -1;
    for (int b = 0; b < B; ++b)
        if (seqlens[b] < 0 || seqlens[b] > Smax) return -2;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
#pragma omp parallel
    {
        const size_t len = (size_t)(Smax > 0 ? Smax : 1);
        double *s_row = (double *)malloc(len * sizeof(double));
        double *p_row = (double *)malloc(len * sizeof(double));
        if (!s_row || !p_row) failed = 1;
#pragma omp for schedule(dynamic, 1)
        for (int bh = 0; bh < B * Hq; ++bh) {
            if (!s_row || !p_row) continue;
            const int b = bh / Hq, h = bh % Hq;
            attention_row(&pb, b, h, 0, 1, seqlens[b], s_row, p_row,
                          O + ((int64_t)b * Hq + h) * d, &LSE[(int64_t)b * Hq + h]);
        }
        free(s_row);
        free(p_row);
    }
    return failed ? -4 : 0;
}

/*
 * A second, structurally different routine used only to pin the ones above on
 * tiny inputs: extended precision, no max subtraction, the softmax written as
 * exp(s_j) / sum_j exp(s_j) directly, visibility tested per element from the
 * mask inequality. Contiguous [B,S,H,d] double inputs. Only valid while
 * exp(score) stays far from overflow.
 */
int oracle_bruteforce(const double *q, const double *k, const double *v, int B, int Hq,
                      int Hkv, int Sq, int Skv, int d, int causal, double scale, double *O,
                      double *LSE)
{
    if (!q || !k || !v || !O || !LSE) return -1;
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv || d <= 0) return -2;
    const int g = Hq / Hkv;
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < Sq; ++i)
            for (int h = 0; h < Hq; ++h) {
                const int hk = h / g;
                long double denom = 0.0L;
                long double num[64];
                if (d > 64) return -2;
                for (int t = 0; t < d; ++t) num[t] = 0.0L;
                for (int j = 0; j < Skv; ++j) {
                    if (causal && j > i + (Skv - Sq)) continue;
                    long double s = 0.0L;
                    for (int t = 0; t < d; ++t)
                        s += (long double)q[(((int64_t)b * Sq + i) * Hq + h) * d + t] *
                             (long double)k[(((int64_t)b * Skv + j) * Hkv + hk) * d + t];
                    long double e = expl((long double)scale * s);
                    denom += e;
                    for (int t = 0; t < d; ++t)
                        num[t] += e * (long double)v[(((int64_t)b * Skv + j) * Hkv + hk) * d + t];
                }
                double *o_row = O + (((int64_t)b * Sq + i) * Hq + h) * d;
                for (int t = 0; t < d; ++t)
                    o_row[t] = denom > 0.0L ? (double)(num[t] / denom) : 0.0;
                LSE[((int64_t)b * Hq + h) * Sq + i] =
                    denom > 0.0L ? (double)logl(denom) : -INFINITY;
            }
    return 0;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
