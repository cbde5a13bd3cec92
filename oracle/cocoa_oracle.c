/*
 * CPU oracle for one CoCoA round with a local stochastic (dual) coordinate-descent solver.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain reference that the GPU library is checked
 * against. It shares no code with the CUDA path, is never used as a fallback, and may only be built
 * and called by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * What it follows (paper sections):
 *   - Sec. 2.2, Eq. 1 and Eq. 2: an iteration refines the shared model from K local updates that are
 *     computed independently on K disjoint partitions and then combined.
 *   - Sec. 2.2 (worker structure, Fig. 2): each worker takes H sequential steps of L samples and updates
 *     its local model after every step, so later steps see earlier ones.
 *   - Sec. 2.2 "CoCoA": L = 1, the local optimiser is SCD over the partition, K is the data parallelism.
 *   - Sec. 5.1 "CoCoA": SVM trained with SCD, H = number of local samples, sigma = number of tasks.
 *   - Sec. 4.1 / Sec. 5 (metrics): the duality gap is the convergence metric.
 * The paper prints no formulas for CoCoA/SCD; the arithmetic below is the standard CoCoA+ "adding"
 * formulation for the objective
 *       P(w) = (1/n) sum_i loss_i(x_i . w) + (lambda/2) |w|^2 ,     w(alpha) = v / (lambda n),  v = X^T alpha
 * (dual losses), and the primal-mapped form for ridge regression over feature partitions.
 *
 * Everything floating point is fp64 on the caller's fp32 inputs. One partition is processed by one
 * thread from start to end; partitions share nothing inside a round, so the result does not depend on
 * the number of threads.
 *
 * Parity pins (tests/test_oracle_pins.py): mix64 against the published SplitMix64 outputs; partition and
 * permutation against their defining properties; hinge against a brute-force QP; ridge against the normal
 * equations; logistic against bisection and a Newton solve of the primal; K=1 against a separately written
 * SDCA loop; orthogonal rows against the closed form; the sigma' factor of the local model by a K = 2,
 * sigma' = 2 case worked by hand and by every step maximising its task's explicitly evaluated sigma'-subproblem
 * along its coordinate; Fenchel-Young non-negativity; v == X^T alpha; dual ascent; weak duality across
 * rounds; repartition invariance. Parity with the paper's own (unreleased) implementation and its
 * random streams: parity unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_HINGE = 0, ORC_LOGISTIC = 1, ORC_RIDGE = 2 };

/* ---- integer part: mixer, partition, permutation -------------------------------------------------- */

/* One SplitMix64 output for state x (Steele, Lea, Flood 2014): add the golden-ratio increment, then the
 * three-stage xor-shift-multiply finaliser. A bijection on 64-bit words. */
uint64_t orc_mix64(uint64_t x)
{
    uint64_t z = x + 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* Odd constant that separates the permutation stream from the partition stream. */
#define ORC_PERM_STREAM 0xD1B54A32D192ED03ULL

typedef struct { uint64_t key; int32_t id; } orc_pair;

static int orc_pair_cmp(const void *pa, const void *pb)
{
    const orc_pair *a = (const orc_pair *)pa, *b = (const orc_pair *)pb;
    if (a->key != b->key) return a->key < b->key ? -1 : 1;
    if (a->id != b->id) return a->id < b->id ? -1 : 1;
    return 0;
}

static int orc_i32_cmp(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/* Random equal split of coordinates 0..n-1 into K disjoint covering partitions (Sec. 2.2: disjoint
 * partitions D_k; Appendix, baseline comparisons: random assignment of data to tasks). Sort ids by (mix64(mix64(seed) ^ id), id),
 * cut the sorted list into K consecutive blocks, the first n mod K blocks one longer; inside a partition
 * the members are listed in ascending id.  Returns 0, or -1 on bad arguments / out of memory. */
static int orc_partition_cut(int64_t n, int32_t K, uint64_t seed, const int64_t *sizes, int32_t *owner, int64_t *part_off,
                             int32_t *members);

int orc_partition(int64_t n, int32_t K, uint64_t seed, int32_t *owner, int64_t *part_off, int32_t *members)
{
    return orc_partition_cut(n, K, seed, NULL, owner, part_off, members);
}

/* The same random order of the coordinates cut into K consecutive blocks of the given sizes (each >= 1, summing to
 * n): tasks may hold different numbers of samples (Sec. 3, load balancing: data is moved from slow to fast tasks;
 * Sec. 4.5, rebalancing policy). Returns 0, or -1 on bad arguments / out of memory. */
int orc_partition_sizes(int64_t n, int32_t K, uint64_t seed, const int64_t *sizes, int32_t *owner, int64_t *part_off,
                        int32_t *members)
{
    if (!sizes) return -1;
    return orc_partition_cut(n, K, seed, sizes, owner, part_off, members);
}

static int orc_partition_cut(int64_t n, int32_t K, uint64_t seed, const int64_t *sizes, int32_t *owner, int64_t *part_off,
                             int32_t *members)
{
    if (n <= 0 || K <= 0 || (int64_t)K > n) return -1;
    if (sizes) {
        int64_t tot = 0;
        for (int32_t k = 0; k < K; ++k) {
            if (sizes[k] < 1) return -1;
            tot += sizes[k];
        }
        if (tot != n) return -1;
    }
    orc_pair *p = (orc_pair *)malloc((size_t)n * sizeof(orc_pair));
    if (!p) return -1;
    const uint64_t s = orc_mix64(seed);
    for (int64_t i = 0; i < n; ++i) { p[i].key = orc_mix64(s ^ (uint64_t)i); p[i].id = (int32_t)i; }
    qsort(p, (size_t)n, sizeof(orc_pair), orc_pair_cmp);
    const int64_t base = n / K, extra = n % K;
    part_off[0] = 0;
    for (int32_t k = 1; k <= K; ++k)
        part_off[k] = sizes ? part_off[k - 1] + sizes[k - 1] : (int64_t)k * base + (k < extra ? k : extra);
    for (int32_t k = 0; k < K; ++k) {
        for (int64_t pos = part_off[k]; pos < part_off[k + 1]; ++pos) {
            owner[p[pos].id] = k;
            members[pos] = p[pos].id;
        }
        qsort(members + part_off[k], (size_t)(part_off[k + 1] - part_off[k]), sizeof(int32_t), orc_i32_cmp);
    }
    free(p);
    return 0;
}

/* Visiting order of one partition in local epoch `epoch` of round `round` (Sec. 5.1: H = local sample
 * count, read as sampling without replacement): members sorted by
 * (mix64(mix64(seed ^ STREAM) ^ mix64(round * 2^32 + epoch) ^ id), id). */
int orc_permutation(const int32_t *members_k, int64_t n_k, uint64_t seed, int64_t round, int64_t epoch,
                    int32_t *out)
{
    if (n_k < 0) return -1;
    if (n_k == 0) return 0;
    orc_pair *p = (orc_pair *)malloc((size_t)n_k * sizeof(orc_pair));
    if (!p) return -1;
    const uint64_t a = orc_mix64(seed ^ ORC_PERM_STREAM);
    const uint64_t b = orc_mix64(((uint64_t)round << 32) + (uint64_t)epoch);
    for (int64_t j = 0; j < n_k; ++j) {
        p[j].id = members_k[j];
        p[j].key = orc_mix64(a ^ b ^ (uint64_t)(uint32_t)members_k[j]);
    }
    qsort(p, (size_t)n_k, sizeof(orc_pair), orc_pair_cmp);
    for (int64_t j = 0; j < n_k; ++j) out[j] = p[j].id;
    free(p);
    return 0;
}

/* ---- coordinate vectors --------------------------------------------------------------------------- */

/* The matrix is stored coordinate-major: coordinate c (an example for the dual losses, a feature for
 * ridge) owns either the compressed slice indptr[c]..indptr[c+1] of (indices, values), or, when indptr
 * is NULL, the dense slice values[c*ld .. c*ld+dim). */
typedef struct {
    int64_t n_coord, dim, ld;
    const int64_t *indptr;
    const int32_t *indices;
    const float *values;
} orc_mat;

static double orc_dot(const orc_mat *A, int64_t c, const double *vec)
{
    double s = 0.0;
    if (A->indptr) {
        for (int64_t e = A->indptr[c]; e < A->indptr[c + 1]; ++e) s += (double)A->values[e] * vec[A->indices[e]];
    } else {
        const float *row = A->values + c * A->ld;
        for (int64_t j = 0; j < A->dim; ++j) s += (double)row[j] * vec[j];
    }
    return s;
}

static double orc_sqnorm(const orc_mat *A, int64_t c)
{
    double s = 0.0;
    if (A->indptr) {
        for (int64_t e = A->indptr[c]; e < A->indptr[c + 1]; ++e) s += (double)A->values[e] * (double)A->values[e];
    } else {
        const float *row = A->values + c * A->ld;
        for (int64_t j = 0; j < A->dim; ++j) s += (double)row[j] * (double)row[j];
    }
    return s;
}

static void orc_axpy(const orc_mat *A, int64_t c, double t, double *vec)
{
    if (A->indptr) {
        for (int64_t e = A->indptr[c]; e < A->indptr[c + 1]; ++e) vec[A->indices[e]] += t * (double)A->values[e];
    } else {
        const float *row = A->values + c * A->ld;
        for (int64_t j = 0; j < A->dim; ++j) vec[j] += t * (double)row[j];
    }
}

/* ---- scalar steps --------------------------------------------------------------------------------- */

static double orc_sigmoid(double z)
{
    if (z >= 0.0) return 1.0 / (1.0 + exp(-z));
    double e = exp(z);
    return e / (1.0 + e);
}

/* Hinge: maximise  a' - (a'-a) m - (q/2)(a'-a)^2  over a' in [0,1]. */
double orc_step_hinge(double a, double m, double q)
{
    if (q <= 0.0) return 1.0;            /* zero row: the objective is linear and increasing in a' */
    double t = a + (1.0 - m) / q;
    return t < 0.0 ? 0.0 : (t > 1.0 ? 1.0 : t);
}

/* Logistic: maximise  -[a' log a' + (1-a') log(1-a')] - (a'-a) m - (q/2)(a'-a)^2  over a' in (0,1).
 * With a' = sigmoid(z) the stationarity condition is  F(z) = z + q sigmoid(z) - c = 0,  c = q a - m.
 * F is continuous and strictly increasing (F' = 1 + q p (1-p) >= 1), and since 0 <= sigmoid <= 1 the unique
 * root lies in [c - q, c]. It is found the plain way: a bracket [lo, hi] with F(lo) <= 0 <= F(hi) that every
 * evaluation narrows; the next point is Newton's when that falls strictly inside the bracket and the steps are
 * at least halving, else the midpoint (the textbook safeguarded Newton iteration); stop when |F| <= 1e-12 or the bracket has no interior point in fp64 (for |c| of 1e4 and more the
 * spacing of doubles near the root is itself above 1e-12). q = 0 (zero row) gives a' = sigmoid(-m) exactly.
 * The residual F at the returned point is written to *resid when resid != NULL. */
double orc_step_logistic(double a, double m, double q, double *resid)
{
    const double c = q * a - m;
    double lo = c - q, hi = c;              /* F(lo) <= 0 <= F(hi) */
    double z = 0.5 * (lo + hi);
    double step_before = hi - lo, step = step_before;
    for (int it = 0; it < 400; ++it) {
        const double p = orc_sigmoid(z);
        const double F = z + q * p - c;
        if (fabs(F) <= 1e-12) break;
        if (F > 0.0) hi = z; else lo = z;
        const double Fp = 1.0 + q * p * (1.0 - p);
        const double zn = z - F / Fp;
        /* Newton's point if it lies inside the bracket and the steps are at least halving, else the midpoint */
        if (zn > lo && zn < hi && fabs(2.0 * F) <= fabs(step_before * Fp)) {
            step_before = step;
            step = F / Fp;
            z = zn;
        } else {
            step_before = step;
            step = 0.5 * (hi - lo);
            const double mid = lo + step;
            if (!(mid > lo && mid < hi)) break;   /* lo and hi are neighbouring doubles */
            z = mid;
        }
    }
    const double p = orc_sigmoid(z);
    if (resid) *resid = z + q * p - c;
    return p;
}

static double orc_xlogx(double x) { return x > 0.0 ? x * log(x) : 0.0; }

static double orc_softplus(double t) /* log(1 + e^t) */
{
    return t > 0.0 ? t + log1p(exp(-t)) : log1p(exp(t));
}

/* ---- one CoCoA round ------------------------------------------------------------------------------ */

/* Runs the local solver of partition k for `steps` coordinate steps against vloc (a private copy of the
 * shared vector) and accumulates the partition's update in dv. state[] is alpha (signed dual variables)
 * for the dual losses and w for ridge; labels[] is y per coordinate for the dual losses and the target
 * vector (length dim) for ridge. `scale_n` is the number of examples n in the objective. */
static int orc_local_solver(int loss, const orc_mat *A, const float *labels, double lambda, double scale_n,
                            double *state, const int32_t *members_k, int64_t n_k, uint64_t seed, int64_t round,
                            int64_t steps, double sigma_p, double *vloc, double *dv, double *max_resid)
{
    int32_t *perm = (int32_t *)malloc((size_t)(n_k > 0 ? n_k : 1) * sizeof(int32_t));
    if (!perm) return -1;
    const double lam_n = lambda * scale_n;
    int64_t epoch = -1;
    for (int64_t t = 0; t < steps; ++t) {
        const int64_t e = t / n_k, pos = t % n_k;
        if (e != epoch) {
            epoch = e;
            if (orc_permutation(members_k, n_k, seed, round, epoch, perm) != 0) { free(perm); return -1; }
        }
        const int64_t c = perm[pos];
        const double s = orc_sqnorm(A, c);
        double delta;
        if (loss == ORC_RIDGE) {
            /* vloc holds X w_local; gradient of (1/2n)|v - y|^2 along column c, plus the l2 term */
            double g = 0.0;
            if (A->indptr) {
                for (int64_t q = A->indptr[c]; q < A->indptr[c + 1]; ++q) {
                    const int32_t r = A->indices[q];
                    g += (double)A->values[q] * (vloc[r] - (double)labels[r]);
                }
            } else {
                const float *col = A->values + c * A->ld;
                for (int64_t r = 0; r < A->dim; ++r) g += (double)col[r] * (vloc[r] - (double)labels[r]);
            }
            g = g / scale_n + lambda * state[c];
            delta = -g / (sigma_p * s / scale_n + lambda);
        } else {
            const double y = (double)labels[c];
            const double m = y * orc_dot(A, c, vloc) / lam_n;
            const double q = sigma_p * s / lam_n;
            const double a = y * state[c];
            double a_new;
            if (loss == ORC_HINGE) {
                a_new = orc_step_hinge(a, m, q);
            } else {
                double r = 0.0;
                a_new = orc_step_logistic(a, m, q, &r);
                if (fabs(r) > *max_resid) *max_resid = fabs(r);
            }
            delta = y * (a_new - a);
        }
        state[c] += delta;
        orc_axpy(A, c, delta, dv);
        orc_axpy(A, c, sigma_p * delta, vloc);
    }
    free(perm);
    return 0;
}

/* One round (Eq. 1 + Eq. 2 with the updates added, gamma = 1): every partition solves locally from the
 * same v, then v += sum_k dv_k with k ascending.  H = 0 means one local epoch (n_k steps).
 * newton_resid (nullable) receives the largest |g| left by a logistic step in this round.
 * Returns 0 on success, -1 on bad arguments or allocation failure. */
static int orc_round_impl(int loss, int64_t n_coord, int64_t dim, const int64_t *indptr, const int32_t *indices,
                          const float *values, int64_t ld, const float *labels, double lambda,
                          double *state, double *v, int32_t K, const int64_t *part_off, const int32_t *members,
                          uint64_t seed, int64_t round, int64_t H, const int64_t *steps_k, double sigma_p, int nthreads,
                          double *newton_resid);

int orc_round(int loss, int64_t n_coord, int64_t dim, const int64_t *indptr, const int32_t *indices,
              const float *values, int64_t ld, const float *labels, double lambda,
              double *state, double *v, int32_t K, const int64_t *part_off, const int32_t *members,
              uint64_t seed, int64_t round, int64_t H, double sigma_p, int nthreads, double *newton_resid)
{
    return orc_round_impl(loss, n_coord, dim, indptr, indices, values, ld, labels, lambda, state, v, K, part_off, members,
                          seed, round, H, NULL, sigma_p, nthreads, newton_resid);
}

/* The same round with a step budget of its own for every partition (Sec. 3, load balancing: a task processes a
 * number of samples per iteration that suits its speed): partition k takes steps_k[k] >= 0 coordinate steps of its
 * visiting order (0: it sits the round out). */
int orc_round_steps(int loss, int64_t n_coord, int64_t dim, const int64_t *indptr, const int32_t *indices,
                    const float *values, int64_t ld, const float *labels, double lambda,
                    double *state, double *v, int32_t K, const int64_t *part_off, const int32_t *members,
                    uint64_t seed, int64_t round, const int64_t *steps_k, double sigma_p, int nthreads, double *newton_resid)
{
    if (!steps_k) return -1;
    for (int32_t k = 0; k < K; ++k)
        if (steps_k[k] < 0) return -1;
    return orc_round_impl(loss, n_coord, dim, indptr, indices, values, ld, labels, lambda, state, v, K, part_off, members,
                          seed, round, 0, steps_k, sigma_p, nthreads, newton_resid);
}

static int orc_round_impl(int loss, int64_t n_coord, int64_t dim, const int64_t *indptr, const int32_t *indices,
                          const float *values, int64_t ld, const float *labels, double lambda,
                          double *state, double *v, int32_t K, const int64_t *part_off, const int32_t *members,
                          uint64_t seed, int64_t round, int64_t H, const int64_t *steps_k, double sigma_p, int nthreads,
                          double *newton_resid)
{
    if (K <= 0 || n_coord <= 0 || dim <= 0 || lambda <= 0.0 || sigma_p <= 0.0 || H < 0) return -1;
    orc_mat A = { n_coord, dim, ld, indptr, indices, values };
    const double scale_n = (loss == ORC_RIDGE) ? (double)dim : (double)n_coord;
    double *dv_all = (double *)calloc((size_t)K * (size_t)dim, sizeof(double));
    double *resid_k = (double *)calloc((size_t)K, sizeof(double));
    int *rc_k = (int *)calloc((size_t)K, sizeof(int));
    if (!dv_all || !resid_k || !rc_k) { free(dv_all); free(resid_k); free(rc_k); return -1; }
    if (nthreads < 1) nthreads = 1;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(nthreads)
#endif
    for (int32_t k = 0; k < K; ++k) {
        const int64_t n_k = part_off[k + 1] - part_off[k];
        if (n_k <= 0) continue;
        double *vloc = (double *)malloc((size_t)dim * sizeof(double));
        if (!vloc) { rc_k[k] = -1; continue; }
        memcpy(vloc, v, (size_t)dim * sizeof(double));
        const int64_t steps = steps_k ? steps_k[k] : ((H == 0) ? n_k : H);
        if (steps == 0) continue;
        rc_k[k] = orc_local_solver(loss, &A, labels, lambda, scale_n, state, members + part_off[k], n_k, seed,
                                   round, steps, sigma_p, vloc, dv_all + (size_t)k * (size_t)dim, &resid_k[k]);
        free(vloc);
    }
    int rc = 0;
    double worst = 0.0;
    for (int32_t k = 0; k < K; ++k) {
        if (rc_k[k] != 0) rc = -1;
        if (resid_k[k] > worst) worst = resid_k[k];
    }
    if (rc == 0) {
        for (int32_t k = 0; k < K; ++k) {
            const double *dv = dv_all + (size_t)k * (size_t)dim;
            for (int64_t j = 0; j < dim; ++j) v[j] += dv[j];
        }
    }
    if (newton_resid) *newton_resid = worst;
    free(dv_all); free(resid_k); free(rc_k);
    return rc;
}

/* ---- duality gap ---------------------------------------------------------------------------------- */

/* out[0] = gap, out[1] = primal, out[2] = dual, out[3] = smallest per-coordinate Fenchel-Young term
 * (dual losses; 0 for ridge). terms (nullable, length n_coord) receives the per-example gap terms of the
 * dual losses.  Returns 0, or -1 if a dual variable is outside its domain by more than 1e-9. */
int orc_gap(int loss, int64_t n_coord, int64_t dim, const int64_t *indptr, const int32_t *indices,
            const float *values, int64_t ld, const float *labels, double lambda,
            const double *state, const double *v, double *out, double *terms)
{
    orc_mat A = { n_coord, dim, ld, indptr, indices, values };
    if (loss == ORC_RIDGE) {
        const double n = (double)dim;
        double f = 0.0, uu = 0.0, uy = 0.0, ww = 0.0, cc = 0.0;
        double *u = (double *)malloc((size_t)dim * sizeof(double));
        if (!u) return -1;
        for (int64_t r = 0; r < dim; ++r) {
            const double res = v[r] - (double)labels[r];
            u[r] = res / n;
            f += res * res;
            uu += u[r] * u[r];
            uy += u[r] * (double)labels[r];
        }
        for (int64_t c = 0; c < n_coord; ++c) {
            const double t = orc_dot(&A, c, u);
            cc += t * t;
            ww += state[c] * state[c];
        }
        free(u);
        const double primal = f / (2.0 * n) + 0.5 * lambda * ww;
        const double dual = -(0.5 * n * uu + uy) - cc / (2.0 * lambda);
        out[0] = primal - dual; out[1] = primal; out[2] = dual; out[3] = 0.0;
        return 0;
    }
    const double n = (double)n_coord, lam_n = lambda * n;
    double loss_sum = 0.0, gap_sum = 0.0, vv = 0.0, min_term = INFINITY;
    int rc = 0;
    for (int64_t j = 0; j < dim; ++j) vv += v[j] * v[j];
    for (int64_t i = 0; i < n_coord; ++i) {
        const double y = (double)labels[i];
        const double mu = y * orc_dot(&A, i, v) / lam_n;       /* y_i x_i . w */
        double a = y * state[i];
        if (a < -1e-9 || a > 1.0 + 1e-9) rc = -1;
        if (a < 0.0) a = 0.0;
        if (a > 1.0) a = 1.0;
        double l, conj;
        if (loss == ORC_HINGE) {
            l = 1.0 - mu > 0.0 ? 1.0 - mu : 0.0;
            conj = -a;
        } else {
            l = orc_softplus(-mu);
            conj = orc_xlogx(a) + orc_xlogx(1.0 - a);
        }
        const double term = l + conj + a * mu;
        if (terms) terms[i] = term;
        if (term < min_term) min_term = term;
        loss_sum += l;
        gap_sum += term;
    }
    const double primal = loss_sum / n + 0.5 * lambda * vv / (lam_n * lam_n);
    const double gap = gap_sum / n;
    out[0] = gap; out[1] = primal; out[2] = primal - gap; out[3] = min_term;
    return rc;
}

/* v = X^T alpha (dual) or X w (ridge) from scratch, fp64. */
void orc_shared_vector(int64_t n_coord, int64_t dim, const int64_t *indptr, const int32_t *indices,
                       const float *values, int64_t ld, const double *state, double *v)
{
    orc_mat A = { n_coord, dim, ld, indptr, indices, values };
    for (int64_t j = 0; j < dim; ++j) v[j] = 0.0;
    for (int64_t c = 0; c < n_coord; ++c) orc_axpy(&A, c, state[c], v);
}
