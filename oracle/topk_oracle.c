/*
 * CPU oracle for the per-step compression pipeline of bidirectional top_K SGD
 * (arXiv 2209.15203).  TEST INFRASTRUCTURE ONLY: this file exists so that the
 * CUDA library can be checked against something plain and slow.  It shares no
 * code, header, table or helper with the CUDA path and must never be called
 * from it.  Every function here is pinned by tests that do not use the oracle
 * to check itself (brute-force rank counting, closed forms, the contraction
 * bound of Eq. "topk_bound", a hand-computed iteration of Algorithm 2).
 *
 * What it computes, and where the paper says so:
 *
 *   Top_K(x)    keep the K components of largest magnitude, zero the rest
 *               (Section 1, definition of top_K sparsification; Assumption 3.2).
 *               Here written out literally as a full STABLE sort of all d
 *               components by magnitude, descending; stability makes equal
 *               magnitudes keep ascending index order, so the lower index wins
 *               a tie (the paper does not fix a tie rule; this is the reading
 *               the library documents).  The message is then listed in
 *               ascending index order with the original signed values.
 *
 *   aggregate   g = sum_{q=1..N} p_q Top_K(a^q)  (Algorithm 1, server step;
 *               Algorithm 2, server step with delta_0 = 0), accumulated in
 *               worker order q = 1..N starting from +0, one rounded fp32
 *               multiply and one rounded fp32 add per term.
 *
 *   downlink    Top_K(g) (Algorithm 2, server step).  Algorithm 1 sends g
 *               itself.
 *
 *   update      w <- w - alpha * message  (Algorithm 1 / Algorithm 2, last
 *               worker step; the step size multiplies the message instead of
 *               the gradient, which selects the same components because
 *               Top_K is positively homogeneous).
 *
 *   ref_step_ef, at the end of this file, is the iteration exactly as printed,
 *   with the error memories epsilon and delta and the step size inside a^q.
 *
 * Magnitudes are compared through the integer key  bits(x) & 0x7fffffff,
 * which orders finite floats exactly like |x| does, makes -0 equal +0 and keeps
 * denormals distinct.  NaN/Inf are ordered by that bit pattern.
 *
 * Build: gcc -O2 -std=c99 -ffp-contract=off -fno-fast-math -shared -fPIC -pthread
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <pthread.h>
#include <math.h>

typedef struct {
    uint32_t key; /* magnitude key */
    int32_t idx;  /* position in the vector */
} ref_item;

static uint32_t ref_key(float x)
{
    uint32_t b;
    memcpy(&b, &x, sizeof b);
    return b & 0x7fffffffu;
}

/* Stable bottom-up merge sort of items by key, DESCENDING.  On equal keys the
 * left run's item is taken first, so the initial ascending index order is
 * preserved inside every group of equal keys. */
static void ref_stable_sort_desc(ref_item *a, ref_item *tmp, int64_t n)
{
    ref_item *src = a, *dst = tmp;
    for (int64_t width = 1; width < n; width *= 2) {
        for (int64_t lo = 0; lo < n; lo += 2 * width) {
            int64_t mid = lo + width < n ? lo + width : n;
            int64_t hi = lo + 2 * width < n ? lo + 2 * width : n;
            int64_t i = lo, j = mid, k = lo;
            while (i < mid && j < hi) {
                if (src[j].key > src[i].key)
                    dst[k++] = src[j++];
                else
                    dst[k++] = src[i++];
            }
            while (i < mid) dst[k++] = src[i++];
            while (j < hi) dst[k++] = src[j++];
        }
        ref_item *t = src; src = dst; dst = t;
    }
    if (src != a) memcpy(a, src, (size_t)n * sizeof *a);
}

static int ref_cmp_idx(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/* Top_K of one vector.  idx_out[K] ascending, val_out[K] = x[idx] bit for bit.
 * Returns 0, or -1 on bad arguments / out of memory. */
int ref_topk(const float *x, int64_t d, int64_t K, int32_t *idx_out, float *val_out)
{
    if (!x || !idx_out || !val_out || d < 1 || d >= ((int64_t)1 << 31) || K < 1 || K > d)
        return -1;
    ref_item *items = (ref_item *)malloc((size_t)d * sizeof *items);
    ref_item *tmp = (ref_item *)malloc((size_t)d * sizeof *tmp);
    if (!items || !tmp) { free(items); free(tmp); return -1; }
    for (int64_t j = 0; j < d; ++j) {
        items[j].key = ref_key(x[j]);
        items[j].idx = (int32_t)j;
    }
    ref_stable_sort_desc(items, tmp, d);
    for (int64_t k = 0; k < K; ++k) idx_out[k] = items[k].idx;
    qsort(idx_out, (size_t)K, sizeof *idx_out, ref_cmp_idx);
    for (int64_t k = 0; k < K; ++k) val_out[k] = x[idx_out[k]];
    free(items);
    free(tmp);
    return 0;
}

/* ---- rows in parallel: one row is one unit of work, handed out in order ---- */
typedef struct {
    const float *x;
    int64_t rows, d, K;
    int32_t *idx_out;
    float *val_out;
    int64_t next_row;
    int failed;
    pthread_mutex_t mu;
} ref_rows_job;

static void *ref_rows_worker(void *arg)
{
    ref_rows_job *job = (ref_rows_job *)arg;
    for (;;) {
        pthread_mutex_lock(&job->mu);
        int64_t r = job->next_row++;
        pthread_mutex_unlock(&job->mu);
        if (r >= job->rows) break;
        int rc = ref_topk(job->x + r * job->d, job->d, job->K,
                          job->idx_out + r * job->K, job->val_out + r * job->K);
        if (rc != 0) {
            pthread_mutex_lock(&job->mu);
            job->failed = 1;
            pthread_mutex_unlock(&job->mu);
        }
    }
    return NULL;
}

/* Top_K of every row of x[rows][d]; rows are independent (each worker
 * compresses its own vector).  nthreads <= 1 runs them one after another. */
int ref_topk_rows(const float *x, int64_t rows, int64_t d, int64_t K,
                  int32_t *idx_out, float *val_out, int nthreads)
{
    if (rows < 1) return -1;
    ref_rows_job job;
    job.x = x; job.rows = rows; job.d = d; job.K = K;
    job.idx_out = idx_out; job.val_out = val_out;
    job.next_row = 0; job.failed = 0;
    pthread_mutex_init(&job.mu, NULL);
    if (nthreads > rows) nthreads = (int)rows;
    if (nthreads <= 1) {
        ref_rows_worker(&job);
    } else {
        pthread_t *th = (pthread_t *)malloc((size_t)nthreads * sizeof *th);
        if (!th) return -1;
        int started = 0;
        for (int t = 0; t < nthreads; ++t)
            if (pthread_create(&th[t], NULL, ref_rows_worker, &job) == 0) ++started;
        if (started == 0) ref_rows_worker(&job);
        for (int t = 0; t < started; ++t) pthread_join(th[t], NULL);
        free(th);
    }
    pthread_mutex_destroy(&job.mu);
    return job.failed ? -1 : 0;
}

/* Server sum  A[j] = sum_q p_q v_{q,j}  over the N sparse messages, q ascending,
 * from A = +0:  A[j] = fl32(A[j] + fl32(p_q * v)).  touched[j] is set to 1 for
 * every index that appears in some message (the union U; |U| <= N K). */
int ref_aggregate(const int32_t *up_idx, const float *up_val, int64_t N, int64_t K_up,
                  const float *p, int64_t d, float *A, uint8_t *touched)
{
    if (!up_idx || !up_val || !p || !A || !touched) return -1;
    for (int64_t j = 0; j < d; ++j) { A[j] = 0.0f; touched[j] = 0; }
    for (int64_t q = 0; q < N; ++q) {
        for (int64_t k = 0; k < K_up; ++k) {
            int32_t j = up_idx[q * K_up + k];
            if (j < 0 || j >= d) return -1;
            volatile float term = p[q] * up_val[q * K_up + k];
            volatile float sum = A[j] + term;
            A[j] = sum;
            touched[j] = 1;
        }
    }
    return 0;
}

/*
 * One memory-free iteration (Algorithm 2 with epsilon_0 = delta_0 = 0, or
 * Algorithm 1 when mode == 0).
 *
 *   w        [d]      updated in place
 *   G        [N][d]   the workers' vectors, row q = worker q
 *   mode     0 = unidirectional (downlink sends the aggregate itself)
 *            1 = bidirectional  (downlink sends Top_{K_down} of the aggregate)
 * Optional outputs (NULL to skip):
 *   up_idx, up_val   [N][K_up]  the uplink messages
 *   A_out            [d]        the dense aggregate
 *   touched_out      [d]        1 where some worker sent that index
 *   msg_idx, msg_val [cap]      the downlink message, ascending index;
 *                               cap = K_down (bi) or N*K_up (uni)
 *   msg_count                   its length: K_down (bi) or |U| (uni)
 */
int ref_step(float *w, const float *G, int64_t N, int64_t d, int64_t K_up, int64_t K_down,
             const float *p, float alpha, int mode,
             int32_t *up_idx_out, float *up_val_out, float *A_out, uint8_t *touched_out,
             int32_t *msg_idx_out, float *msg_val_out, int64_t *msg_count_out, int nthreads)
{
    if (!w || !G || !p || N < 1 || d < 1 || K_up < 1 || K_up > d || (mode != 0 && mode != 1))
        return -1;
    if (mode == 1 && (K_down < 1 || K_down > d)) return -1;
    int rc = -1;
    int64_t cap = mode == 1 ? K_down : N * K_up;
    if (cap > d) cap = d;
    int32_t *up_idx = (int32_t *)malloc((size_t)(N * K_up) * sizeof *up_idx);
    float *up_val = (float *)malloc((size_t)(N * K_up) * sizeof *up_val);
    float *A = (float *)malloc((size_t)d * sizeof *A);
    uint8_t *touched = (uint8_t *)malloc((size_t)d);
    int32_t *msg_idx = (int32_t *)malloc((size_t)cap * sizeof *msg_idx);
    float *msg_val = (float *)malloc((size_t)cap * sizeof *msg_val);
    int64_t count = 0;
    if (!up_idx || !up_val || !A || !touched || !msg_idx || !msg_val) goto done;

    /* worker side: every worker compresses its own vector */
    if (ref_topk_rows(G, N, d, K_up, up_idx, up_val, nthreads) != 0) goto done;
    /* server side: weighted sum in worker order */
    if (ref_aggregate(up_idx, up_val, N, K_up, p, d, A, touched) != 0) goto done;
    /* downlink message */
    if (mode == 1) {
        if (ref_topk(A, d, K_down, msg_idx, msg_val) != 0) goto done;
        count = K_down;
    } else {
        for (int64_t j = 0; j < d; ++j)
            if (touched[j]) { msg_idx[count] = (int32_t)j; msg_val[count] = A[j]; ++count; }
    }
    /* worker side: apply the message */
    for (int64_t k = 0; k < count; ++k) {
        volatile float upd = alpha * msg_val[k];
        volatile float nw = w[msg_idx[k]] - upd;
        w[msg_idx[k]] = nw;
    }

    if (up_idx_out) memcpy(up_idx_out, up_idx, (size_t)(N * K_up) * sizeof *up_idx);
    if (up_val_out) memcpy(up_val_out, up_val, (size_t)(N * K_up) * sizeof *up_val);
    if (A_out) memcpy(A_out, A, (size_t)d * sizeof *A);
    if (touched_out) memcpy(touched_out, touched, (size_t)d);
    if (msg_idx_out) memcpy(msg_idx_out, msg_idx, (size_t)count * sizeof *msg_idx);
    if (msg_val_out) memcpy(msg_val_out, msg_val, (size_t)count * sizeof *msg_val);
    if (msg_count_out) *msg_count_out = count;
    rc = 0;
done:
    free(up_idx); free(up_val); free(A); free(touched); free(msg_idx); free(msg_val);
    return rc;
}

/*
 * One iteration of Algorithm 1 (mode 0) or Algorithm 2 (mode 1) as printed,
 * with the error memories: epsilon^q per worker, delta on the server.
 *
 *   worker q:  a^q   = epsilon^q + alpha * g^q             (first worker line)
 *              msg^q = Top_K_up(a^q)
 *              epsilon^q <- a^q - msg^q                     (second worker line)
 *   server:    S = sum_q p_q msg^q   in worker order, from +0
 *     mode 0:  g = S;            the downlink carries g;          w <- w - g
 *     mode 1:  g = S + delta;    the downlink carries Top_K_down(g);
 *              delta <- g - Top_K_down(g);                        w <- w - Top_K_down(g)
 *
 * Every operation is one rounded fp32 operation: a = fl(eps + fl(alpha*g)),
 * S as in ref_aggregate, g = fl(S + delta), w = fl(w - msg).  Subtracting the
 * message from a (or g) leaves exactly +0 at the sent positions and the value
 * itself elsewhere.
 *
 *   w [d], eps [N][d], delta [d] (mode 1 only; may be NULL in mode 0): updated in place
 *   G [N][d]
 * Optional outputs as in ref_step: up_idx/up_val [N][K_up]; msg_idx/msg_val/msg_count the
 * downlink message (mode 1: exactly K_down entries; mode 0: the union, ascending).
 */
int ref_step_ef(float *w, float *eps, float *delta, const float *G, int64_t N, int64_t d,
                int64_t K_up, int64_t K_down, const float *p, float alpha, int mode,
                int32_t *up_idx_out, float *up_val_out,
                int32_t *msg_idx_out, float *msg_val_out, int64_t *msg_count_out, int nthreads)
{
    if (!w || !eps || !G || !p || N < 1 || d < 1 || K_up < 1 || K_up > d || (mode != 0 && mode != 1))
        return -1;
    if (mode == 1 && (!delta || K_down < 1 || K_down > d)) return -1;
    int rc = -1;
    int64_t cap = mode == 1 ? K_down : N * K_up;
    if (cap > d) cap = d;
    int32_t *up_idx = (int32_t *)malloc((size_t)(N * K_up) * sizeof *up_idx);
    float *up_val = (float *)malloc((size_t)(N * K_up) * sizeof *up_val);
    float *S = (float *)malloc((size_t)d * sizeof *S);
    uint8_t *touched = (uint8_t *)malloc((size_t)d);
    int32_t *msg_idx = (int32_t *)malloc((size_t)cap * sizeof *msg_idx);
    float *msg_val = (float *)malloc((size_t)cap * sizeof *msg_val);
    int64_t count = 0;
    if (!up_idx || !up_val || !S || !touched || !msg_idx || !msg_val) goto done;

    /* workers: error-compensated value, kept in eps */
    for (int64_t q = 0; q < N; ++q)
        for (int64_t j = 0; j < d; ++j) {
            volatile float scaled = alpha * G[q * d + j];
            volatile float a = eps[q * d + j] + scaled;
            eps[q * d + j] = a;
        }
    if (ref_topk_rows(eps, N, d, K_up, up_idx, up_val, nthreads) != 0) goto done;
    /* eps <- a - Top_K(a) */
    for (int64_t q = 0; q < N; ++q)
        for (int64_t k = 0; k < K_up; ++k) eps[q * d + up_idx[q * K_up + k]] = 0.0f;
    /* server */
    if (ref_aggregate(up_idx, up_val, N, K_up, p, d, S, touched) != 0) goto done;
    if (mode == 1) {
        for (int64_t j = 0; j < d; ++j) {
            volatile float g = S[j] + delta[j];
            delta[j] = g;
        }
        if (ref_topk(delta, d, K_down, msg_idx, msg_val) != 0) goto done;
        count = K_down;
        for (int64_t k = 0; k < count; ++k) delta[msg_idx[k]] = 0.0f;
    } else {
        for (int64_t j = 0; j < d; ++j)
            if (touched[j]) { msg_idx[count] = (int32_t)j; msg_val[count] = S[j]; ++count; }
    }
    for (int64_t k = 0; k < count; ++k) {
        volatile float nw = w[msg_idx[k]] - msg_val[k];
        w[msg_idx[k]] = nw;
    }
    if (up_idx_out) memcpy(up_idx_out, up_idx, (size_t)(N * K_up) * sizeof *up_idx);
    if (up_val_out) memcpy(up_val_out, up_val, (size_t)(N * K_up) * sizeof *up_val);
    if (msg_idx_out) memcpy(msg_idx_out, msg_idx, (size_t)count * sizeof *msg_idx);
    if (msg_val_out) memcpy(msg_val_out, msg_val, (size_t)count * sizeof *msg_val);
    if (msg_count_out) *msg_count_out = count;
    rc = 0;
done:
    free(up_idx); free(up_val); free(S); free(touched); free(msg_idx); free(msg_val);
    return rc;
}

/*
 * The "1 - gamma" diagnostic of the appendix:  ||Top_K(x) - x||_2^2 / ||x||_2^2  for a
 * message (idx[K]) taken from x[d], in double precision.  Top_K(x) - x is -x off the message
 * and 0 on it, so the numerator is the sum of squares of the components NOT sent.
 * Returns 0 for the zero vector.
 */
double ref_lost_energy(const float *x, int64_t d, const int32_t *idx, int64_t K)
{
    uint8_t *sent = (uint8_t *)calloc((size_t)d, 1);
    if (!sent) return -1.0;
    for (int64_t k = 0; k < K; ++k) sent[idx[k]] = 1;
    double lost = 0.0, total = 0.0;
    for (int64_t j = 0; j < d; ++j) {
        double v = (double)x[j];
        total += v * v;
        if (!sent[j]) lost += v * v;
    }
    free(sent);
    return total > 0.0 ? lost / total : 0.0;
}

/*
 * The gap constants of the convergence analysis, as the experiments estimate them per
 * iteration (Section 4, "Convergence Bound Constants"; Assumptions on the gap, uni- and
 * bidirectional).  With  a^q = eps^q + alpha g^q  (or a^q = g^q and delta = 0 for the
 * memory-free iteration, where the step size cancels from the ratio), D_a = sum_q p_q a^q,
 * D_g = sum_q p_q g^q and S = sum_q p_q Top_{K_up}(a^q):
 *   mode 0:  rho_hat = || Top_K(D_a) - S ||_2                                / || scale D_g ||_2
 *   mode 1:  rho     = || Top_K(delta + D_a) - Top_K(delta + S) ||_2         / || scale D_g ||_2
 * with K = K_down for the server-side Top_K, scale = alpha with memories and 1 without.
 * (The assumptions write Top_K(p_q a) where the algorithms write p_q Top_K(a); they agree for
 * p_q > 0 and the algorithms' form is used.)  The dense sums are formed like everything else
 * here: fp32, worker order, one rounding per multiply and per add; the norms in double.
 * eps and delta are the memories BEFORE the iteration (NULL = zero / memory-free).
 * Returns the ratio, 0 when the denominator is 0, or -1 on bad arguments.
 */
double ref_rho(const float *G, const float *eps, const float *delta, int64_t N, int64_t d,
               int64_t K_up, int64_t K_down, const float *p, float alpha, int mode, int nthreads)
{
    if (!G || !p || N < 1 || d < 1 || K_up < 1 || K_up > d || K_down < 1 || K_down > d || (mode != 0 && mode != 1))
        return -1.0;
    double result = -1.0;
    const int memories = eps != NULL;
    float *a = (float *)malloc((size_t)(N * d) * sizeof *a);
    float *Da = (float *)malloc((size_t)d * sizeof *Da);
    float *Dg = (float *)malloc((size_t)d * sizeof *Dg);
    float *S = (float *)malloc((size_t)d * sizeof *S);
    float *left = (float *)calloc((size_t)d, sizeof *left);
    float *right = (float *)calloc((size_t)d, sizeof *right);
    uint8_t *touched = (uint8_t *)malloc((size_t)d);
    int32_t *up_idx = (int32_t *)malloc((size_t)(N * K_up) * sizeof *up_idx);
    float *up_val = (float *)malloc((size_t)(N * K_up) * sizeof *up_val);
    int32_t *t_idx = (int32_t *)malloc((size_t)K_down * sizeof *t_idx);
    float *t_val = (float *)malloc((size_t)K_down * sizeof *t_val);
    if (!a || !Da || !Dg || !S || !left || !right || !touched || !up_idx || !up_val || !t_idx || !t_val) goto done;

    for (int64_t q = 0; q < N; ++q)
        for (int64_t j = 0; j < d; ++j) {
            if (memories) {
                volatile float scaled = alpha * G[q * d + j];
                volatile float v = eps[q * d + j] + scaled;
                a[q * d + j] = v;
            } else {
                a[q * d + j] = G[q * d + j];
            }
        }
    for (int64_t j = 0; j < d; ++j) {
        float sa = 0.0f, sg = 0.0f;
        for (int64_t q = 0; q < N; ++q) {
            volatile float ta = p[q] * a[q * d + j];
            volatile float na = sa + ta;
            sa = na;
            volatile float tg = p[q] * G[q * d + j];
            volatile float ng = sg + tg;
            sg = ng;
        }
        Da[j] = sa;
        Dg[j] = sg;
    }
    if (ref_topk_rows(a, N, d, K_up, up_idx, up_val, nthreads) != 0) goto done;
    if (ref_aggregate(up_idx, up_val, N, K_up, p, d, S, touched) != 0) goto done;
    if (mode == 1 && delta) {
        for (int64_t j = 0; j < d; ++j) {
            volatile float va = delta[j] + Da[j];
            Da[j] = va;
            volatile float vs = S[j] + delta[j];
            S[j] = vs;
        }
    }
    /* left = Top_K(D_a [+ delta]) */
    if (ref_topk(Da, d, K_down, t_idx, t_val) != 0) goto done;
    for (int64_t k = 0; k < K_down; ++k) left[t_idx[k]] = t_val[k];
    /* right = S (mode 0) or Top_K(S [+ delta]) (mode 1) */
    if (mode == 1) {
        if (ref_topk(S, d, K_down, t_idx, t_val) != 0) goto done;
        for (int64_t k = 0; k < K_down; ++k) right[t_idx[k]] = t_val[k];
    } else {
        memcpy(right, S, (size_t)d * sizeof *S);
    }
    {
        double num = 0.0, den = 0.0;
        for (int64_t j = 0; j < d; ++j) {
            double df = (double)left[j] - (double)right[j];
            num += df * df;
            double g = (memories ? (double)alpha : 1.0) * (double)Dg[j];
            den += g * g;
        }
        result = den > 0.0 ? sqrt(num) / sqrt(den) : 0.0;
    }
done:
    free(a); free(Da); free(Dg); free(S); free(left); free(right); free(touched);
    free(up_idx); free(up_val); free(t_idx); free(t_val);
    return result;
}
