/*
 * fp64 CPU oracle for the BiGLA forward pass (ViG, arXiv 2405.18425).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA path is checked against.  It shares no code, headers, tables or helpers
 * with the CUDA library and must never be called from the product path.
 *
 * What it computes (paper Eq. 6, one (batch, head) unit at a time, heads are
 * independent because the paper drops the multi-head index, Sec. 3):
 *
 *   forward  state  S>_t = diag(alpha>_t) S>_{t-1} + k_t^T v_t ,  S>_0     = 0
 *   backward state  S<_t = diag(alpha<_t) S<_{t+1} + k_t^T v_t ,  S<_{L+1} = 0
 *   o>_t = q_t S>_t ,  o<_t = q_t S<_t ,  o_t = (o>_t + o<_t) / 2
 *
 * G_t = alpha_t^T 1 (Eq. 5/6): the decay of row i of the dk x dv state is
 * alpha_t[i], the same for every value column.  Gates arrive as natural logs,
 * log alpha = logsigmoid(g) / tau  (Eq. 5 line 1, tau = 16).
 *
 * No chunking, no blocking, no reordering: the loops below are the recurrence
 * in the paper's order.  Threads only split the independent (b, h) units.
 *
 * Layout of every tensor: dense row-major [B, H, L, d].
 * Parity status: pinned (explicit quadratic form, alpha == 1, flip symmetry,
 * geometric closed form, gate wall, diagonal limit; see tests/test_oracle_pins.py).
 */
#include <math.h>
#include <pthread.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    const double *q, *k, *v, *la_f, *la_b;
    double *out, *out_f, *out_b; /* out_f / out_b may be NULL */
    long L, dk, dv;
    long unit_begin, unit_end;
} job_t;

/* One direction of Eq. 6 for one unit.  step = +1: t = 0..L-1 with the
 * forward gate; step = -1: t = L-1..0 with the backward gate. */
static void scan_one_direction(const double *q, const double *k, const double *v,
                               const double *la, double *o, long L, long dk,
                               long dv, int step, double *S)
{
    memset(S, 0, sizeof(double) * (size_t)(dk * dv));
    long t = step > 0 ? 0 : L - 1;
    for (long n = 0; n < L; ++n, t += step) {
        const double *qt = q + t * dk, *kt = k + t * dk, *at = la + t * dk;
        const double *vt = v + t * dv;
        double *ot = o + t * dv;
        for (long i = 0; i < dk; ++i) {
            const double alpha = exp(at[i]); /* alpha_t[i] in (0, 1] */
            double *Si = S + i * dv;
            for (long j = 0; j < dv; ++j)
                Si[j] = alpha * Si[j] + kt[i] * vt[j]; /* S_t = G_t . S_prev + k_t^T v_t */
        }
        for (long j = 0; j < dv; ++j) {
            double acc = 0.0;
            for (long i = 0; i < dk; ++i)
                acc += qt[i] * S[i * dv + j]; /* o_t = q_t S_t */
            ot[j] = acc;
        }
    }
}

static void *worker(void *arg)
{
    job_t *J = (job_t *)arg;
    const long L = J->L, dk = J->dk, dv = J->dv;
    double *S = (double *)malloc(sizeof(double) * (size_t)(dk * dv));
    double *of = (double *)malloc(sizeof(double) * (size_t)(L * dv));
    double *ob = (double *)malloc(sizeof(double) * (size_t)(L * dv));
    for (long u = J->unit_begin; u < J->unit_end; ++u) {
        const double *q = J->q + u * L * dk, *k = J->k + u * L * dk;
        const double *v = J->v + u * L * dv;
        scan_one_direction(q, k, v, J->la_f + u * L * dk, of, L, dk, dv, +1, S);
        scan_one_direction(q, k, v, J->la_b + u * L * dk, ob, L, dk, dv, -1, S);
        double *o = J->out + u * L * dv;
        for (long x = 0; x < L * dv; ++x)
            o[x] = (of[x] + ob[x]) / 2.0; /* Eq. 6 last line */
        if (J->out_f) memcpy(J->out_f + u * L * dv, of, sizeof(double) * (size_t)(L * dv));
        if (J->out_b) memcpy(J->out_b + u * L * dv, ob, sizeof(double) * (size_t)(L * dv));
    }
    free(S); free(of); free(ob);
    return NULL;
}

/* Returns the number of threads actually used (>= 1), or -1 on bad arguments. */
int oracle_bigla_fwd(const double *q, const double *k, const double *v,
                     const double *la_f, const double *la_b,
                     double *out, double *out_f, double *out_b,
                     long B, long H, long L, long dk, long dv, int nthreads)
{
    if (!q || !k || !v || !la_f || !la_b || !out) return -1;
    if (B < 0 || H < 0 || L < 0 || dk <= 0 || dv <= 0) return -1;
    const long units = B * H;
    if (units == 0 || L == 0) return 1;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > units) nthreads = (int)units;
    if (nthreads > 256) nthreads = 256;
    pthread_t th[256];
    job_t jobs[256];
    for (int w = 0; w < nthreads; ++w) {
        job_t J = { q, k, v, la_f, la_b, out, out_f, out_b, L, dk, dv,
                    units * w / nthreads, units * (w + 1) / nthreads };
        jobs[w] = J;
    }
    for (int w = 1; w < nthreads; ++w) pthread_create(&th[w], NULL, worker, &jobs[w]);
    worker(&jobs[0]);
    for (int w = 1; w < nthreads; ++w) pthread_join(th[w], NULL);
    return nthreads;
}

/* Gate preparation, Eq. 5 line 1 / Eq. 6 line 1 with the logit g given:
 * log alpha = log(sigmoid(g)^(1/tau)) = logsigmoid(g) / tau, written in the
 * overflow-free form  logsigmoid(g) = min(g, 0) - log1p(exp(-|g|)). */
int oracle_gate_prep(const double *g, double *log_alpha, long n, double tau)
{
    if (!g || !log_alpha || n < 0 || !(tau > 0.0)) return -1;
    for (long x = 0; x < n; ++x) {
        const double gx = g[x];
        const double ls = (gx < 0.0 ? gx : 0.0) - log1p(exp(-fabs(gx)));
        log_alpha[x] = ls / tau;
    }
    return 0;
}
