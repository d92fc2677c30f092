/*
 * CLT-k oracle, all host cores -- TEST INFRASTRUCTURE, not part of the product path.
 *
 * The "parallel CPU baseline" of the benchmark: one iteration of Algorithm 1 computed by the very
 * routines of cltk_oracle.c (oracle_accumulate, oracle_topk, oracle_learner, oracle_reduce's
 * arithmetic, oracle_apply), with their loops handed out to POSIX threads:
 *   - the leader's accumulation and the reduction are cut into coordinate ranges;
 *   - Eq. 2: every thread takes the exact top-k of its own range (at most k of its coordinates can be
 *     among the k largest overall), and the k largest of those candidates -- kept in ascending index
 *     order, so that the stable tie rule "lower index first" carries over -- are the global set;
 *   - the learners (gather Eq. 3 + memory update Eq. 4) are dealt to the threads one at a time.
 * Results are identical, bit for bit, to oracle_step_f32 (a test checks exactly that); only the wall
 * clock differs.  fp32 only: this file exists for timing, the fp64 pins use the plain oracle.
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

void oracle_accumulate_f32(const float *g, const float *m, int64_t d, float *acc);
int oracle_topk_f32(const float *x, int64_t d, int64_t k, int32_t *idx_out, uint8_t *sel);
void oracle_learner_f32(const float *g, float *m, int64_t d, const int32_t *idx, int64_t k, const uint8_t *sel,
                        float beta, float *gathered);
void oracle_apply_f32(float *theta, const int32_t *idx, const float *val, int64_t k, float lr);

typedef struct {
    int tid, nthreads, phase;
    const float *const *g;
    float *const *m;
    int32_t n, leader;
    int64_t d, k;
    float beta;
    float *accL;            /* [d] */
    int32_t *cand_idx;      /* [nthreads * k] per-range winners, global indices, ascending inside a range */
    int64_t *cand_cnt;      /* [nthreads] */
    const int32_t *idx;     /* [k] the global set (phases 2, 3) */
    const uint8_t *sel;     /* [d] */
    float *G;               /* [n * k] */
    float *val;             /* [k] */
    int rc;
} job_t;

static void range_of(int64_t total, int tid, int nthreads, int64_t *lo, int64_t *hi)
{
    *lo = total * tid / nthreads;
    *hi = total * (tid + 1) / nthreads;
}

static void *worker(void *arg)
{
    job_t *J = (job_t *)arg;
    int64_t lo, hi;
    J->rc = 0;
    if (J->phase == 0) {                       /* leader: acc = m + g on this thread's range */
        range_of(J->d, J->tid, J->nthreads, &lo, &hi);
        oracle_accumulate_f32(J->g[J->leader] + lo, J->m[J->leader] + lo, hi - lo, J->accL + lo);
    } else if (J->phase == 1) {                /* Eq. 2 inside the range */
        range_of(J->d, J->tid, J->nthreads, &lo, &hi);
        const int64_t kk = J->k < hi - lo ? J->k : hi - lo;
        int32_t *out = J->cand_idx + (int64_t)J->tid * J->k;
        J->cand_cnt[J->tid] = kk;
        if (kk > 0) {
            J->rc = oracle_topk_f32(J->accL + lo, hi - lo, kk, out, 0);
            for (int64_t j = 0; j < kk; ++j) out[j] += (int32_t)lo;
        }
    } else if (J->phase == 2) {                /* learners tid, tid + T, ... */
        for (int32_t i = J->tid; i < J->n; i += J->nthreads)
            oracle_learner_f32(J->g[i], J->m[i], J->d, J->idx, J->k, J->sel, J->beta, J->G + (int64_t)i * J->k);
    } else {                                   /* Algorithm 1 line 10 on this thread's share of the k coordinates */
        range_of(J->k, J->tid, J->nthreads, &lo, &hi);
        for (int64_t j = lo; j < hi; ++j) {
            float s = J->G[j];
            for (int32_t i = 1; i < J->n; ++i) s = s + J->G[(int64_t)i * J->k + j];
            J->val[j] = s / (float)J->n;
        }
    }
    return 0;
}

static int run_phase(job_t *jobs, int nthreads, int phase)
{
    pthread_t *th = (pthread_t *)malloc((size_t)nthreads * sizeof *th);
    int rc = th ? 0 : -1;
    for (int t = 0; t < nthreads && rc == 0; ++t) {
        jobs[t].phase = phase;
        if (pthread_create(&th[t], 0, worker, &jobs[t]) != 0) {
            for (int u = 0; u < t; ++u) pthread_join(th[u], 0);
            rc = -1;
        }
    }
    if (rc == 0)
        for (int t = 0; t < nthreads; ++t) {
            pthread_join(th[t], 0);
            if (jobs[t].rc != 0) rc = -1;
        }
    free(th);
    return rc;
}

/* oracle_step_f32 with its loops spread over `nthreads` threads.  Same arguments, same results. */
int oracle_step_threads_f32(const float *const *g, float *const *m, float *theta, int64_t t, int32_t n, int64_t d,
                            int64_t k, float beta, float lr, int32_t nthreads, int32_t *idx, float *val, float *G)
{
    if (nthreads < 1) nthreads = 1;
    if ((int64_t)nthreads > d) nthreads = (int32_t)d;
    const int32_t leader = (int32_t)(t % n);
    float *accL = (float *)malloc((size_t)d * sizeof *accL);
    uint8_t *sel = (uint8_t *)malloc((size_t)d);
    float *Gbuf = G ? G : (float *)malloc((size_t)n * (size_t)k * sizeof *Gbuf);
    int32_t *cand_idx = (int32_t *)malloc((size_t)nthreads * (size_t)k * sizeof *cand_idx);
    int64_t *cand_cnt = (int64_t *)calloc((size_t)nthreads, sizeof *cand_cnt);
    job_t *jobs = (job_t *)calloc((size_t)nthreads, sizeof *jobs);
    int rc = -1;
    if (accL && sel && Gbuf && cand_idx && cand_cnt && jobs) {
        for (int q = 0; q < nthreads; ++q) {
            job_t *J = &jobs[q];
            J->tid = q; J->nthreads = nthreads; J->g = g; J->m = m; J->n = n; J->leader = leader; J->d = d; J->k = k;
            J->beta = beta; J->accL = accL; J->cand_idx = cand_idx; J->cand_cnt = cand_cnt; J->idx = idx; J->sel = sel;
            J->G = Gbuf; J->val = val;
        }
        rc = run_phase(jobs, nthreads, 0);
        if (rc == 0) rc = run_phase(jobs, nthreads, 1);
        if (rc == 0) {
            /* the candidates of all ranges, in ascending index order; their k largest are the answer */
            int64_t total = 0;
            for (int q = 0; q < nthreads; ++q) total += cand_cnt[q];
            int32_t *cidx = (int32_t *)malloc((size_t)total * sizeof *cidx);
            float *cval = (float *)malloc((size_t)total * sizeof *cval);
            int32_t *pick = (int32_t *)malloc((size_t)k * sizeof *pick);
            rc = (cidx && cval && pick) ? 0 : -1;
            if (rc == 0) {
                int64_t o = 0;
                for (int q = 0; q < nthreads; ++q)
                    for (int64_t j = 0; j < cand_cnt[q]; ++j) {
                        cidx[o] = cand_idx[(int64_t)q * k + j];
                        cval[o] = accL[cidx[o]];
                        ++o;
                    }
                rc = oracle_topk_f32(cval, total, k, pick, 0);
            }
            if (rc == 0) {
                memset(sel, 0, (size_t)d);
                for (int64_t j = 0; j < k; ++j) { idx[j] = cidx[pick[j]]; sel[idx[j]] = 1; }   /* pick is ascending */
            }
            free(cidx); free(cval); free(pick);
        }
        if (rc == 0) rc = run_phase(jobs, nthreads, 2);
        if (rc == 0) rc = run_phase(jobs, nthreads, 3);
        if (rc == 0 && theta) oracle_apply_f32(theta, idx, val, k, lr);
    }
    free(accL); free(sel); free(cand_idx); free(cand_cnt); free(jobs);
    if (!G) free(Gbuf);
    return rc;
}
