/*
 * Second CPU oracle for the SJA round: dense per-step prefix arrays and a plain binary search per pair.
 *
 * TEST INFRASTRUCTURE ONLY.  Written separately from the step-by-step walk (sja_oracle.c) and from the
 * CUDA path; it shares no code, header or table with either.  Its purpose is speed: the walk needs hours
 * for the 1000-round streaming configuration, this file needs minutes, so it carries full trajectories
 * while the walk re-checks sampled rounds from this file's state (oracle/trajectory.py).
 *
 * What it computes is the same round (rules R1-R6 in the header of sja_oracle.c; Sections 3.1, 3.5, 3.7,
 * 3.8, 3.9 and 4.2 of the paper), restated through four per-step arrays per job, k = 0..len:
 *
 *     D[k] = sum d[0..k)              cumulative duration from the job's first step
 *     W[k] = sum d[i]*m[i], i < k     cumulative work
 *     L[k] = largest safe end index <= k (the job's end always counts), 0 if there is none
 *     M[k] = max m[p..k), k > p       running maximum of the memory envelope from the progress point p
 *                                     (the window-max test of Section 3.9); rebuilt when p moves
 *
 * D and M are non-decreasing in k, so for a gap (start, T, C) and a job at progress p
 *
 *     k_T = largest k in [p, len] with D[k] - D[p] <= T        (binary search on D)
 *     k_C = largest k in [p, len] with M[k] <= C               (binary search on M; k_C = p if m[p] > C)
 *     k*  = L[min(k_T, k_C)],  interest iff the job is eligible (R1) and k* > p
 *                                                              (min(k_T, k_C) = the same search on D cut at k_C)
 *
 * because every end index up to min(k_T, k_C) satisfies both bounds and a subjob may only end on a safe
 * boundary (Section 3.7).  dur = D[k*] - D[p], work = W[k*] - W[p], peak = M[k*].
 * Score (R4), per-gap argmax with ties to the lowest job id (R5) and the commit rule (R6) are written out
 * again below, independently of the walk.
 *
 * Loop order: jobs outermost (spread over threads), gaps innermost, so one job's arrays stay in cache for the
 * whole batch; every thread keeps its own best candidate per gap and the threads are folded at the end.
 * The duration thresholds, window options and power caps of the walk are not implemented here.
 *
 * Pins (tests/test_oracle_fast_pins.py): equality with the walk on the small published configurations,
 * scaled versions of the large ones over committed rounds under all policies, exhaustive enumeration on
 * tiny inputs, zero-length / finished / not-ready jobs, and the commit rule against the walk's.
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define O3_NO_JOB 0xFFFFFFFFu

typedef struct {
    uint32_t slice, start_ms, T_ms, C_MiB;
} o3_gap;

typedef struct {
    uint32_t job, end_step, dur_ms, granted;
    uint64_t score;
} o3_award;

enum { O3_EFFICIENCY = 0, O3_FAIRNESS = 1, O3_SLA = 2, O3_TIGHT_FIT = 3 };

typedef struct {
    uint32_t n_jobs;
    const uint64_t *off;   /* borrowed: [n_jobs + 1] */
    const uint32_t *m;     /* borrowed: per-step memory (M is rebuilt from it) */
    uint64_t *D, *W;       /* entry (j, k) at off[j] + j + k */
    uint32_t *L, *M;
    uint32_t *p_cached;    /* progress point M was built for; 0xFFFFFFFF = never */
} o3_state;

typedef struct {
    uint32_t cls;          /* priority class (SLA), else 0 */
    uint64_t score;
    uint32_t job, k, dur;
    int have;
} o3_cand;

void o3_destroy(o3_state *s)
{
    if (!s) return;
    free(s->D); free(s->W); free(s->L); free(s->M); free(s->p_cached);
    free(s);
}

/* Builds D, W and L for every job.  off, m must stay valid for the life of the state. */
o3_state *o3_create(uint32_t n_jobs, const uint64_t *off, const uint32_t *dur_ms, const uint32_t *mem_MiB,
                    const uint32_t *safe_bits)
{
    o3_state *s = (o3_state *)calloc(1, sizeof(o3_state));
    if (!s) return NULL;
    const uint64_t n_entries = off[n_jobs] + n_jobs;
    s->n_jobs = n_jobs;
    s->off = off;
    s->m = mem_MiB;
    s->D = (uint64_t *)malloc(n_entries * sizeof(uint64_t));
    s->W = (uint64_t *)malloc(n_entries * sizeof(uint64_t));
    s->L = (uint32_t *)malloc(n_entries * sizeof(uint32_t));
    s->M = (uint32_t *)malloc(n_entries * sizeof(uint32_t));
    s->p_cached = (uint32_t *)malloc((size_t)n_jobs * sizeof(uint32_t) + 4);
    if (!s->D || !s->W || !s->L || !s->M || !s->p_cached) { o3_destroy(s); return NULL; }
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t j = 0; j < (int64_t)n_jobs; ++j) {
        const uint64_t b = off[j], len = off[j + 1] - off[j], e = b + (uint64_t)j;
        uint64_t accD = 0, accW = 0;
        uint32_t last_safe = 0;
        s->D[e] = 0; s->W[e] = 0; s->L[e] = 0; s->M[e] = 0;
        for (uint64_t k = 1; k <= len; ++k) {
            const uint64_t i = b + k - 1;
            accD += dur_ms[i];
            accW += (uint64_t)dur_ms[i] * (uint64_t)mem_MiB[i];
            if (((safe_bits[i >> 5] >> (i & 31u)) & 1u) || k == len) last_safe = (uint32_t)k;
            s->D[e + k] = accD;
            s->W[e + k] = accW;
            s->L[e + k] = last_safe;
            s->M[e + k] = 0;
        }
        s->p_cached[j] = 0xFFFFFFFFu;
    }
    return s;
}

/* M[k] = max m[p..k) for k in (p, len], for every job whose progress point moved since the last call. */
static void o3_sync(o3_state *s, const uint32_t *progress)
{
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t j = 0; j < (int64_t)s->n_jobs; ++j) {
        const uint32_t p = progress[j];
        if (s->p_cached[j] == p) continue;
        const uint64_t b = s->off[j], len = s->off[j + 1] - s->off[j], e = b + (uint64_t)j;
        uint32_t run = 0;
        for (uint64_t k = (uint64_t)p + 1; k <= len; ++k) {
            if (s->m[b + k - 1] > run) run = s->m[b + k - 1];
            s->M[e + k] = run;
        }
        s->p_cached[j] = p;
    }
}

/* Number of leading entries of a[0..n) that are <= v (a non-decreasing). */
/* (binary search that halves the remaining length; the window [first, first + n) always holds the answer's
 * predecessor, and the conditional advance compiles to a conditional move instead of a branch) */
static uint64_t count_le_u64(const uint64_t *a, uint64_t n, uint64_t v)
{
    if (n == 0) return 0;
    const uint64_t *first = a;
    while (n > 1) {
        const uint64_t half = n >> 1;
        first = (first[half - 1] <= v) ? first + half : first;
        n -= half;
    }
    return (uint64_t)(first - a) + (first[0] <= v ? 1u : 0u);
}

static uint64_t count_le_u32(const uint32_t *a, uint64_t n, uint32_t v)
{
    if (n == 0) return 0;
    const uint32_t *first = a;
    while (n > 1) {
        const uint64_t half = n >> 1;
        first = (first[half - 1] <= v) ? first + half : first;
        n -= half;
    }
    return (uint64_t)(first - a) + (first[0] <= v ? 1u : 0u);
}

/* candidate a beats b: larger class, then larger score, then lower job id (R4, R5) */
static int cand_beats(const o3_cand *a, const o3_cand *b)
{
    if (!b->have) return 1;
    if (a->cls != b->cls) return a->cls > b->cls;
    if (a->score != b->score) return a->score > b->score;
    return a->job < b->job;
}

/*
 * R1-R5 for a batch of gaps from the given state.  Returns 0, -1 for an unknown policy or a missing
 * attribute array, -2 when out of memory.
 */
int o3_select(o3_state *s, const uint32_t *progress, const uint32_t *ready_ms, const uint32_t *wait_ms,
              const uint8_t *prio, uint32_t n_gaps, const o3_gap *gaps, uint32_t policy, o3_award *awards)
{
    if (policy > O3_TIGHT_FIT) return -1;
    if (policy == O3_FAIRNESS && !wait_ms) return -1;
    if (policy == O3_SLA && !prio) return -1;
    o3_sync(s, progress);

    int n_threads = 1;
#ifdef _OPENMP
    n_threads = omp_get_max_threads();
#endif
    o3_cand *best = (o3_cand *)calloc((size_t)n_threads * (size_t)n_gaps + 1, sizeof(o3_cand));
    if (!best) return -2;

#pragma omp parallel
    {
        int t = 0;
#ifdef _OPENMP
        t = omp_get_thread_num();
#endif
        o3_cand *mine = best + (size_t)t * n_gaps;
#pragma omp for schedule(dynamic, 16)
        for (int64_t jj = 0; jj < (int64_t)s->n_jobs; ++jj) {
            const uint32_t j = (uint32_t)jj;
            const uint64_t len = s->off[j + 1] - s->off[j];
            const uint32_t p = progress[j];
            if ((uint64_t)p >= len) continue;                      /* R1: finished (or empty) job */
            const uint64_t e = s->off[j] + (uint64_t)j;
            const uint64_t *D = s->D + e, *W = s->W + e;
            const uint32_t *L = s->L + e, *M = s->M + e;
            const uint64_t n_after = len - p;                      /* end indices p+1 .. len */
            const uint32_t ready = ready_ms[j];
            /* k_C depends on the job and the capacity only: remember it per distinct capacity of the batch */
            uint32_t memo_C[8];
            uint64_t memo_k[8];
            int n_memo = 0;
            for (uint32_t g = 0; g < n_gaps; ++g) {
                if (gaps[g].start_ms < ready) continue;            /* R1: the gap opens before the job is ready */
                const uint32_t C = gaps[g].C_MiB;
                uint64_t kC = 0;
                int hit = 0;
                for (int q = 0; q < n_memo; ++q)
                    if (memo_C[q] == C) { kC = memo_k[q]; hit = 1; break; }
                if (!hit) {
                    kC = (uint64_t)p + count_le_u32(M + p + 1, n_after, C);
                    if (n_memo < 8) { memo_C[n_memo] = C; memo_k[n_memo] = kC; ++n_memo; }
                }
                if (kC == p) continue;                             /* the next step alone exceeds the capacity */
                /* min(k_T, k_C): the search for k_T need not look beyond k_C */
                const uint64_t kmin = (uint64_t)p + count_le_u64(D + p + 1, kC - p, D[p] + (uint64_t)gaps[g].T_ms);
                const uint32_t k = L[kmin];
                if (k <= p) continue;                              /* no safe boundary inside both bounds: decline */
                o3_cand c;
                c.have = 1;
                c.job = j;
                c.k = k;
                c.dur = (uint32_t)(D[k] - D[p]);
                c.cls = 0;
                c.score = W[k] - W[p];
                if (policy == O3_FAIRNESS) c.score *= (uint64_t)(1u + wait_ms[j] / 1000u);
                else if (policy == O3_SLA) c.cls = prio[j];
                else if (policy == O3_TIGHT_FIT) c.score = M[k];
                if (cand_beats(&c, &mine[g])) mine[g] = c;
            }
        }
    }
    for (uint32_t g = 0; g < n_gaps; ++g) {
        o3_cand w;
        memset(&w, 0, sizeof(w));
        for (int t = 0; t < n_threads; ++t) {
            const o3_cand *c = &best[(size_t)t * n_gaps + g];
            if (c->have && cand_beats(c, &w)) w = *c;
        }
        awards[g].job = w.have ? w.job : O3_NO_JOB;
        awards[g].end_step = w.have ? w.k : 0;
        awards[g].dur_ms = w.have ? w.dur : 0;
        awards[g].granted = 0;
        awards[g].score = w.have ? w.score : 0;
    }
    free(best);
    return 0;
}

/*
 * R6: every job that won at least one gap accepts the one with the largest end step, ties to the lowest gap
 * id; that gap is granted, the job's progress moves to the end step and its ready time to start + dur.
 * Returns the number of grants, -1 if start + dur does not fit in 32 bits, -2 when out of memory.
 */
int64_t o3_commit(uint32_t n_jobs, uint32_t *progress, uint32_t *ready_ms, uint32_t n_gaps, const o3_gap *gaps,
                  o3_award *awards)
{
    uint32_t *accepted = (uint32_t *)malloc((size_t)n_jobs * sizeof(uint32_t) + 4);   /* gap id per job */
    if (!accepted) return -2;
    for (uint32_t j = 0; j < n_jobs; ++j) accepted[j] = O3_NO_JOB;
    for (uint32_t g = 0; g < n_gaps; ++g) {                        /* ascending gap id: ">" keeps the lowest on ties */
        awards[g].granted = 0;
        const uint32_t j = awards[g].job;
        if (j == O3_NO_JOB || j >= n_jobs) continue;
        if (accepted[j] == O3_NO_JOB || awards[g].end_step > awards[accepted[j]].end_step) accepted[j] = g;
    }
    int64_t granted = 0;
    for (uint32_t g = 0; g < n_gaps; ++g) {
        const uint32_t j = awards[g].job;
        if (j == O3_NO_JOB || j >= n_jobs || accepted[j] != g) continue;
        const uint64_t new_ready = (uint64_t)gaps[g].start_ms + (uint64_t)awards[g].dur_ms;
        if (new_ready > 0xFFFFFFFFull) { free(accepted); return -1; }
        awards[g].granted = 1;
        progress[j] = awards[g].end_step;
        ready_ms[j] = (uint32_t)new_ready;
        ++granted;
    }
    free(accepted);
    return granted;
}

int o3_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
