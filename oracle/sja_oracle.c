/*
 * CPU oracle for the SJA advertise / signal / select / commit round.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code, header, table or helper with the
 * CUDA path and must never be linked into, or called from, the product path.
 *
 * What it computes, and where the paper defines it:
 *   - A subjob is a self-contained fragment of a job that fits the offered window
 *     in time and stays below the slice capacity for its whole lifetime (Section 3.1).
 *   - A job is admissible in a window of length T on a slice of capacity C when the
 *     maximum of its (risk-adjusted) memory envelope U over the window is <= C
 *     (Section 3.8, and the window-max test of Section 3.9).  The per-step mem_MiB
 *     array is U sampled per step; memory is constant within a step.
 *   - A subjob ends at a safe boundary, the natural cut point where a job can be
 *     paused with a checkpoint (Section 3.7).
 *   - Three-phase protocol: the scheduler advertises gaps, each job signals interest
 *     or declines, the scheduler applies its policy and grants the slot; nothing is
 *     materialised before the grant (Section 3.5).  Greedy slot filling without
 *     lookahead is the intended design (Section 4.2).
 *   - The granted job resumes later from the end of its last completed fragment
 *     (Sections 3.1, 3.5).
 *
 * Integer formalisation used here (the paper is prose; every choice is a stated reading):
 *   R1 eligibility : p_j < len_j and start_g >= ready_j.
 *   R2 candidates  : k in (p_j, len_j] with step k-1 safe (the last step of a job always
 *                    counts as safe), sum d[p_j..k) <= T_g, max m[p_j..k) <= C_g (inclusive).
 *   R3 signal      : interest iff eligible and a candidate exists; the subjob is the
 *                    longest one, k* = max candidates; dur = sum d, work = sum d*m (u64).
 *   R4 score       : efficiency  work;
 *                    fairness    work * (1 + wait_j/1000), truncating division, u64;
 *                    SLA         lexicographic (prio_j, work), larger prio = more urgent;
 *                    tight fit   peak = max m over the subjob: the job that leaves the least slack
 *                                C_g - peak on the slice wins (the slack-minimising principle of
 *                                Section 3.9, applied by the scheduler across jobs).
 *   R5 select      : per gap, the interested job with the largest key; ties go to the
 *                    lowest job id; no interested job -> SJA_NO_JOB and zeros.
 *   R2' bounds     : optional subjob duration thresholds (Section 4.3, item 5: minimum and maximum
 *                    subjob duration enforced at the framework level): a candidate also needs
 *                    tau_min <= sum d[p_j..k) <= tau_max.  tau_min = 0 and tau_max = 2^32-1 switch
 *                    them off.
 *   R6 commit      : a job that won several gaps accepts the one with the largest k*,
 *                    ties to the lowest gap id; that gap is granted, the others are not;
 *                    then p_j = k*, ready_j = start_g + dur.
 *   R1'' options   : two optional refinements of the window a pair sees, both off by default.
 *                    Late start: a job that becomes ready inside the window may begin then, so
 *                    begin = max(start_g, ready_j), eligible iff begin <= start_g + T_g, and only
 *                    the rest of the window counts: sum d <= T_g - (begin - start_g); the commit
 *                    sets ready_j = begin + dur.  Deadline (Section 4.4, item 2: admit only
 *                    subjobs that complete by their deadline; the risk margin lives in the
 *                    durations, as it does in the memory envelope): a candidate also needs
 *                    begin + sum d <= deadline_j; 2^32-1 means no deadline.
 *   R2'' power     : optional second resource envelope (Section 4.4, item 1: offers carry a power
 *                    cap, subjobs answer with a predicted power trace, admission keeps
 *                    max_t P(t) <= power_cap with the risk margin in the trace): with a per-step
 *                    power_W array and a per-gap cap, a candidate also needs
 *                    max power_W[p_j..k) <= cap_g; a cap of 2^32-1 means none.
 *
 *   R3h hysteresis : optional guard against over-fragmentation (Section 3.9: a further subdivision is accepted
 *                    only if it gains a minimum of slack).  Let k_T be the longest candidate when the memory
 *                    capacity bound is lifted (every other rule stays) and k* the longest candidate proper.
 *                    k* < k_T means the capacity forces the job to cut earlier than the window would allow -- a
 *                    further subdivision.  What the cut gains is the demand it sheds,
 *                    max m[p_j..k_T) - max m[p_j..k*); the job signals interest only if that gain is at least
 *                    min_slack_gain MiB, else it declines and keeps the longer fragment for a window it fits.
 *                    min_slack_gain = 0 switches the rule off.
 *   R4' locality   : optional state- and locality-aware admission (Section 4.4, item 5; the Preference signal of
 *                    Section 3.5): jobs declare a predicted checkpoint size ckpt_MiB_j and remember the slice
 *                    their last fragment ran on.  A window on another slice means moving that state, so the
 *                    policy score (the work for SLA, whose class stays) is lowered by weight * ckpt_MiB_j,
 *                    not below zero; a window on the same slice, and a job that has not run yet, pay nothing.
 *                    The commit records the granted gap's slice as the job's last slice.
 *
 * The walk below visits one step at a time, exactly in that order: no prefix arrays,
 * no search, no blocking.  OpenMP only spreads independent gaps over host threads.
 *
 * Pins (tests/test_oracle_pins.py and the other tests/test_oracle_*_pins.py): exhaustive prefix enumeration on tiny inputs,
 * closed forms, reductions to numpy cumsum / searchsorted, monotonicity and symmetry
 * properties, the rigid-job special case, hand-computed policy examples, and the paper's
 * illustrative scenario.  The paper prints no numeric award values, so beyond those pins
 * the award values are "parity unpinned".
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_NO_JOB 0xFFFFFFFFu

typedef struct {
    uint32_t slice, start_ms, T_ms, C_MiB;
} orc_gap;

typedef struct {
    uint32_t job, end_step, dur_ms, granted;
    uint64_t score;
} orc_award;

enum { ORC_EFFICIENCY = 0, ORC_FAIRNESS = 1, ORC_SLA = 2, ORC_TIGHT_FIT = 3 };

static int step_is_safe(const uint32_t *safe_bits, uint64_t i)
{
    return (int)((safe_bits[i >> 5] >> (i & 31u)) & 1u);
}

/*
 * The walk of one pair: the longest candidate end index under the given bounds.  `begin` is when the subjob
 * would start, `window_end` when the gap closes.  Returns 1 and fills k / dur / work / peak, or 0.
 */
static int walk_pair(const uint32_t *dur_ms, const uint32_t *mem_MiB, const uint32_t *safe_bits,
                     uint64_t s, uint64_t e, uint32_t p, uint64_t begin, uint64_t window_end, uint32_t C_MiB,
                     uint32_t tau_min_ms, uint32_t tau_max_ms, int has_deadline, uint32_t deadline_ms,
                     const uint32_t *power_W, int has_cap, uint32_t power_cap_W,
                     uint32_t *k_out, uint32_t *dur_out, uint64_t *work_out, uint32_t *peak_out)
{
    uint64_t acc = 0, work = 0;
    uint32_t peak = 0, power_peak = 0;
    int found = 0;
    for (uint64_t i = s + p; i < e; ++i) {
        acc += dur_ms[i];
        if (mem_MiB[i] > peak) peak = mem_MiB[i];
        work += (uint64_t)dur_ms[i] * (uint64_t)mem_MiB[i];
        if (begin + acc > window_end || peak > C_MiB) break;   /* R2: window or capacity broken */
        if (has_cap) {
            if (power_W[i] > power_peak) power_peak = power_W[i];
            if (power_peak > power_cap_W) break;               /* R2'': above the power cap of the offer */
        }
        if (has_deadline && begin + acc > (uint64_t)deadline_ms) break;   /* R1'': would finish after the deadline */
        if (acc > (uint64_t)tau_max_ms) break;             /* R2': longer than the maximum subjob */
        if ((step_is_safe(safe_bits, i) || i + 1 == e)     /* R2: safe boundary after step i */
            && acc >= (uint64_t)tau_min_ms) {              /* R2': not shorter than the minimum subjob */
            found = 1;
            *k_out = (uint32_t)(i + 1 - s);
            *dur_out = (uint32_t)acc;
            *work_out = work;
            *peak_out = peak;
        }
    }
    return found;
}

/*
 * R1-R3 for one (gap, job) pair.  Returns 1 for interest (and fills k, dur, work),
 * 0 for decline.  [s, e) is the job's range of global step indices, p its progress.
 */
int orc_pair(const uint32_t *dur_ms, const uint32_t *mem_MiB, const uint32_t *safe_bits,
             uint64_t s, uint64_t e, uint32_t p, uint32_t ready_ms,
             uint32_t start_ms, uint32_t T_ms, uint32_t C_MiB,
             uint32_t tau_min_ms, uint32_t tau_max_ms,
             int late_start, uint32_t deadline_ms,
             const uint32_t *power_W /* per step like mem_MiB, or NULL */, uint32_t power_cap_W,
             uint32_t min_slack_gain_MiB /* R3h, 0 = off */,
             uint32_t *k_out, uint32_t *dur_out, uint64_t *work_out, uint32_t *peak_out /* may be NULL */)
{
    uint64_t len = e - s;
    if ((uint64_t)p >= len) return 0;            /* R1: finished job */
    uint64_t begin = start_ms;                   /* when the subjob would start running */
    if (start_ms < ready_ms) {
        if (!late_start) return 0;               /* R1: gap opens before the job is ready */
        begin = ready_ms;                        /* R1'': start inside the window */
    }
    uint64_t window_end = (uint64_t)start_ms + (uint64_t)T_ms;
    if (begin > window_end) return 0;            /* R1'': ready only after the window has closed */
    const int has_deadline = deadline_ms != 0xFFFFFFFFu;          /* 2^32-1: no deadline */
    if (has_deadline && begin > (uint64_t)deadline_ms) return 0; /* R1'': deadline already passed */
    const int has_cap = power_W != NULL && power_cap_W != 0xFFFFFFFFu;

    uint32_t k = 0, dur = 0, peak = 0;
    uint64_t work = 0;
    if (!walk_pair(dur_ms, mem_MiB, safe_bits, s, e, p, begin, window_end, C_MiB, tau_min_ms, tau_max_ms,
                   has_deadline, deadline_ms, power_W, has_cap, power_cap_W, &k, &dur, &work, &peak))
        return 0;
    if (min_slack_gain_MiB > 0) {
        /* R3h: the fragment the window alone would allow (capacity bound lifted) */
        uint32_t k_T = 0, dur_T = 0, peak_T = 0;
        uint64_t work_T = 0;
        walk_pair(dur_ms, mem_MiB, safe_bits, s, e, p, begin, window_end, 0xFFFFFFFFu, tau_min_ms, tau_max_ms,
                  has_deadline, deadline_ms, power_W, has_cap, power_cap_W, &k_T, &dur_T, &work_T, &peak_T);
        if (k_T > k && peak_T - peak < min_slack_gain_MiB) return 0;   /* the cut gains too little: decline */
    }
    *k_out = k;
    *dur_out = dur;
    *work_out = work;
    if (peak_out) *peak_out = peak;
    return 1;
}

/* R4: the policy key of an interested job, as (class, score). */
static void policy_key(uint32_t policy, uint64_t work, uint32_t peak, uint32_t j,
                       const uint32_t *wait_ms, const uint8_t *prio, uint64_t penalty,
                       uint32_t *cls_out, uint64_t *score_out)
{
    *cls_out = 0;
    *score_out = work;
    if (policy == ORC_FAIRNESS) {
        *score_out = work * (uint64_t)(1u + wait_ms[j] / 1000u);
    } else if (policy == ORC_SLA) {
        *cls_out = prio[j];
    } else if (policy == ORC_TIGHT_FIT) {
        *score_out = peak;      /* largest peak <=> least slack C_g - peak */
    }
    /* R4': the cost of moving the job's state to another slice, never below zero */
    *score_out -= penalty < *score_out ? penalty : *score_out;
}

/*
 * R1-R5 for a batch of gaps.  progress / ready_ms are read, never written
 * (no subjob state exists before a grant, Section 3.5).
 * Returns 0, or -1 for an unknown policy / missing attribute array.
 */
int orc_select(uint32_t n_jobs, const uint64_t *off,
               const uint32_t *dur_ms, const uint32_t *mem_MiB, const uint32_t *safe_bits,
               const uint32_t *progress, const uint32_t *ready_ms,
               const uint32_t *wait_ms, const uint8_t *prio,
               uint32_t n_gaps, const orc_gap *gaps, uint32_t policy,
               uint32_t tau_min_ms, uint32_t tau_max_ms,
               int late_start, const uint32_t *deadline_ms /* per job, or NULL = none */,
               const uint32_t *power_W /* per step, or NULL */, const uint32_t *power_cap_W /* per gap, or NULL */,
               uint32_t min_slack_gain_MiB /* R3h, 0 = off */,
               const uint32_t *ckpt_MiB /* R4': per job, or NULL = off */,
               const uint32_t *last_slice /* per job, 2^32-1 = has not run yet; NULL = none has */,
               uint32_t locality_weight,
               orc_award *awards)
{
    if (policy > ORC_TIGHT_FIT) return -1;
    if (policy == ORC_FAIRNESS && !wait_ms) return -1;
    if (policy == ORC_SLA && !prio) return -1;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t g = 0; g < (int64_t)n_gaps; ++g) {
        orc_gap gap = gaps[g];
        int have = 0;
        uint32_t best_cls = 0, best_job = ORC_NO_JOB, best_k = 0, best_dur = 0;
        uint64_t best_score = 0;
        for (uint32_t j = 0; j < n_jobs; ++j) {
            uint32_t k, dur, peak;
            uint64_t work;
            if (!orc_pair(dur_ms, mem_MiB, safe_bits, off[j], off[j + 1], progress[j],
                          ready_ms[j], gap.start_ms, gap.T_ms, gap.C_MiB, tau_min_ms, tau_max_ms,
                          late_start, deadline_ms ? deadline_ms[j] : 0xFFFFFFFFu,
                          power_W, power_cap_W ? power_cap_W[g] : 0xFFFFFFFFu, min_slack_gain_MiB,
                          &k, &dur, &work, &peak))
                continue;                                      /* decline */
            uint32_t cls;
            uint64_t score, penalty = 0;
            if (ckpt_MiB && last_slice && last_slice[j] != 0xFFFFFFFFu && last_slice[j] != gap.slice)
                penalty = (uint64_t)locality_weight * (uint64_t)ckpt_MiB[j];   /* R4': the state has to move */
            policy_key(policy, work, peak, j, wait_ms, prio, penalty, &cls, &score);
            /* jobs are visited in ascending id, so a strict ">" keeps the lowest id on ties */
            if (!have || cls > best_cls || (cls == best_cls && score > best_score)) {
                have = 1;
                best_cls = cls;
                best_score = score;
                best_job = j;
                best_k = k;
                best_dur = dur;
            }
        }
        orc_award a;
        a.job = have ? best_job : ORC_NO_JOB;
        a.end_step = have ? best_k : 0;
        a.dur_ms = have ? best_dur : 0;
        a.granted = 0;
        a.score = have ? best_score : 0;
        awards[g] = a;
    }
    return 0;
}

/*
 * R6.  Marks granted gaps in awards[], advances progress / ready_ms of the granted
 * jobs, returns the number of grants (or -1 if begin + dur does not fit in 32 bits).
 */
int64_t orc_commit(uint32_t n_jobs, uint32_t *progress, uint32_t *ready_ms,
                   uint32_t n_gaps, const orc_gap *gaps, orc_award *awards, int late_start,
                   uint32_t *last_slice /* R4': per job, updated for granted jobs; may be NULL */)
{
    int64_t granted = 0;
    for (uint32_t g = 0; g < n_gaps; ++g) awards[g].granted = 0;
    for (uint32_t g = 0; g < n_gaps; ++g) {
        uint32_t j = awards[g].job;
        if (j == ORC_NO_JOB || j >= n_jobs) continue;
        /* is g the gap this job accepts?  largest k*, then lowest gap id */
        int accept = 1;
        for (uint32_t h = 0; h < n_gaps; ++h) {
            if (h == g || awards[h].job != j) continue;
            if (awards[h].end_step > awards[g].end_step ||
                (awards[h].end_step == awards[g].end_step && h < g)) {
                accept = 0;
                break;
            }
        }
        if (accept) awards[g].granted = 1;
    }
    for (uint32_t g = 0; g < n_gaps; ++g) {
        if (!awards[g].granted) continue;
        uint32_t j = awards[g].job;
        uint64_t begin = gaps[g].start_ms;
        if (late_start && ready_ms[j] > gaps[g].start_ms) begin = ready_ms[j];   /* R1'': began inside the window */
        uint64_t new_ready = begin + (uint64_t)awards[g].dur_ms;
        if (new_ready > 0xFFFFFFFFull) return -1;
        progress[j] = awards[g].end_step;
        ready_ms[j] = (uint32_t)new_ready;
        if (last_slice) last_slice[j] = gaps[g].slice;     /* R4': where the job's state now lives */
        ++granted;
    }
    return granted;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
