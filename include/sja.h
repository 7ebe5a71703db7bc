/*
 * libsja -- the advertise / signal / select / commit round of Scheduler-Driven Job
 * Atomization (SJA) on one NVIDIA B200 (sm_100a).
 *
 * The paper defines the round in prose: the scheduler advertises execution gaps (a time
 * window on a MIG slice of some capacity), every waiting job answers "interest" if a
 * subjob of its own would fit that window and capacity safely, the scheduler picks one
 * interested job per gap by its policy, and only the granted job materialises the subjob
 * (Section 3.5; admissibility test in Sections 3.8 and 3.9; greedy slot filling in
 * Section 4.2).  This library fixes that prose as integer arithmetic:
 *
 *   job j        steps i = 0..len_j-1 with duration d[i] (ms), memory envelope m[i] (MiB,
 *                the risk-adjusted envelope U of Section 3.9 sampled per step) and a
 *                safe-boundary bit s[i] (a checkpoint cut after step i, Section 3.7); the
 *                end of a job always counts as a boundary.  State: progress p_j (steps
 *                already granted) and ready_j (ms).
 *   gap g        (slice, start, T, C).
 *   signal       j is interested in g iff p_j < len_j, start_g >= ready_j and some
 *                k in (p_j, len_j] ends on a boundary with sum d[p_j..k) <= T_g and
 *                max m[p_j..k) <= C_g (all bounds inclusive).  Its subjob is the longest
 *                such k; dur = sum d, work = sum d*m over [p_j, k).
 *   score        EFFICIENCY work; FAIRNESS work * (1 + wait_j/1000) (truncating division);
 *                SLA (prio_j, work) compared lexicographically, larger prio more urgent;
 *                TIGHT_FIT max m over [p_j, k).
 *   select       per gap the interested job with the largest score, ties to the lowest job id.
 *   commit       a job that won several gaps accepts the one with the largest k, ties to
 *                the lowest gap id; p_j = k, ready_j = start_g + dur.
 *
 * All pointers are plain C pointers.  Every array argument is either a HOST pointer or a
 * DEVICE pointer on the context's device, as said by the `where` argument of the call.
 * The caller owns every buffer it passes; the library copies what it needs before the
 * call's work completes on the context's stream and never keeps a caller pointer.
 * Calls with device-memspace arguments are ordered on the context's stream and return
 * without waiting for the GPU, so that a round (sja_advertise, sja_select, sja_commit) can be
 * queued without a host round trip; the exceptions say so in their own comment (the loads
 * return validation results and therefore wait).  Calls with host-memspace arguments wait:
 * host inputs may be reused and host outputs are complete when the call returns.  Device
 * input arrays dur_ms, mem_MiB, safe_bits and power_W must be 16-byte aligned.
 *
 * No call aborts the process or traps the device.  Every call returns an sja_status;
 * sja_last_error() gives a text for the most recent failure on that context.
 * SJA_ERR_INVALID_ARG, SJA_ERR_BAD_PROFILE and SJA_ERR_STATE leave the context as it was.
 * After SJA_ERR_CUDA the context is unusable except for sja_destroy().
 * A context is not thread-safe; use one per host thread or lock around it.
 */
#ifndef SJA_H
#define SJA_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sja_ctx sja_ctx; /* opaque; owns all device memory it allocates */

typedef enum {
    SJA_OK = 0,
    SJA_ERR_INVALID_ARG = 1, /* NULL pointer, zero count, unknown policy, misaligned device array */
    SJA_ERR_BAD_PROFILE = 2, /* off[0] != 0, off not monotone, a job longer than 2^32-1 steps, progress > len */
    SJA_ERR_OVERFLOW = 3,    /* a job's total duration >= 2^32 ms, total work or a score too large, start + dur >= 2^32 */
    SJA_ERR_STATE = 4,       /* call order: select before advertise/load, commit before select or twice */
    SJA_ERR_OOM = 5,         /* device or host allocation failed */
    SJA_ERR_CUDA = 6,        /* a CUDA call failed; context poisoned */
    SJA_ERR_TIMEOUT = 7      /* reserved: no kernel of this library waits on another */
} sja_status;

typedef enum { SJA_MEM_HOST = 0, SJA_MEM_DEVICE = 1 } sja_memspace;

/* One advertised execution gap: a window in time on a slice of a given memory capacity (Section 3.5). 16 bytes. */
typedef struct {
    uint32_t slice;    /* MIG slice label; only sja_set_locality makes it count in scoring */
    uint32_t start_ms; /* absolute start of the window */
    uint32_t T_ms;     /* window length */
    uint32_t C_MiB;    /* slice memory capacity */
} sja_gap;

typedef enum {
    SJA_POLICY_EFFICIENCY = 0, /* score = work */
    SJA_POLICY_FAIRNESS = 1,   /* score = work * (1 + wait_ms/1000); needs wait_ms at load */
    SJA_POLICY_SLA = 2,        /* key = (prio, work); needs prio at load; reported score = work */
    SJA_POLICY_TIGHT_FIT = 3   /* score = peak memory (MiB) of the subjob: the job that leaves the least slack
                                  C - peak on the slice wins (slack-minimising principle of Section 3.9, applied
                                  by the scheduler across jobs); ties to the lowest job id */
} sja_policy_kind;

/* sja_policy.flags.  By default select runs the tile-sweep kernel over the gaps ordered by
 * (capacity, T), or the per-pair search for rounds of fewer than 65 536 pairs.  Bit 0:
 * evaluate every pair with the per-pair binary search over the boundary table.  Bit 1: use
 * the per-gap merge kernel.  Bit 2: use the tile-sweep kernel whatever the size.  Same
 * results on every path; the bits exist for testing and comparison (bit 0 wins over the
 * others, and an unsorted or many-capacity batch always takes the search). */
#define SJA_FLAG_FORCE_SEARCH 1u
#define SJA_FLAG_FORCE_MERGE 2u
#define SJA_FLAG_FORCE_TILE 4u

typedef struct {
    uint32_t kind;  /* sja_policy_kind */
    uint32_t flags; /* SJA_FLAG_* */
} sja_policy;

#define SJA_NO_JOB 0xFFFFFFFFu

/* The scheduler's decision for one gap (third protocol phase, Section 3.5). 24 bytes. */
typedef struct {
    uint32_t job;      /* winner, or SJA_NO_JOB (then end_step = dur_ms = score = 0) */
    uint32_t end_step; /* k: the subjob is steps [p_job, k) of the winner */
    uint32_t dur_ms;   /* its cumulative duration, <= T_ms */
    uint32_t granted;  /* 0 until sja_commit; then 1 iff the winner accepted this gap */
    uint64_t score;    /* policy score of the winner (work for SLA, peak memory in MiB for TIGHT_FIT) */
} sja_award;

/* Device times (CUDA events on the context's stream) accumulated while profiling is on. */
typedef struct {
    float scan_ms;      /* segmented prefix scan kernel (profile -> boundary table) */
    float prep_ms;      /* validation, row counting, row offsets and state initialisation of a load */
    float advertise_ms; /* gap upload and ordering */
    float select_ms;    /* feasibility + score + per-gap argmax kernels of sja_select */
    float commit_ms;    /* commit kernels */
    uint32_t scan_launches, prep_launches, advertise_launches, select_launches, commit_launches;
} sja_timing;

/*
 * Create a context on CUDA device `device`.  `cuda_stream` is a cudaStream_t (as void*)
 * all work is ordered on; NULL means the legacy default stream.  The stream stays the
 * caller's.  *out is set only on SJA_OK.
 */
sja_status sja_create(sja_ctx** out, int device, void* cuda_stream);

/* Free the context and every device buffer it owns.  NULL is accepted. */
sja_status sja_destroy(sja_ctx* ctx);

/*
 * Load J job profiles (ragged CSR) and run the segmented scan (the "on demand"
 * segmentation of Section 3.9: the envelope may be refined, so the scan is re-runnable;
 * a new load replaces the previous one and clears any advertised gaps, the deadlines of
 * sja_set_window_options and the trace of sja_load_power).
 *   off        u64[J+1], off[0] = 0, non-decreasing; job j owns steps [off[j], off[j+1]).
 *   dur_ms     u32[N], N = off[J]         per-step duration
 *   mem_MiB    u32[N]                     per-step memory envelope
 *   safe_bits  u32[ceil(N/32)]            bit (i % 32) of word (i / 32), LSB first
 *   ready_ms   u32[J]                     earliest start of each job
 *   progress   u32[J] or NULL (= all 0)   steps already granted; must be <= len_j
 *   wait_ms    u32[J] or NULL             needed for SJA_POLICY_FAIRNESS
 *   prio       u8[J]  or NULL             needed for SJA_POLICY_SLA
 * For each job the scan computes, at every safe end index k above its progress point, the
 * cumulative duration, the running maximum of the memory envelope (the window-max test of
 * Section 3.9), the maximum over the segment since the previous boundary, and the prefix
 * work sum d*m.  Waits for completion (it returns validation results).
 */
sja_status sja_load_profiles(sja_ctx* ctx, uint32_t J, const uint64_t* off,
                             const uint32_t* dur_ms, const uint32_t* mem_MiB,
                             const uint32_t* safe_bits, const uint32_t* ready_ms,
                             const uint32_t* progress, const uint32_t* wait_ms,
                             const uint8_t* prio, sja_memspace where);

/*
 * First protocol phase (Section 3.5): make G gaps visible to all jobs.  Replaces the
 * previous batch (also when the call fails after its argument checks: the context then has
 * no batch).  Gaps are taken as given (overlaps on a slice are not checked).  A device batch
 * is read when the stream gets there: keep it unchanged until then.
 */
sja_status sja_advertise(sja_ctx* ctx, uint32_t G, const sja_gap* gaps, sja_memspace where);

/*
 * Second and third phase (Section 3.5): every (gap, job) pair is tested for the longest
 * feasible subjob, interested jobs are scored under `policy`, one winner per gap is
 * chosen.  Does not change any job state (no subjob state exists before a grant).
 * `out` (G awards, in the order the gaps were advertised) may be NULL; the awards are
 * kept in the context either way.  May be called repeatedly.
 */
sja_status sja_select(sja_ctx* ctx, const sja_policy* policy, sja_award* out, sja_memspace where);

/*
 * sja_select for callers that must not allocate.  (The paper has no counterpart: this is
 * a deployment variant of the call above, with identical results.)
 *
 * Who needs it: a scheduler loop that runs where device allocation is off limits -- for
 * instance a service that handed all device memory to its own pool at start-up, so a
 * cudaMalloc from a library would fail or fragment it, or a latency-bound control loop that
 * cannot afford the device-wide synchronisation an allocation or free implies.  sja_select
 * grows a context buffer for its per-CTA candidate rows whenever a larger job or gap count
 * comes along; this call instead keeps those rows in a fixed array of
 * SJA_STATIC_SCRATCH_BYTES that is part of the library image.  It calls no cudaMalloc,
 * cudaFree or other allocating routine and records no profiling events.
 *
 * Cost and limit: every GPU on which the library is used holds the array until the process
 * exits.  The call needs ceil(J / 128) * G candidate slots of 16 bytes (one per gap and per
 * chunk of 128 jobs, the chunk of the per-pair search kernel, which runs or stands by in every
 * select); if that exceeds the array it returns SJA_ERR_INVALID_ARG with the numbers in
 * sja_last_error() and does nothing.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 * the context's device current); make that first call before starting any stream capture.
 * All contexts and all calls on one device share the one array.  It keeps whatever the last
 * call left in it; this call overwrites every slot it later reads, so no clearing is needed,
 * but two calls that overlap on the GPU (different streams or contexts on the same device)
 * race on it: serialise them.  Arguments, outputs, state rules and errors are otherwise those
 * of sja_select, and sja_commit / sja_get_awards follow it in the same way.
 */
#define SJA_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
sja_status sja_select_static(sja_ctx* ctx, const sja_policy* policy, sja_award* out, sja_memspace where);

/*
 * Grant (Section 3.5: only the selected job materialises its subjob; Sections 3.1, 3.5:
 * the parent job later resumes from the end of the fragment).  Resolves jobs that won
 * several gaps, advances progress and ready time of the granted jobs, refreshes their
 * running-maximum column.  `n_granted` is a HOST pointer or NULL; when given, the call
 * waits for completion.  One commit per select.
 */
sja_status sja_commit(sja_ctx* ctx, uint32_t* n_granted);

/*
 * sja_commit for a round in which some grants are not taken up: a subjob that failed or was
 * never started affects only itself, its parent job stays at the last completed fragment
 * (Section 3.10).  accept is u8[G] in the order the gaps were advertised; a gap with
 * accept[g] = 0 takes no part in the commit (its award keeps granted = 0, and a job that also
 * won an accepted gap is granted that one).  Otherwise identical to sja_commit.
 */
sja_status sja_commit_masked(sja_ctx* ctx, const uint8_t* accept, sja_memspace where, uint32_t* n_granted);

/*
 * One whole round with re-auction of orphaned gaps: sja_select + sja_commit, then again for
 * the gaps that had a winner but were not granted because that winner accepted another
 * gap, until no such gap is left, a pass grants nothing, or max_passes passes ran
 * (0 = no limit).  Jobs granted in an earlier pass of the call decline in later passes: one
 * subjob per job and round (one progress point per job, Sections 3.1 and 3.5).  Greedy slot
 * filling without lookahead is the paper's design (Section 4.2); the re-auction only keeps
 * it from wasting windows that further jobs had signalled interest in.
 * A pass-0-only call (max_passes = 1) equals sja_select followed by sja_commit.
 * The award of a gap (sja_get_awards) is the one of the last pass the gap took part in.
 * n_granted / n_passes are HOST pointers or NULL.  Waits for the GPU after every batch of up to 16 passes.
 * Uses up the advertised batch like sja_commit.
 */
sja_status sja_round_reauction(sja_ctx* ctx, const sja_policy* policy, uint32_t max_passes, uint32_t* n_granted,
                               uint32_t* n_passes);

/*
 * Subjob granularity guard (Section 4.3, item 5: minimum and maximum subjob duration thresholds
 * enforced at the framework level).  From the next select on, a subjob is a candidate only if
 * tau_min_ms <= its duration <= tau_max_ms, on top of the window and capacity bounds: the
 * longest subjob with duration <= min(T, tau_max) is taken, and the job declines if that one
 * is shorter than tau_min.  Defaults 0 and 0xFFFFFFFF switch the guard off.  Stays in force
 * until changed; tau_min_ms > tau_max_ms is SJA_ERR_INVALID_ARG.
 */
sja_status sja_set_duration_bounds(sja_ctx* ctx, uint32_t tau_min_ms, uint32_t tau_max_ms);

/*
 * Window options: two refinements of the window a (gap, job) pair sees, both off by default.
 *
 * late_start = 1: a job that becomes ready inside an advertised window may begin then instead
 * of declining: the subjob begins at max(start, ready_j), the job is eligible iff that is not
 * later than start + T, only the rest of the window counts (sum d <= T - (begin - start)),
 * and the commit sets ready_j = begin + dur.  (The paper leaves open whether a window has to
 * be taken from its first millisecond; the default is the strict reading.)
 *
 * deadline_ms (u32[J], or NULL for none; an entry of 0xFFFFFFFF means no deadline for that
 * job): deadline- and SLO-aware admission (Section 4.4, item 2: admit only subjobs whose
 * completion time stays below their deadline).  A candidate also needs
 * begin + sum d <= deadline_j; the tolerated risk of a violation lives in the per-step
 * durations, as the memory risk lives in the envelope.  The array is copied.
 *
 * With either option on, every select runs the per-pair search kernel (the usable window
 * then differs from pair to pair, which the ordered-gap kernels cannot follow); results obey
 * the same rules otherwise and sja_round_reauction / sja_commit_masked work unchanged.
 * Call after sja_load_profiles (a new load clears the deadlines and keeps late_start).  A
 * select that has not been committed yet is discarded by the call: select again before commit.
 */
sja_status sja_set_window_options(sja_ctx* ctx, uint32_t late_start, const uint32_t* deadline_ms, sja_memspace where);

/*
 * Hysteresis on slack gain (Section 3.9: against over-fragmentation by short-lived spikes, a further
 * subdivision is accepted only if it gains a minimum of slack; longer, more stable fragments are preferred
 * otherwise).  Reading taken here: let k_T be the longest subjob the window alone would allow (every rule but
 * the memory capacity) and k* the longest one that also fits the capacity.  k* < k_T means the capacity
 * forces the job to cut earlier -- a further subdivision -- and what the cut gains is the demand it sheds,
 * max m[p..k_T) - max m[p..k*).  With min_slack_gain_MiB > 0 the job signals interest in such a pair only if
 * that gain is at least the threshold; else it declines and keeps the longer fragment for a window it fits
 * whole.  0 (the default) switches the rule off; a forced cut always sheds at least 1 MiB, so 1 changes
 * nothing either.  Stays in force until changed.  With the rule on, every select runs the per-pair search
 * kernel.  A select that has not been committed yet is discarded by the call.
 */
sja_status sja_set_hysteresis(sja_ctx* ctx, uint32_t min_slack_gain_MiB);

/*
 * State- and locality-aware admission (Section 4.4, item 5; the Preference signal of Section 3.5: jobs declare
 * a predicted checkpoint size and a preference for the slice they ran on last, and admission penalises large
 * checkpoints and favours locality).
 *   ckpt_MiB    u32[J]  predicted checkpoint size of each job; NULL switches the feature off
 *   last_slice  u32[J]  slice label (sja_gap.slice) of the job's last fragment, 0xFFFFFFFF = has not run yet;
 *                       NULL = no job has run yet
 *   weight              score units charged per MiB of checkpoint that has to move
 * In a select, a job bidding for a gap on another slice than its last one has weight * ckpt_MiB_j taken off
 * its policy score (off the work for SJA_POLICY_SLA, whose class stays), not below zero: a zero score still
 * bids.  A gap on the same slice, and a job that has not run yet, pay nothing.  The reported score is the
 * lowered one.  sja_commit records the slice of the granted gap as the job's last slice;
 * sja_get_locality copies the current last slices out.  The arrays are copied; a new load drops them.  With
 * the feature on every select runs the per-pair search kernel.  sja_set_locality discards a select that has
 * not been committed yet.
 */
sja_status sja_set_locality(sja_ctx* ctx, const uint32_t* ckpt_MiB, const uint32_t* last_slice, uint32_t weight,
                            sja_memspace where);
sja_status sja_get_locality(sja_ctx* ctx, uint32_t* last_slice, sja_memspace where);

/*
 * One scheduler over several GPUs (the paper has no counterpart; the round itself is Section 3.5).  The jobs
 * are sharded over the GPUs in contiguous id ranges, the gaps are advertised on every GPU, every GPU selects
 * among its own jobs, and the only exchange of a round is one bid per gap and GPU:
 *
 *     sja_select(...)                                   on every GPU, over its shard
 *     sja_get_bids(ctx, job_base, rank, bids, ...)      its winner per gap with the totally ordered policy key
 *     all-gather of the G bids of every GPU             by the caller (e.g. NCCL), rank r at all[r * G]
 *     sja_reduce_bids(ctx, n, rank, all, accept, ...)   global winner per gap: largest key, lowest global job id
 *     sja_commit_masked(ctx, accept, ...)               the owner of a winner grants; the others grant nothing
 *
 * The result equals that of one GPU holding all jobs: the per-gap rule is the same argmax, and a job that won
 * several gaps resolves them on its owner.  job_base is the global id of the shard's first job; `rank` is
 * carried in the bids so that sja_reduce_bids can tell whose winner a gap's is.  sja_get_bids needs a select
 * that has not been committed; sja_reduce_bids needs the advertised batch (G).  global_awards may be NULL;
 * otherwise it receives the winning award per gap with global job ids (granted = 0).
 */
typedef struct {
    uint64_t key;      /* 0 = no interested job in this shard; else larger wins */
    uint32_t job;      /* global job id (job_base + local id), or SJA_NO_JOB */
    uint32_t end_step, dur_ms;
    uint32_t rank;     /* the GPU that made the bid */
    uint64_t score;
} sja_bid;             /* 32 bytes */
sja_status sja_get_bids(sja_ctx* ctx, uint32_t job_base, uint32_t rank, sja_bid* out, sja_memspace where);
sja_status sja_reduce_bids(sja_ctx* ctx, uint32_t n_ranks, uint32_t my_rank, const sja_bid* all, uint8_t* accept,
                           sja_award* global_awards, sja_memspace where);

/*
 * Power envelope, a second resource channel beside memory (Section 4.4, item 1: offers carry power caps,
 * subjobs answer with predicted power traces, and admission keeps max_t P(t) <= power_cap; as with memory,
 * the tolerated risk lives in the trace, which is a risk-adjusted envelope).
 *
 * sja_load_power: per-step predicted power in watts, u32[N], aligned step for step with the arrays given to
 * sja_load_profiles; `off` is the same CSR offset array again (the library does not keep it; a different
 * job length is SJA_ERR_BAD_PROFILE).  Builds, for every boundary row above the jobs' progress points, the
 * running maximum of the trace.  Call after sja_load_profiles, at any time between rounds; a new load
 * drops the trace.  Waits for completion.
 *
 * sja_advertise_power_caps: cap_W u32[G] for the batch just advertised, in the order of its gaps; an entry
 * of 0xFFFFFFFF, or cap_W = NULL, means no cap.  A new sja_advertise drops the caps.  With a trace loaded
 * and caps advertised, a candidate subjob also needs max power_W[p_j..k) <= cap_g, and every select runs
 * the per-pair search kernel (the cap differs from gap to gap inside a capacity class, which the
 * ordered-gap kernels cannot follow).  sja_commit keeps the running maximum current for granted jobs.
 * Both calls discard a select that has not been committed yet.
 */
sja_status sja_load_power(sja_ctx* ctx, const uint64_t* off, const uint32_t* power_W, sja_memspace where);
sja_status sja_advertise_power_caps(sja_ctx* ctx, const uint32_t* cap_W, sja_memspace where);

/*
 * Re-profile one job.  Segmentation happens on demand, at offer time, because the envelope U(t) can change
 * between offers as predictions improve (Section 3.9): this call replaces the per-step durations and memory values of
 * the steps job `job` has not been granted yet, steps p_job .. len_job - 1, n_steps = len_job - p_job of
 * them (SJA_ERR_BAD_PROFILE otherwise).  The job's safe boundaries stay where they are (a refined
 * prediction changes how long and how large a phase is, not where the checkpoints are), so only the
 * contents of the job's boundary rows are recomputed; no other job is touched and nothing is rescanned.
 * dur_ms / mem_MiB are u32[n_steps], host or device as `where` says, copied before the call returns.
 * SJA_ERR_OVERFLOW (total duration >= 2^32 ms or total work >= 2^63) leaves the job as it was.
 * Waits for completion.  A select that has not been committed yet is discarded: select again.
 */
sja_status sja_update_profile(sja_ctx* ctx, uint32_t job, uint32_t n_steps, const uint32_t* dur_ms,
                              const uint32_t* mem_MiB, sja_memspace where);

/* Copy the G awards of the last select (with `granted` set if it was committed). */
sja_status sja_get_awards(sja_ctx* ctx, sja_award* out, sja_memspace where);

/* Copy the per-job state: progress u32[J] and ready_ms u32[J] (either may be NULL). */
sja_status sja_get_state(sja_ctx* ctx, uint32_t* progress, uint32_t* ready_ms, sja_memspace where);

/* Number of rows of the boundary table built by the last load (sum over jobs). */
sja_status sja_scan_size(sja_ctx* ctx, uint64_t* n_boundaries);

/*
 * Copy out the scan result (any pointer may be NULL).  Row r of job j is at
 * boff[j] + r, r = 0 .. boff[j+1]-boff[j]-1, ascending in k:
 *   boff u64[J+1]; k u32 safe end index; D u32 cumulative duration of [p, k);
 *   M u32 max m[p_now..k) from the job's CURRENT progress point (rows below it are stale);
 *   S u32 max m over the segment since the previous boundary; W u64 sum d*m over [p, k).
 * D and W count from the progress point given at load.
 */
sja_status sja_get_scan(sja_ctx* ctx, uint64_t* boff, uint32_t* k, uint32_t* D, uint32_t* M,
                        uint32_t* S, uint64_t* W, sja_memspace where);

/* Per-kernel CUDA-event timing: 0 off, 1 every phase, 2 the scan kernel only (two event records per load
 * instead of about fourteen per round, for timing a whole step with little disturbance).  Resets the counters. */
sja_status sja_profile_enable(sja_ctx* ctx, int on);

/* Wait for the stream and read the accumulated kernel times. */
sja_status sja_profile_read(sja_ctx* ctx, sja_timing* out);

/* Text of the most recent error on this context ("" if none).  Owned by the context. */
const char* sja_last_error(const sja_ctx* ctx);

/*
 * Testing aid (the paper has no counterpart): host-side fault injection for the library's own device
 * allocations.  After the call, the nth time (counting from 1) that a context buffer has to grow, the
 * allocation is reported as failed (SJA_ERR_OOM) without being attempted; nth = 0 switches the injector off.
 * Nothing on the GPU is touched: the failure is made on the host, so that the error paths of the entry
 * points can be exercised without exhausting device memory.  A buffer whose growth fails keeps its old
 * block; an sja_advertise that fails leaves the context without a batch (select / commit then return
 * SJA_ERR_STATE) and with the loaded profiles intact.
 */
sja_status sja_debug_fail_alloc(sja_ctx* ctx, int nth);

#ifdef __cplusplus
}
#endif
#endif /* SJA_H */
