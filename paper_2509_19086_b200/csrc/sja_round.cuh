// Signal / score / select / commit kernels (protocol phases two and three, Section 3.5).
#pragma once
#include "sja_common.cuh"

namespace sja {

struct Gap { uint32_t slice, start, T, C; };                     // same layout as sja_gap
struct Award { uint32_t job, end_step, dur, granted; uint64_t score; };  // same layout as sja_award
struct __align__(16) Partial { uint64_t key; uint32_t job; uint32_t cnt; };

struct JobView {
    const uint64_t* boff;   // [J+1]
    const uint32_t* pb;     // rows consumed
    const uint32_t* Dp;     // D at the progress point
    const uint64_t* Wp;     // W at the progress point
    const uint32_t* ready;
    const uint32_t* wait;   // may be nullptr
    const uint8_t* prio;    // may be nullptr
    const uint4* A;
    const uint2* B;
    const uint32_t* blocked;  // may be nullptr; jobs with a non-zero entry decline every gap
    uint32_t tau_min, tau_max;  // subjob duration thresholds (Section 4.3, item 5); 0 / 0xFFFFFFFF = off
    const uint32_t* deadline;   // may be nullptr; per job, 0xFFFFFFFF = none (Section 4.4, item 2)
    uint32_t late_start;        // non-zero: a job that turns ready inside a window may begin then
    const uint2* PW;            // may be nullptr; per row {running max, segment max} of the power trace (Section 4.4, item 1)
    const uint32_t* caps;       // may be nullptr; per gap (caller's index) power cap, 0xFFFFFFFF = none
    uint32_t min_gain;          // hysteresis (Section 3.9): least slack gain that justifies a capacity-forced cut; 0 = off
    const uint32_t* ckpt;       // may be nullptr; per job predicted checkpoint size in MiB (Section 4.4, item 5)
    const uint32_t* last_slice; // with ckpt: per job the slice of its last fragment, 0xFFFFFFFF = has not run yet
    uint32_t loc_weight;        // score units per MiB of checkpoint that has to move to another slice
    const uint4* gaps_orig;     // the batch in the caller's order (the slice of a gap: ordered copies carry the index there)
    uint32_t J;
};

// What a select launch has to find out on the device before it does anything.  The host queues the kernels of a
// round without waiting for the GPU, so two facts may only exist in device memory when a kernel starts: how
// many gaps are left (a later pass of a re-auction: `gaps_left`), and how many capacity classes the ordered
// batch has (`n_classes`: with more than `max_classes` of them the ordered-gap kernels would restart their
// cursors too often, and the per-pair search serves the round instead; both kernels are queued and the one
// the count does not call for returns at once).
struct LaunchGate {
    const uint32_t* gaps_left;   // may be nullptr: all G gaps
    const uint32_t* n_classes;   // may be nullptr: this launch runs whatever the class count
    uint32_t max_classes;
    uint32_t run_if_many;        // 0: run when n_classes <= max_classes, 1: run when it is larger
    // Re-auction (several passes over a shrinking gap list inside one round): the candidate row of a job chunk
    // stays valid from pass to pass unless one of its jobs was granted, so only the chunks marked dirty are
    // evaluated again.  For that the rows are addressed by the gaps' original indices (stable while the list
    // is compacted) and have the full batch as their length.
    const uint32_t* dirty;       // may be nullptr (every chunk runs); else one word per block of 128 jobs
    uint32_t row_len;            // length of a candidate row; 0 = the G the launch was sized for
    uint32_t stable;             // non-zero: slot of a gap in a row = its original index, else its list position
};
constexpr uint32_t DIRTY_SHIFT = 7;   // jobs per dirty-flag block = 128 (every select kernel's chunk is a multiple)

// Number of gaps this launch serves: 0 when the class count calls for the other kernel.
__device__ __forceinline__ uint32_t gate_gaps(const LaunchGate& g, uint32_t G) {
    if (g.n_classes) {
        const bool many = *g.n_classes > g.max_classes;
        if (many != (g.run_if_many != 0u)) return 0u;
    }
    return g.gaps_left ? min(G, *g.gaps_left) : G;
}

// Does the chunk of `n` jobs from job `first` have to be evaluated in this launch?
__device__ __forceinline__ bool chunk_dirty(const LaunchGate& g, uint32_t first, uint32_t n) {
    if (!g.dirty) return true;
    bool any = false;
    for (uint32_t b = first >> DIRTY_SHIFT; b <= (first + n - 1u) >> DIRTY_SHIFT; ++b) any = any || g.dirty[b] != 0u;
    return any;
}

// Slot of (job chunk, gap) in the candidate rows: `pos` is the gap's position in the list of this launch, `orig`
// its original index.
__device__ __forceinline__ size_t row_slot(const LaunchGate& g, uint32_t G, uint32_t chunk, uint32_t pos, uint32_t orig) {
    return (size_t)chunk * (g.row_len ? g.row_len : G) + (g.stable ? orig : pos);
}

__device__ __forceinline__ uint32_t policy_factor(const JobView& jv, uint32_t kind, uint32_t j) {
    if (kind == 1) return 1u + __ldg(jv.wait + j) / 1000u;
    if (kind == 2) return (uint32_t)__ldg(jv.prio + j);
    return 0u;
}

// ---------------------------------------------------------------------------------------
// Per-pair search kernel.  Every (gap, job) pair is searched on its own: the number of the job's boundary rows
// that satisfy both monotone bounds (D - Dp <= T and running max <= C) is found by a binary search over the rows
// above the progress point, the last such row becomes a policy key, and the largest key per gap (ties: lowest job
// id) is the candidate.  Because nothing is carried from one pair to the next, this is also the kernel for
// everything that makes the test differ from pair to pair: a late start (the subjob begins at max(start, ready)
// and only the rest of the window counts), a deadline (it must be over by then), a power cap (a second running
// maximum), the hysteresis rule (a second search with the capacity lifted) and the locality penalty (the key
// depends on the gap's slice).
//
// Work split: a CTA stages the first SEARCH_ROWS rows of a chunk of jobs in shared memory (most windows end
// inside them; only longer answers continue in global memory) and owns a range of the gaps.  A THREAD owns a
// gap and walks the staged jobs in ascending id: all lanes of a warp look at the same job at the same time, so
// the job's constants are broadcast reads, the five probes of the lanes fall into the 32 banks of the job's
// 128-byte row block without conflict, and the running best of a gap lives in its thread's registers -- no
// reduction across lanes, no staging of candidates, one coalesced candidate row per CTA at the end.
constexpr int SEARCH_THREADS = 256;
#ifndef SJA_SEARCH_JOBS
#define SJA_SEARCH_JOBS 128
#endif
#ifndef SJA_SEARCH_ROWS
#define SJA_SEARCH_ROWS 16
#endif
#ifndef SJA_SEARCH_U
#define SJA_SEARCH_U 4
#endif
constexpr int SEARCH_U = SJA_SEARCH_U;                // jobs a thread has in flight
constexpr int SEARCH_JOBS = SJA_SEARCH_JOBS;          // most jobs a CTA stages (a launch may ask for fewer)
constexpr int SEARCH_GT = SEARCH_THREADS;             // granularity of a gap split: one gap per thread
constexpr int SEARCH_ROWS = SJA_SEARCH_ROWS;          // boundary rows staged per job (a power of two)
// per staged job: rows {D - Dp, M} and their policy payload, 14 words of constants; with power caps the rows'
// running power maxima as well
constexpr int SEARCH_JOB_WORDS = 14;
constexpr int SEARCH_SMEM_BYTES = SEARCH_JOBS * (SEARCH_ROWS * 16 + SEARCH_JOB_WORDS * 4);
constexpr int SEARCH_SMEM_BYTES_POWER = SEARCH_SMEM_BYTES + SEARCH_JOBS * SEARCH_ROWS * 4;
static_assert((SEARCH_ROWS & (SEARCH_ROWS - 1)) == 0 && SEARCH_ROWS == 16, "a half-warp stages the rows of one job");

// Policy key with the locality penalty taken off the score first (never below zero).
__device__ __forceinline__ uint64_t policy_key_less(uint32_t kind, uint64_t payload, uint32_t factor, uint64_t penalty) {
    uint64_t score = kind == 1 ? payload * (uint64_t)factor : payload;
    score -= min(score, penalty);
    return kind == 2 ? ((uint64_t)factor << KEY_SLA_SHIFT) + score + 1ull : score + 1ull;
}

// OPTS: something that differs from pair to pair is in force (compiled out otherwise).
// jobs_per_cta: jobs of one chunk (<= SEARCH_JOBS); the candidate row of chunk c is partial_out[c * G ...].
template <bool OPTS>
__global__ void __launch_bounds__(SEARCH_THREADS) select_search_kernel(
    JobView jv, const Gap* __restrict__ gaps, uint32_t G, uint32_t gaps_per_split, uint32_t kind,
    Partial* __restrict__ partial_out, LaunchGate gate, uint32_t jobs_per_cta) {
    dep_wait();
    dep_launch();
    const uint32_t G_now = gate_gaps(gate, G);   // gaps actually left
    if (blockIdx.y * gaps_per_split >= G_now) return;
    if (!chunk_dirty(gate, blockIdx.x * jobs_per_cta, jobs_per_cta)) return;   // its candidate row still stands
    extern __shared__ __align__(16) unsigned char search_smem[];
    uint2* sDM = reinterpret_cast<uint2*>(search_smem);                                   // [job][row] {D - Dp, M}
    uint2* sPay = sDM + SEARCH_JOBS * SEARCH_ROWS;                                        // [job][row] policy payload
    uint32_t* sJob = reinterpret_cast<uint32_t*>(sPay + SEARCH_JOBS * SEARCH_ROWS);       // [word][job] constants
    uint32_t* sPow = sJob + SEARCH_JOB_WORDS * SEARCH_JOBS;                               // [job][row], with power caps
    // words of sJob: 0 n, 1 ready, 2 factor, 3 deadline, 4 home slice, 5 Dp, 6-7 first row index, 8-9 Wp, 10-11 penalty
    const bool with_caps = OPTS && jv.PW != nullptr && jv.caps != nullptr;
    const bool with_locality = OPTS && jv.ckpt != nullptr && jv.last_slice != nullptr;
    const uint32_t min_gain = OPTS ? jv.min_gain : 0u;
    const bool late = OPTS && jv.late_start != 0u;
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    const uint32_t job0 = blockIdx.x * jobs_per_cta;
    const uint32_t n_jobs = min(jobs_per_cta, jv.J - job0);

    // ---- stage the chunk: a half-warp per job, one row per lane (a coalesced 256-byte read of the table)
    for (uint32_t jj = wid * 2u + (lane >> 4); jj < n_jobs; jj += (SEARCH_THREADS / 32) * 2u) {
        const uint32_t j = job0 + jj, r = lane & 15u;
        const uint64_t b0 = jv.boff[j], b1 = jv.boff[j + 1];
        const uint32_t pb = jv.pb[j];
        const uint64_t base = b0 + pb;
        uint32_t n = (uint32_t)(b1 - b0) - pb;
        if (jv.blocked && jv.blocked[j]) n = 0;
        const uint32_t Dp = jv.Dp[j];
        const uint64_t Wp = jv.Wp[j];
        // rows beyond the job's last one hold a sentinel that no window admits (T = C = 2^32-1 is clamped below)
        uint2 dm = make_uint2(0xFFFFFFFFu, 0xFFFFFFFFu), pay = make_uint2(0u, 0u);
        uint32_t pw = 0xFFFFFFFFu;
        if (r < n) {
            const uint4 row = __ldg(jv.A + base + r);
            const uint64_t pl = policy_payload(kind, row, Wp);
            dm = make_uint2(row.x - Dp, row.y);
            pay = make_uint2((uint32_t)pl, (uint32_t)(pl >> 32));
            if (with_caps) pw = __ldg(&jv.PW[base + r].x);
        }
        sDM[jj * SEARCH_ROWS + r] = dm;
        sPay[jj * SEARCH_ROWS + r] = pay;
        if (with_caps) sPow[jj * SEARCH_ROWS + r] = pw;
        if (r == 0) {
            uint64_t penalty = 0;
            uint32_t home = 0xFFFFFFFFu;
            if (with_locality) {
                home = jv.last_slice[j];
                penalty = (uint64_t)jv.loc_weight * (uint64_t)jv.ckpt[j];
            }
            sJob[0 * SEARCH_JOBS + jj] = n;
            sJob[1 * SEARCH_JOBS + jj] = jv.ready[j];
            sJob[2 * SEARCH_JOBS + jj] = policy_factor(jv, kind, j);
            sJob[3 * SEARCH_JOBS + jj] = (OPTS && jv.deadline) ? jv.deadline[j] : 0xFFFFFFFFu;
            sJob[4 * SEARCH_JOBS + jj] = home;
            sJob[5 * SEARCH_JOBS + jj] = Dp;
            sJob[6 * SEARCH_JOBS + jj] = (uint32_t)base;
            sJob[7 * SEARCH_JOBS + jj] = (uint32_t)(base >> 32);
            sJob[8 * SEARCH_JOBS + jj] = (uint32_t)Wp;
            sJob[9 * SEARCH_JOBS + jj] = (uint32_t)(Wp >> 32);
            sJob[10 * SEARCH_JOBS + jj] = (uint32_t)penalty;
            sJob[11 * SEARCH_JOBS + jj] = (uint32_t)(penalty >> 32);
        }
    }
    __syncthreads();

    const uint32_t g_begin = blockIdx.y * gaps_per_split;
    const uint32_t g_end = min(G_now, g_begin + gaps_per_split);
    for (uint32_t g = g_begin + threadIdx.x; g < g_end; g += SEARCH_THREADS) {
        const uint4 gq = __ldg(reinterpret_cast<const uint4*>(gaps) + g);
        const uint32_t start = gq.y, C = gq.w;
        // (the caller's gap index travels in the slice field of the ordered copy)
        const uint32_t cap = with_caps ? __ldg(jv.caps + gq.x) : 0xFFFFFFFFu;
        const uint32_t slice = with_locality ? __ldg(&jv.gaps_orig[gq.x].x) : 0u;
        uint64_t best_key = 0;
        uint32_t best_job = 0xFFFFFFFFu, best_cnt = 0;

        // SEARCH_U jobs are in flight per thread: their probe chains are independent, so the shared-memory latency
        // of one search hides behind the others.
        for (uint32_t j0 = 0; j0 < n_jobs; j0 += SEARCH_U) {
            uint32_t Tq[SEARCH_U], nq[SEARCH_U], lo[SEARCH_U];
            bool elig[SEARCH_U];
#pragma unroll
            for (int u = 0; u < SEARCH_U; ++u) {
                const uint32_t jj = min(j0 + (uint32_t)u, n_jobs - 1u);      // (a pass beyond the chunk repeats its last job, not eligible)
                const uint32_t n = sJob[0 * SEARCH_JOBS + jj];
                const uint32_t ready = sJob[1 * SEARCH_JOBS + jj];
                uint32_t T = gq.z;
                bool eligible = n != 0u && j0 + (uint32_t)u < n_jobs;
                if (OPTS) {
                    // the window this pair sees: what is left of the gap once the job can begin, cut at its deadline
                    const uint32_t deadline = sJob[3 * SEARCH_JOBS + jj];
                    uint32_t begin = start;
                    if (start < ready) {
                        const uint32_t late_by = ready - start;
                        if (!late || late_by > T) eligible = false;
                        begin = ready;
                        T -= min(late_by, T);
                    }
                    if (deadline != 0xFFFFFFFFu) {
                        if (begin > deadline) eligible = false;
                        T = min(T, deadline - min(begin, deadline));
                    }
                } else {
                    eligible = eligible && start >= ready;
                }
                Tq[u] = min(T, jv.tau_max);
                nq[u] = n;
                elig[u] = eligible;
                lo[u] = 0;
            }
            // does staged row idx of job jj fit a window of T ms under capacity Cx (and the gap's power cap)?
            auto fits = [&](uint32_t jj, uint32_t idx, uint32_t T, uint32_t Cx, uint32_t ns) -> bool {
                const uint2 r = sDM[jj * SEARCH_ROWS + idx];
                bool ok = r.x <= T && r.y <= Cx;
                if (OPTS && cap != 0xFFFFFFFFu && ok && idx < ns) ok = sPow[jj * SEARCH_ROWS + idx] <= cap;
                return ok;
            };
            // the probe chains, level by level: five probes per search, no branches
#pragma unroll
            for (uint32_t sp = SEARCH_ROWS / 2; sp > 0; sp >>= 1) {
#pragma unroll
                for (int u = 0; u < SEARCH_U; ++u) {
                    const uint32_t jj = min(j0 + (uint32_t)u, n_jobs - 1u);
                    lo[u] += fits(jj, lo[u] + sp - 1, Tq[u], C, min(nq[u], (uint32_t)SEARCH_ROWS)) ? sp : 0u;
                }
            }
#pragma unroll
            for (int u = 0; u < SEARCH_U; ++u) {
                const uint32_t jj = min(j0 + (uint32_t)u, n_jobs - 1u);
                const uint32_t n = nq[u], T = Tq[u];
                const uint32_t ns = min(n, (uint32_t)SEARCH_ROWS);
                // every staged row fits: rows ns, ns + 1, ns + 3, ... in global memory, then a binary search in the bracket
                auto continue_global = [&](uint32_t lo_, uint32_t Cx) -> uint32_t {
                    const uint64_t base = pack64(sJob[6 * SEARCH_JOBS + jj], sJob[7 * SEARCH_JOBS + jj]);
                    const uint32_t Dp = sJob[5 * SEARCH_JOBS + jj];
                    uint32_t hi = n, step = 1;
                    for (uint32_t idx = ns;;) {
                        if (idx >= n) { hi = n; break; }
                        const uint4 r = __ldg(jv.A + base + idx);
                        bool ok = r.x - Dp <= T && r.y <= Cx;
                        if (OPTS && ok && cap != 0xFFFFFFFFu) ok = __ldg(&jv.PW[base + idx].x) <= cap;
                        if (ok) { lo_ = idx + 1; idx += step; step <<= 1; }
                        else { hi = idx; break; }
                    }
                    while (lo_ < hi) {
                        const uint32_t mid = lo_ + ((hi - lo_) >> 1);
                        const uint4 r = __ldg(jv.A + base + mid);
                        bool ok = r.x - Dp <= T && r.y <= Cx;
                        if (OPTS && ok && cap != 0xFFFFFFFFu) ok = __ldg(&jv.PW[base + mid].x) <= cap;
                        if (ok) lo_ = mid + 1; else hi = mid;
                    }
                    return lo_;
                };
                uint32_t cnt = lo[u] + (fits(jj, lo[u], T, C, ns) ? 1u : 0u);
                cnt = elig[u] ? min(cnt, ns) : 0u;
                if (cnt == ns && ns < n && elig[u]) cnt = continue_global(cnt, C);
                if (cnt == 0u) continue;
                uint32_t dur, peak;
                uint64_t pay;
                if (cnt <= ns) {
                    const uint2 r = sDM[jj * SEARCH_ROWS + cnt - 1];
                    const uint2 pw = sPay[jj * SEARCH_ROWS + cnt - 1];
                    dur = r.x; peak = r.y;
                    pay = pack64(pw.x, pw.y);
                } else {
                    const uint64_t base = pack64(sJob[6 * SEARCH_JOBS + jj], sJob[7 * SEARCH_JOBS + jj]);
                    const uint4 r = __ldg(jv.A + base + cnt - 1);
                    dur = r.x - sJob[5 * SEARCH_JOBS + jj]; peak = r.y;
                    pay = policy_payload(kind, r, pack64(sJob[8 * SEARCH_JOBS + jj], sJob[9 * SEARCH_JOBS + jj]));
                }
                if (dur < jv.tau_min) continue;    // the longest fitting subjob is shorter than the minimum: decline
                if constexpr (OPTS) {
                    if (min_gain != 0u && cnt < n) {
                        // hysteresis: how far would the window alone let the job run (capacity lifted)?  If further,
                        // the capacity forces this cut, and it is taken only if it sheds at least min_gain MiB
                        uint32_t lt = 0;
#pragma unroll
                        for (uint32_t sp = SEARCH_ROWS / 2; sp > 0; sp >>= 1) lt += fits(jj, lt + sp - 1, T, 0xFFFFFFFFu, ns) ? sp : 0u;
                        lt += fits(jj, lt, T, 0xFFFFFFFFu, ns) ? 1u : 0u;
                        lt = min(lt, ns);
                        if (lt == ns && ns < n) lt = continue_global(lt, 0xFFFFFFFFu);
                        if (lt > cnt) {
                            uint32_t peak_t;
                            if (lt <= ns) peak_t = sDM[jj * SEARCH_ROWS + lt - 1].y;
                            else peak_t = __ldg(jv.A + pack64(sJob[6 * SEARCH_JOBS + jj], sJob[7 * SEARCH_JOBS + jj]) + lt - 1).y;
                            if (peak_t - peak < min_gain) continue;
                        }
                    }
                }
                const uint32_t factor = sJob[2 * SEARCH_JOBS + jj];
                uint64_t key;
                if (OPTS) {
                    uint64_t pen = 0;
                    const uint32_t home = sJob[4 * SEARCH_JOBS + jj];
                    if (with_locality && home != 0xFFFFFFFFu && home != slice)
                        pen = pack64(sJob[10 * SEARCH_JOBS + jj], sJob[11 * SEARCH_JOBS + jj]);
                    key = policy_key_less(kind, pay, factor, pen);
                } else {
                    key = policy_key(kind, pay, factor);
                }
                // jobs come in ascending id: only a larger key replaces the best, so ties stay with the lowest id
                if (key > best_key) { best_key = key; best_job = job0 + jj; best_cnt = cnt; }
            }
        }

        Partial pr;
        pr.key = best_key; pr.job = best_job; pr.cnt = best_cnt;
        partial_out[row_slot(gate, G, blockIdx.x, g, gq.x)] = pr;
    }
}

// ---------------------------------------------------------------------------------------
// Final reduction: fold the candidate rows of all CTAs into the award of every gap.  A CTA of 8 warps
// owns 32 consecutive gaps, one per lane, so that a warp reads 512 contiguous bytes of a candidate row;
// warp w folds rows w, w + 8, ..., then the 8 warps are folded through shared memory.
constexpr int FINALIZE_WARPS = 8;

__global__ void __launch_bounds__(FINALIZE_WARPS * 32) finalize_awards_kernel(
    JobView jv, const Partial* __restrict__ partial, uint32_t n_rows, uint32_t n_rows_many,
    const Gap* __restrict__ sgaps, uint32_t G, uint32_t kind, Award* __restrict__ awards, uint32_t* __restrict__ widx,
    LaunchGate gate) {
    dep_wait();
    dep_launch();
    __shared__ Partial fold[FINALIZE_WARPS][32];
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    const uint32_t g = blockIdx.x * 32u + lane;     // position in the advertised (sorted) order
    const uint32_t G_now = gate.gaps_left ? min(G, *gate.gaps_left) : G;   // G stays the row length of `partial`
    // the kernel that ran wrote one candidate row per job chunk of its own size
    if (gate.n_classes && *gate.n_classes > gate.max_classes) n_rows = n_rows_many;
    Partial best;
    best.key = 0; best.job = 0xFFFFFFFFu; best.cnt = 0;
    if (g < G_now) {
        const uint32_t slot = gate.stable ? sgaps[g].slice : g;
        const size_t row_len = gate.row_len ? gate.row_len : G;
        for (uint32_t r = wid; r < n_rows; r += FINALIZE_WARPS) {
            const Partial c = partial[(size_t)r * row_len + slot];
            if (c.key > best.key || (c.key == best.key && c.job < best.job)) best = c;
        }
    }
    fold[wid][lane] = best;
    __syncthreads();
    if (wid != 0 || g >= G_now) return;
#pragma unroll
    for (int w = 1; w < FINALIZE_WARPS; ++w) {
        const Partial c = fold[w][lane];
        if (c.key > best.key || (c.key == best.key && c.job < best.job)) best = c;
    }
    const uint32_t orig = sgaps[g].slice;   // caller's gap index
    Award a;
    if (best.key == 0) {
        a.job = 0xFFFFFFFFu; a.end_step = 0; a.dur = 0; a.granted = 0; a.score = 0;
        widx[orig] = 0;
    } else {
        const uint32_t j = best.job;
        const uint64_t row = jv.boff[j] + jv.pb[j] + best.cnt - 1;
        a.job = j;
        a.end_step = jv.B[row].x;
        a.dur = jv.A[row].x - jv.Dp[j];
        a.granted = 0;
        a.score = key_to_score(kind, best.key);
        widx[orig] = best.cnt;
    }
    awards[orig] = a;
}

// ---------------------------------------------------------------------------------------
// Commit, step 1: every winning job records the gap it accepts: largest end_step, then
// lowest gap id (one atomicMax on a packed key; the order of the atomics does not matter).
__device__ __forceinline__ void commit_vote_one(const Award* __restrict__ awards, uint32_t g,
                                                unsigned long long* __restrict__ jobwin,
                                                const uint8_t* __restrict__ accept) {
    if (accept && !accept[g]) return;   // grant not taken up (failed subjob): no part in the commit
    const uint32_t j = awards[g].job;
    if (j == 0xFFFFFFFFu || awards[g].granted) return;   // granted: settled in an earlier pass of this round
    const unsigned long long key = ((unsigned long long)awards[g].end_step << 32) | (0xFFFFFFFFu - g);
    atomicMax(jobwin + j, key);
}

__global__ void __launch_bounds__(256) commit_vote_kernel(const Award* __restrict__ awards, uint32_t G,
                                                          unsigned long long* __restrict__ jobwin,
                                                          uint32_t* __restrict__ n_granted,
                                                          const uint8_t* __restrict__ accept) {
    dep_wait();
    dep_launch();
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g == 0) *n_granted = 0;
    if (g >= G) return;
    commit_vote_one(awards, g, jobwin, accept);
}

// What the apply step works on (one struct, so that the stand-alone kernel and the re-auction's one-CTA kernel
// share the code).
struct CommitArgs {
    Award* awards; const Gap* gaps; const uint32_t* widx; unsigned long long* jobwin; const uint64_t* boff;
    uint4* A; const uint2* B; uint32_t *p, *ready, *pb, *Dp; uint64_t* Wp; uint32_t *winners, *n_granted, *flags;
    uint32_t* blocked; const uint8_t* accept; uint32_t late_start; uint32_t* last_slice; uint32_t* dirty_next;
    uint2* PW;
};

// Commit, step 2: the accepted gap of each job is granted and the job's state advances.
__device__ __forceinline__ void commit_apply_one(const CommitArgs& c, uint32_t g) {
    if (c.accept && !c.accept[g]) return;
    Award a = c.awards[g];
    if (a.job == 0xFFFFFFFFu || a.granted) return;   // granted: settled in an earlier pass of this round
    const unsigned long long key = ((unsigned long long)a.end_step << 32) | (0xFFFFFFFFu - g);
    if (c.jobwin[a.job] != key) { c.awards[g].granted = 0; return; }
    const uint32_t j = a.job;
    const uint32_t row_rel = c.pb[j] + c.widx[g] - 1;
    const uint4 r = c.A[c.boff[j] + row_rel];
    // the subjob began when the gap opened, or when the job turned ready inside it (late start)
    const uint32_t begin = c.late_start ? max(c.gaps[g].start, c.ready[j]) : c.gaps[g].start;
    const uint64_t new_ready = (uint64_t)begin + (uint64_t)a.dur;
    if (new_ready > 0xFFFFFFFFull) atomicOr(c.flags, FLAG_OVF_READY);
    c.awards[g].granted = 1;
    c.p[j] = a.end_step;
    c.ready[j] = new_ready > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)new_ready;
    c.pb[j] = row_rel + 1;
    c.Dp[j] = r.x;
    c.Wp[j] = pack64(r.z, r.w);
    if (c.blocked) c.blocked[j] = 1u;   // re-auction: one subjob per job and round
    if (c.dirty_next) c.dirty_next[j >> DIRTY_SHIFT] = 1u;   // ... and its chunk's candidates have to be found again
    if (c.last_slice) c.last_slice[j] = c.gaps[g].slice;   // where the job's state lives from now on (Section 4.4, item 5)
    c.winners[atomicAdd(c.n_granted, 1u)] = j;
}

__global__ void __launch_bounds__(256) commit_apply_kernel(CommitArgs c, uint32_t G) {
    dep_wait();
    dep_launch();
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= G) return;
    commit_apply_one(c, g);
}

// Commit, step 3: one warp per granted job rebuilds the running-maximum column from the
// new progress point (the maximum of a window is not derivable from the previous column),
// stopping as soon as the new and the old column agree, and clears the job's vote.
__device__ __forceinline__ void commit_refresh_one(uint32_t j, uint32_t lane, const uint64_t* __restrict__ boff,
                                                   const uint32_t* __restrict__ pb, uint4* __restrict__ A,
                                                   const uint2* __restrict__ B, unsigned long long* __restrict__ jobwin,
                                                   uint2* __restrict__ PW) {
    if (lane == 0) jobwin[j] = 0ull;
    const uint64_t base = boff[j] + pb[j];
    const uint32_t n = (uint32_t)(boff[j + 1] - base);
    uint32_t carry = 0;
    for (uint32_t c = 0; c < n; c += 32) {
        const uint32_t idx = c + lane;
        const bool ok = idx < n;
        uint32_t v = ok ? B[base + idx].y : 0u;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, v, o);
            if (lane >= (uint32_t)o) v = max(v, y);
        }
        v = max(v, carry);
        uint32_t* mcol = reinterpret_cast<uint32_t*>(A + base + idx) + 1;
        const uint32_t old = ok ? *mcol : 0u;
        if (ok && old != v) *mcol = v;
        const uint32_t last = min(31u, n - 1 - c);
        const uint32_t v_last = __shfl_sync(0xFFFFFFFFu, v, last);
        const uint32_t old_last = __shfl_sync(0xFFFFFFFFu, old, last);
        if (v_last == old_last) break;
        carry = v_last;
    }
    if (!PW) return;
    // the same for the running maximum of the power trace
    carry = 0;
    for (uint32_t c = 0; c < n; c += 32) {
        const uint32_t idx = c + lane;
        const bool ok = idx < n;
        const uint2 pw = ok ? PW[base + idx] : make_uint2(0u, 0u);
        uint32_t v = pw.y;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, v, o);
            if (lane >= (uint32_t)o) v = max(v, y);
        }
        v = max(v, carry);
        if (ok && pw.x != v) PW[base + idx].x = v;
        const uint32_t last = min(31u, n - 1 - c);
        const uint32_t v_last = __shfl_sync(0xFFFFFFFFu, v, last);
        const uint32_t old_last = __shfl_sync(0xFFFFFFFFu, pw.x, last);
        if (v_last == old_last) break;
        carry = v_last;
    }
}

__global__ void __launch_bounds__(256) commit_refresh_kernel(
    const uint32_t* __restrict__ winners, const uint32_t* __restrict__ n_granted, uint32_t G,
    const uint64_t* __restrict__ boff, const uint32_t* __restrict__ pb, uint4* __restrict__ A,
    const uint2* __restrict__ B, unsigned long long* __restrict__ jobwin, uint2* __restrict__ PW) {
    dep_wait();
    dep_launch();
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (w >= G || w >= *n_granted) return;
    commit_refresh_one(winners[w], lane, boff, pb, A, B, jobwin, PW);
}

}  // namespace sja

namespace sja {

// ---------------------------------------------------------------------------------------
// Advertise: order the gaps by (capacity, window length, index).  Gaps of one capacity form
// a "class" (the finite capacity set of Section 3.9); inside a class T ascends, so every
// job's answer moves monotonically along its boundary rows and the select kernels can walk
// instead of search.  The order is found by ranking against sorted tiles:
//   1. sort_gap_tiles_kernel: every CTA sorts one tile of 1024 keys in shared memory
//      (bitonic network; key = capacity:T, ties by index);
//   2. rank_gap_tiles_kernel: CTA (q, t) holds sorted tile t in shared memory and adds, for
//      each key of tile q, the number of smaller keys in tile t (a 10-probe binary search)
//      to that gap's rank -- G * G/1024 searches instead of G * G comparisons, no pass
//      waits on another;
//   3. place_gaps_kernel writes gap i to position rank[i]; its last CTA counts the positions whose predecessor has
//      another capacity (the class count, which decides between the ordered-gap kernels and the per-pair search).
constexpr uint32_t SORT_MAX_GAPS = 65536;
constexpr int SORT_TILE = 1024;

struct GapInfo { uint32_t n_classes; uint32_t placed_ctas; uint32_t pad[2]; };

__device__ __forceinline__ bool gap_key_less(uint64_t ka, uint32_t ia, uint64_t kb, uint32_t ib) {
    return ka < kb || (ka == kb && ia < ib);
}

// With `sorted_out` set (a batch of one tile) the kernel finishes the job alone: it writes the ordered gaps and
// the class count.  Otherwise it stores the sorted tile for the ranking pass and clears the ranks and the counter.
// `keep` (optional): the context's own copy of the batch, written here when the caller's array is read in place.
__global__ void __launch_bounds__(SORT_TILE) sort_gap_tiles_kernel(const Gap* __restrict__ gaps, uint32_t G,
                                                                   uint64_t* __restrict__ tile_key,
                                                                   uint32_t* __restrict__ tile_idx,
                                                                   uint32_t* __restrict__ rank, GapInfo* __restrict__ info,
                                                                   Gap* __restrict__ sorted_out, Gap* __restrict__ keep) {
    dep_wait();
    dep_launch();
    __shared__ uint64_t sk[SORT_TILE];
    __shared__ uint32_t si[SORT_TILE];
    const uint32_t t = threadIdx.x;
    const uint32_t i = blockIdx.x * SORT_TILE + t;
    uint64_t k = ~0ull;          // padding sorts last and is never smaller than a real key
    uint32_t x = 0xFFFFFFFFu;
    if (i < G) {
        const Gap g = gaps[i];
        k = ((uint64_t)g.C << 32) | g.T;
        x = i;
        if (keep) keep[i] = g;
    }
    if (i == 0) { info->n_classes = 0; info->placed_ctas = 0; }
    // Bitonic network, one element per thread.  Partners less than 32 apart sit in the same warp and are
    // exchanged by shuffles; only the wider strides go through shared memory (15 barrier stages, not 55).
    for (uint32_t size = 2; size <= SORT_TILE; size <<= 1) {
        const bool ascending = (t & size) == 0;
        for (uint32_t stride = size >> 1; stride >= 32; stride >>= 1) {
            sk[t] = k; si[t] = x;
            __syncthreads();
            const uint32_t p = t ^ stride;
            const uint64_t kp = sk[p];
            const uint32_t xp = si[p];
            // the lower position keeps the smaller key when ascending, the upper one the larger
            const bool partner_less = gap_key_less(kp, xp, k, x);
            const bool take = ((t & stride) == 0) == ascending ? partner_less : !partner_less;
            __syncthreads();
            if (take) { k = kp; x = xp; }
        }
        for (uint32_t stride = min(size >> 1, 16u); stride > 0; stride >>= 1) {
            const uint64_t kp = __shfl_xor_sync(0xFFFFFFFFu, k, stride);
            const uint32_t xp = __shfl_xor_sync(0xFFFFFFFFu, x, stride);
            const bool partner_less = gap_key_less(kp, xp, k, x);
            const bool take = ((t & stride) == 0) == ascending ? partner_less : !partner_less;
            if (take) { k = kp; x = xp; }
        }
    }
    sk[t] = k; si[t] = x;
    __syncthreads();
    if (sorted_out) {            // one tile: position t is final
        const uint32_t src = si[t];
        const bool real = src != 0xFFFFFFFFu;
        if (real) {
            const Gap g = gaps[src];     // (the caller's array: `keep` may not be complete yet for other threads' rows)
            Gap o;
            o.slice = src;       // the original position travels in the slice field
            o.start = g.start; o.T = g.T; o.C = g.C;
            sorted_out[t] = o;
        }
        const bool leader = real && (t == 0 || (uint32_t)(sk[t - 1] >> 32) != (uint32_t)(sk[t] >> 32));
        const uint32_t n = __syncthreads_count(leader);
        if (t == 0) info->n_classes = n;
        return;
    }
    tile_key[i] = sk[t];         // the arrays are padded to whole tiles
    tile_idx[i] = si[t];
    if (i < G) rank[i] = 0;
}

__global__ void __launch_bounds__(SORT_TILE) rank_gap_tiles_kernel(const uint64_t* __restrict__ tile_key,
                                                                   const uint32_t* __restrict__ tile_idx,
                                                                   uint32_t* __restrict__ rank) {
    dep_wait();
    dep_launch();
    __shared__ uint64_t sk[SORT_TILE];
    __shared__ uint32_t si[SORT_TILE];
    const uint32_t t = threadIdx.x;
    sk[t] = tile_key[blockIdx.y * SORT_TILE + t];
    si[t] = tile_idx[blockIdx.y * SORT_TILE + t];
    const uint64_t k = tile_key[blockIdx.x * SORT_TILE + t];
    const uint32_t x = tile_idx[blockIdx.x * SORT_TILE + t];
    __syncthreads();
    if (x == 0xFFFFFFFFu) return;   // padding
    uint32_t pos = 0;               // number of keys of tile blockIdx.y below (k, x)
#pragma unroll
    for (uint32_t s = SORT_TILE / 2; s > 0; s >>= 1) {
        if (gap_key_less(sk[pos + s - 1], si[pos + s - 1], k, x)) pos += s;
    }
    if (gap_key_less(sk[pos], si[pos], k, x)) pos += 1;
    if (pos) atomicAdd(rank + x, pos);
}

// Placement by rank; the CTA that finishes last then counts the capacity classes of the ordered list (positions
// whose predecessor has another capacity).  "Last" is decided by a counter that every CTA bumps after its own
// stores are visible: nobody waits for anybody.
__global__ void __launch_bounds__(256) place_gaps_kernel(const Gap* __restrict__ gaps, uint32_t G,
                                                         const uint32_t* __restrict__ rank, Gap* __restrict__ sorted,
                                                         GapInfo* __restrict__ info) {
    dep_wait();
    dep_launch();
    __shared__ uint32_t is_last;
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < G) {
        const Gap g = gaps[i];
        Gap o;
        o.slice = i;   // the original position travels in the slice field
        o.start = g.start; o.T = g.T; o.C = g.C;
        sorted[rank[i]] = o;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(&info->placed_ctas, 1u) == gridDim.x - 1u ? 1u : 0u;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // every thread takes a contiguous stretch of the list, eight independent loads in flight
    const uint32_t per = (G + blockDim.x - 1) / blockDim.x;
    const uint32_t q0 = threadIdx.x * per, q1 = min(G, q0 + per);
    uint32_t leaders = 0;
    uint32_t prev = (q0 > 0 && q0 < G) ? __ldcg(&sorted[q0 - 1].C) : 0u;
    for (uint32_t q = q0; q < q1; q += 8) {
        uint32_t cv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) cv[u] = (q + u < q1) ? __ldcg(&sorted[q + u].C) : 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (q + u < q1) {
                if (q + u == 0 || cv[u] != prev) ++leaders;
                prev = cv[u];
            }
        }
    }
    const uint32_t n = __reduce_add_sync(0xFFFFFFFFu, leaders);
    if ((threadIdx.x & 31u) == 0 && n) atomicAdd(&info->n_classes, n);
}

// Identity order (used when the batch is too large for the one-CTA sort).
__global__ void __launch_bounds__(256) copy_gaps_kernel(const Gap* __restrict__ gaps, uint32_t G,
                                                        Gap* __restrict__ sorted, Gap* __restrict__ keep) {
    dep_wait();
    dep_launch();
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= G) return;
    Gap g = gaps[i];
    if (keep) keep[i] = g;
    g.slice = i;
    sorted[i] = g;
}

// ---------------------------------------------------------------------------------------
// The commit of a re-auction pass and the compaction of its gap list in ONE launch of one CTA: votes of the
// gaps still in the list, barrier, grants, barrier, running-maximum refresh of the granted jobs (a warp each),
// then the compaction: the gaps that had a winner but were not granted (their winner accepted another gap) are kept,
// in their advertised order, for the next pass (a block-wide exclusive count per tile of 1024; report[0] receives the
// number of gaps kept, report[1] the grants of the pass, report[2] the status flag word and report[3] the number of
// gaps the pass started with, so that the host reads one 16-byte record per pass; G_dev (optional): that number
// lives in device memory).  A pass of a re-auction has at most a few thousand gaps and grants a
// handful of jobs, so four launches that are each bound by their start-up cost become one; every phase only reads
// what earlier phases of this same CTA wrote, so nothing waits on another CTA.
__global__ void __launch_bounds__(1024) reauction_resolve_kernel(CommitArgs c, const Gap* __restrict__ sgaps_in,
                                                                 uint32_t G_in, Gap* __restrict__ sgaps_out,
                                                                 uint32_t* __restrict__ report,
                                                                 const uint32_t* __restrict__ G_dev,
                                                                 uint32_t* __restrict__ dirty_done, uint32_t n_dirty) {
    dep_wait();
    dep_launch();
    if (G_dev) G_in = min(G_in, *G_dev);
    __shared__ uint32_t warp_cnt[32];
    __shared__ uint32_t tile_total;
    const uint32_t t = threadIdx.x, lane = t & 31u, wid = t >> 5;
    for (uint32_t i = t; i < n_dirty; i += blockDim.x) dirty_done[i] = 0u;   // flags this pass's select has consumed
    if (t == 0) *c.n_granted = 0;
    // (awards are stored at the gaps' original indices, which ride in the slice field of the ordered list)
    for (uint32_t i = t; i < G_in; i += blockDim.x) commit_vote_one(c.awards, sgaps_in[i].slice, c.jobwin, nullptr);
    __syncthreads();
    for (uint32_t i = t; i < G_in; i += blockDim.x) commit_apply_one(c, sgaps_in[i].slice);
    __syncthreads();
    const uint32_t n_won = *c.n_granted;
    for (uint32_t w = wid; w < n_won; w += blockDim.x / 32) commit_refresh_one(c.winners[w], lane, c.boff, c.pb, c.A, c.B, c.jobwin, c.PW);
    // keep, in order, the gaps that had a winner but were not granted
    uint32_t carry = 0;
    for (uint32_t base = 0; base < G_in; base += 1024) {
        const uint32_t i = base + t;
        Gap g;
        bool keep = false;
        if (i < G_in) {
            g = sgaps_in[i];
            const Award a = c.awards[g.slice];
            keep = a.job != 0xFFFFFFFFu && a.granted == 0u;
        }
        const uint32_t ball = __ballot_sync(0xFFFFFFFFu, keep);
        const uint32_t before = __popc(ball & ((1u << lane) - 1u));
        if (lane == 0) warp_cnt[wid] = __popc(ball);
        __syncthreads();
        if (wid == 0) {
            const uint32_t v = warp_cnt[lane];
            uint32_t inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                if (lane >= (uint32_t)o) inc += y;
            }
            warp_cnt[lane] = inc - v;
            if (lane == 31) tile_total = inc;
        }
        __syncthreads();
        if (keep) sgaps_out[carry + warp_cnt[wid] + before] = g;
        carry += tile_total;
        __syncthreads();
    }
    if (t == 0) { report[0] = carry; report[1] = G_in ? n_won : 0u; report[2] = *c.flags; report[3] = G_in; }
}

// ---------------------------------------------------------------------------------------
// Merge kernel.  Each lane owns MERGE_R jobs and walks the gaps of its CTA's range in the
// advertised order (capacity class, then T ascending).  Per job it keeps a cursor into the
// job's boundary rows above the progress point: the number w of rows that satisfy both
// bounds for the current gap.  Inside a class w only moves forward, so a pair costs one
// compare against the duration threshold of the next row ("thr", set to the largest u32
// when the next row is out of reach for this class) plus the key comparison.  The next
// rows of every job wait in a per-lane shared-memory ring that is refilled with 16-byte
// cp.async copies, so an advance never waits on global memory in the steady state.  All
// MERGE_R cursors of a lane advance inside ONE divergent region per gap.  Per gap the warp
// reduces its 32 x MERGE_R keys to one candidate (largest key, then lowest job id), the CTA
// folds its warps, and one candidate per (CTA, gap) goes to global memory.
#ifndef SJA_MERGE_WARPS
#define SJA_MERGE_WARPS 16
#endif
#ifndef SJA_MERGE_R
#define SJA_MERGE_R 2
#endif
#ifndef SJA_MERGE_RING
#define SJA_MERGE_RING 4
#endif
#ifndef SJA_MERGE_CTAS_PER_SM
#define SJA_MERGE_CTAS_PER_SM 2
#endif
constexpr int MERGE_WARPS = SJA_MERGE_WARPS;
constexpr int MERGE_R = SJA_MERGE_R;          // jobs per lane
constexpr int MERGE_RING = SJA_MERGE_RING;    // rows per lane-job ring (power of two)
constexpr int MERGE_CTAS_PER_SM = SJA_MERGE_CTAS_PER_SM;
#ifndef SJA_MERGE_GT
#define SJA_MERGE_GT 128
#endif
constexpr int MERGE_GT = SJA_MERGE_GT;        // gaps per staging tile
constexpr int MERGE_JOBS = MERGE_WARPS * MERGE_R * 32;
constexpr int MERGE_RING_BYTES = MERGE_WARPS * MERGE_R * MERGE_RING * 32 * 16;
constexpr int MERGE_SMEM_BYTES = MERGE_RING_BYTES + MERGE_GT * MERGE_WARPS * 16 + MERGE_GT * 16;
static_assert((MERGE_RING & (MERGE_RING - 1)) == 0, "ring size must be a power of two");
static_assert(MERGE_GT <= MERGE_WARPS * 32, "one thread per gap of a tile");

__device__ __forceinline__ void mg_cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void mg_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void mg_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 mg_lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr)
                 : "memory");
    return v;
}

// The u64 warp maximum as two 32-bit hardware reductions (high word, then low word among the
// lanes that hold the maximal high word).
struct WarpBest { uint64_t key; uint32_t writer; bool hit; };

__device__ __forceinline__ WarpBest warp_argmax_lowest_lane(uint64_t best, uint32_t lane) {
    WarpBest o;
    o.key = warp_max_u64(best);
    o.hit = (best == o.key) && (o.key != 0ull);
    const uint32_t ball = __ballot_sync(0xFFFFFFFFu, o.hit);
    o.writer = ball ? (uint32_t)(__ffs((int)ball) - 1) : 0u;   // lowest lane = lowest job id (lane-major jobs)
    o.hit = o.hit && (lane == o.writer);
    return o;
}

// BOUNDED: the subjob duration thresholds are in force (off by default, and then compiled out).
template <uint32_t KIND, bool BOUNDED>
__global__ void __launch_bounds__(MERGE_WARPS * 32, MERGE_CTAS_PER_SM) select_merge_kernel(
    JobView jv, const Gap* __restrict__ sgaps, uint32_t G, uint32_t gaps_per_split, Partial* __restrict__ partial_out,
    LaunchGate gate) {
    dep_wait();
    dep_launch();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (gate_gaps(gate, G) == 0u) return;      // the class count calls for the per-pair search
    if (!chunk_dirty(gate, blockIdx.x * MERGE_JOBS, MERGE_JOBS)) return;
    Partial* stage = reinterpret_cast<Partial*>(smem_raw + MERGE_RING_BYTES);            // [GT][WARPS]
    uint4* sg = reinterpret_cast<uint4*>(smem_raw + MERGE_RING_BYTES + MERGE_GT * MERGE_WARPS * 16);
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(smem_raw);

    // per lane-job state; job of (lane, r) = first job of the warp + lane * MERGE_R + r
    const uint4* next_row[MERGE_R];   // row w + MERGE_RING of the job: the next one to prefetch
    const uint4* row0[MERGE_R];
    uint64_t Wp[MERGE_R], nextW[MERGE_R], curKey[MERGE_R];
    uint32_t n[MERGE_R], Dp[MERGE_R], ready[MERGE_R], factor[MERGE_R];
    uint32_t w[MERGE_R];      // rows that satisfy both bounds for the current gap
    uint32_t thr[MERGE_R];    // duration of row w relative to the progress point, or 0xFFFFFFFF when closed
    uint32_t ring_s[MERGE_R];
    uint32_t open = 0;        // bit r: row w of job r exists and its running max fits the current class
    const uint32_t job0 = blockIdx.x * MERGE_JOBS + wid * MERGE_R * 32;   // first job of this warp
#pragma unroll
    for (int r = 0; r < MERGE_R; ++r) {
        const uint32_t j = job0 + lane * MERGE_R + r;
        ring_s[r] = smem_s + ((wid * MERGE_R + r) * MERGE_RING * 32 + lane) * 16;
        row0[r] = jv.A; next_row[r] = jv.A;
        Wp[r] = 0; nextW[r] = 0; curKey[r] = 0;
        n[r] = 0; Dp[r] = 0; ready[r] = 0xFFFFFFFFu; factor[r] = 0; w[r] = 0; thr[r] = 0xFFFFFFFFu;
        if (j < jv.J) {
            const uint64_t b0 = jv.boff[j], b1 = jv.boff[j + 1];
            const uint32_t pb = jv.pb[j];
            row0[r] = jv.A + b0 + pb;
            n[r] = (uint32_t)(b1 - b0) - pb;
            if (jv.blocked && jv.blocked[j]) n[r] = 0;
            Dp[r] = jv.Dp[j];
            Wp[r] = jv.Wp[j];
            ready[r] = jv.ready[j];
            factor[r] = policy_factor(jv, KIND, j);
        }
    }
    const uint32_t g_begin = blockIdx.y * gaps_per_split;
    const uint32_t g_end = min(G, g_begin + gaps_per_split);
    bool first = true;
    uint32_t curC = 0;

    // Cursor update and lane-local best candidate for one gap.
    auto eval_gap = [&](const uint4 gq, uint64_t& best, uint32_t& best_r, uint32_t& best_cnt) {
        const uint32_t start = gq.y, T = BOUNDED ? min(gq.z, jv.tau_max) : gq.z, C = gq.w;
        if (first || C != curC) {
            // new capacity class: T restarts from its smallest value, so do the cursors
            first = false;
            curC = C;
            mg_wait<0>();
#pragma unroll
            for (int r = 0; r < MERGE_R; ++r) {
                w[r] = 0;
                curKey[r] = 0;
#pragma unroll
                for (int i = 0; i < MERGE_RING; ++i) {
                    if ((uint32_t)i < n[r]) mg_cp_async16(ring_s[r] + i * 32 * 16, row0[r] + i);
                    mg_commit();
                }
                next_row[r] = row0[r] + MERGE_RING;
            }
            mg_wait<0>();
            open = 0;
#pragma unroll
            for (int r = 0; r < MERGE_R; ++r) {
                thr[r] = 0xFFFFFFFFu;
                if (n[r]) {
                    const uint4 row = mg_lds128(ring_s[r]);
                    nextW[r] = policy_payload(KIND, row, Wp[r]);
                    if (row.y <= C) { open |= 1u << r; thr[r] = row.x - Dp[r]; }
                }
            }
        }
        // one cheap test per job; the rare advances of all jobs of the lane share one region
        bool need = false;
#pragma unroll
        for (int r = 0; r < MERGE_R; ++r) need |= (T >= thr[r]);
        if (need) {
#pragma unroll
            for (int r = 0; r < MERGE_R; ++r) {
                while (((open >> r) & 1u) && T >= thr[r]) {
                    // row w qualifies: it becomes the candidate; fetch row w + 1 from the ring
                    // (a subjob shorter than the minimum duration is no candidate; longer rows may be)
                    curKey[r] = (!BOUNDED || thr[r] >= jv.tau_min) ? policy_key(KIND, nextW[r], factor[r]) : 0ull;
                    if (w[r] + MERGE_RING < n[r])
                        mg_cp_async16(ring_s[r] + (w[r] & (MERGE_RING - 1)) * 32 * 16, next_row[r]);
                    mg_commit();
                    ++next_row[r];
                    ++w[r];
                    open &= ~(1u << r);
                    thr[r] = 0xFFFFFFFFu;
                    if (w[r] < n[r]) {
                        mg_wait<MERGE_RING - 1>();
                        const uint4 row = mg_lds128(ring_s[r] + (w[r] & (MERGE_RING - 1)) * 32 * 16);
                        nextW[r] = policy_payload(KIND, row, Wp[r]);
                        if (row.y <= C) { open |= 1u << r; thr[r] = row.x - Dp[r]; }
                    }
                }
            }
        }
        // lane-local best over the MERGE_R jobs as a tournament (independent compares first);
        // on equal keys the lower r, i.e. the lower job id, stays
        uint64_t kk[MERGE_R];
        uint32_t rr[MERGE_R], cc[MERGE_R];
#pragma unroll
        for (int r = 0; r < MERGE_R; ++r) {
            kk[r] = (start >= ready[r]) ? curKey[r] : 0ull;
            rr[r] = (uint32_t)r;
            cc[r] = w[r];
        }
#pragma unroll
        for (int span = 1; span < MERGE_R; span <<= 1) {
#pragma unroll
            for (int r = 0; r + span < MERGE_R; r += 2 * span) {
                if (kk[r + span] > kk[r]) { kk[r] = kk[r + span]; rr[r] = rr[r + span]; cc[r] = cc[r + span]; }
            }
        }
        best = kk[0]; best_r = rr[0]; best_cnt = cc[0];
    };
    auto publish = [&](const WarpBest& wb, uint32_t gi, uint32_t br, uint32_t bc) {
        if (wb.key == 0ull) {
            if (lane == 0) { Partial pr; pr.key = 0; pr.job = 0xFFFFFFFFu; pr.cnt = 0; stage[gi * MERGE_WARPS + wid] = pr; }
        } else if (wb.hit) {
            Partial pr; pr.key = wb.key; pr.job = job0 + lane * MERGE_R + br; pr.cnt = bc;
            stage[gi * MERGE_WARPS + wid] = pr;
        }
    };

    for (uint32_t g0 = g_begin; g0 < g_end; g0 += MERGE_GT) {
        const uint32_t gt = min((uint32_t)MERGE_GT, g_end - g0);
        if (threadIdx.x < gt) sg[threadIdx.x] = __ldg(reinterpret_cast<const uint4*>(sgaps) + g0 + threadIdx.x);
        __syncthreads();
        // two gaps per iteration: their warp reductions are independent and overlap
        for (uint32_t gi = 0; gi < gt; gi += 2) {
            uint64_t bestA, bestB = 0;
            uint32_t rA, cA, rB = 0, cB = 0;
            eval_gap(sg[gi], bestA, rA, cA);
            const bool two = gi + 1 < gt;
            if (two) eval_gap(sg[gi + 1], bestB, rB, cB);
            const WarpBest wa = warp_argmax_lowest_lane(bestA, lane);
            const WarpBest wb = warp_argmax_lowest_lane(bestB, lane);
            publish(wa, gi, rA, cA);
            if (two) publish(wb, gi + 1, rB, cB);
        }
        __syncthreads();
        if (threadIdx.x < gt) {
            Partial bestp = stage[threadIdx.x * MERGE_WARPS];
#pragma unroll
            for (int ww = 1; ww < MERGE_WARPS; ++ww) {
                const Partial c = stage[threadIdx.x * MERGE_WARPS + ww];
                if (c.key > bestp.key || (c.key == bestp.key && c.job < bestp.job)) bestp = c;
            }
            partial_out[row_slot(gate, G, blockIdx.x, g0 + threadIdx.x, sg[threadIdx.x].x)] = bestp;
        }
        __syncthreads();
    }
    mg_wait<0>();
}

}  // namespace sja
