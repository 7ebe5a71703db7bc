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
    uint32_t J;
};

__device__ __forceinline__ uint32_t policy_factor(const JobView& jv, uint32_t kind, uint32_t j) {
    if (kind == 1) return 1u + __ldg(jv.wait + j) / 1000u;
    if (kind == 2) return (uint32_t)__ldg(jv.prio + j);
    return 0u;
}

// ---------------------------------------------------------------------------------------
// Per-pair search kernel.  One thread owns one job and visits every gap of its gap range;
// for each pair it finds the number of boundary rows that satisfy both monotone bounds
// (D - Dp <= T and running max <= C) with a galloping + binary search over the rows above
// the progress point, turns the last such row into a policy key, and the warp reduces the
// 32 keys to one candidate per gap (largest key, then lowest job id).
constexpr int SEARCH_THREADS = 256;
constexpr int SEARCH_GT = 64;   // gaps per staging tile

__global__ void __launch_bounds__(SEARCH_THREADS) select_search_kernel(
    JobView jv, const Gap* __restrict__ gaps, uint32_t G, uint32_t gaps_per_split, uint32_t kind,
    const uint32_t* __restrict__ job_list, uint32_t n_list, Partial* __restrict__ partial_out) {
    __shared__ Partial stage[SEARCH_GT][SEARCH_THREADS / 32];
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    const uint32_t slot = blockIdx.x * SEARCH_THREADS + threadIdx.x;
    // the jobs of this launch: either all jobs (job_list == nullptr) or a list of job ids
    const uint32_t n_jobs = job_list ? n_list : jv.J;
    uint32_t j = SJA_NO_JOB_DEV;
    if (slot < n_jobs) j = job_list ? job_list[slot] : slot;

    uint64_t base = 0, Wp = 0;
    uint32_t n = 0, Dp = 0, ready = 0, factor = 0;
    if (j != SJA_NO_JOB_DEV) {
        const uint64_t b0 = jv.boff[j], b1 = jv.boff[j + 1];
        const uint32_t pb = jv.pb[j];
        base = b0 + pb;
        n = (uint32_t)(b1 - b0) - pb;
        Dp = jv.Dp[j];
        Wp = jv.Wp[j];
        ready = jv.ready[j];
        factor = policy_factor(jv, kind, j);
    }
    const uint32_t g_begin = blockIdx.y * gaps_per_split;
    const uint32_t g_end = min(G, g_begin + gaps_per_split);

    for (uint32_t g0 = g_begin; g0 < g_end; g0 += SEARCH_GT) {
        const uint32_t gt = min((uint32_t)SEARCH_GT, g_end - g0);
        for (uint32_t gi = 0; gi < gt; ++gi) {
            const uint4 gq = __ldg(reinterpret_cast<const uint4*>(gaps) + g0 + gi);
            const uint32_t start = gq.y, T = gq.z, C = gq.w;
            uint32_t cnt = 0;
            uint64_t key = 0;
            if (n != 0 && start >= ready) {
                uint32_t lo = 0, hi = n, idx = 0;
                for (;;) {   // gallop over rows 0, 1, 3, 7, ...
                    if (idx >= n) { hi = n; break; }
                    const uint4 r = __ldg(jv.A + base + idx);
                    if (r.x - Dp <= T && r.y <= C) { lo = idx + 1; idx = idx * 2 + 1; }
                    else { hi = idx; break; }
                }
                while (lo < hi) {
                    const uint32_t mid = lo + ((hi - lo) >> 1);
                    const uint4 r = __ldg(jv.A + base + mid);
                    if (r.x - Dp <= T && r.y <= C) lo = mid + 1; else hi = mid;
                }
                cnt = lo;
                if (cnt) {
                    const uint4 r = __ldg(jv.A + base + cnt - 1);
                    key = policy_key(kind, pack64(r.z, r.w) - Wp, factor);
                }
            }
            const uint64_t mk = warp_max_u64(key);
            const uint32_t jmin = __reduce_min_sync(0xFFFFFFFFu, (key == mk && key != 0) ? j : 0xFFFFFFFFu);
            const uint32_t src = __ffs(__ballot_sync(0xFFFFFFFFu, key == mk && j == jmin)) - 1;
            const uint32_t wcnt = __shfl_sync(0xFFFFFFFFu, cnt, src & 31u);
            if (lane == 0) {
                Partial pr;
                pr.key = mk; pr.job = jmin; pr.cnt = mk ? wcnt : 0u;
                stage[gi][wid] = pr;
            }
        }
        __syncthreads();
        if (threadIdx.x < gt) {
            Partial best = stage[threadIdx.x][0];
#pragma unroll
            for (int w = 1; w < SEARCH_THREADS / 32; ++w) {
                const Partial c = stage[threadIdx.x][w];
                if (c.key > best.key || (c.key == best.key && c.job < best.job)) best = c;
            }
            partial_out[(size_t)blockIdx.x * G + g0 + threadIdx.x] = best;
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------
// Final reduction: one thread per gap folds the candidate rows of all CTAs into the award.
__global__ void __launch_bounds__(256) finalize_awards_kernel(
    JobView jv, const Partial* __restrict__ partial, uint32_t n_rows, uint32_t G, uint32_t kind,
    Award* __restrict__ awards, uint32_t* __restrict__ widx) {
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= G) return;
    Partial best;
    best.key = 0; best.job = 0xFFFFFFFFu; best.cnt = 0;
    for (uint32_t r = 0; r < n_rows; ++r) {
        const Partial c = partial[(size_t)r * G + g];
        if (c.key > best.key || (c.key == best.key && c.job < best.job)) best = c;
    }
    Award a;
    if (best.key == 0) {
        a.job = 0xFFFFFFFFu; a.end_step = 0; a.dur = 0; a.granted = 0; a.score = 0;
        widx[g] = 0;
    } else {
        const uint32_t j = best.job;
        const uint64_t row = jv.boff[j] + jv.pb[j] + best.cnt - 1;
        a.job = j;
        a.end_step = jv.B[row].x;
        a.dur = jv.A[row].x - jv.Dp[j];
        a.granted = 0;
        a.score = key_to_score(kind, best.key);
        widx[g] = best.cnt;
    }
    awards[g] = a;
}

// ---------------------------------------------------------------------------------------
// Commit, step 1: every winning job records the gap it accepts: largest end_step, then
// lowest gap id (one atomicMax on a packed key; the order of the atomics does not matter).
__global__ void __launch_bounds__(256) commit_vote_kernel(const Award* __restrict__ awards, uint32_t G,
                                                          unsigned long long* __restrict__ jobwin,
                                                          uint32_t* __restrict__ n_granted) {
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g == 0) *n_granted = 0;
    if (g >= G) return;
    const uint32_t j = awards[g].job;
    if (j == 0xFFFFFFFFu) return;
    const unsigned long long key = ((unsigned long long)awards[g].end_step << 32) | (0xFFFFFFFFu - g);
    atomicMax(jobwin + j, key);
}

// Commit, step 2: the accepted gap of each job is granted and the job's state advances.
__global__ void __launch_bounds__(256) commit_apply_kernel(
    Award* __restrict__ awards, const Gap* __restrict__ gaps, const uint32_t* __restrict__ widx, uint32_t G,
    const unsigned long long* __restrict__ jobwin, const uint64_t* __restrict__ boff, const uint4* __restrict__ A,
    uint32_t* __restrict__ p, uint32_t* __restrict__ ready, uint32_t* __restrict__ pb, uint32_t* __restrict__ Dp,
    uint64_t* __restrict__ Wp, uint32_t* __restrict__ winners, uint32_t* __restrict__ n_granted,
    uint32_t* __restrict__ flags) {
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= G) return;
    Award a = awards[g];
    if (a.job == 0xFFFFFFFFu) return;
    const unsigned long long key = ((unsigned long long)a.end_step << 32) | (0xFFFFFFFFu - g);
    if (jobwin[a.job] != key) { awards[g].granted = 0; return; }
    const uint32_t j = a.job;
    const uint32_t row_rel = pb[j] + widx[g] - 1;
    const uint4 r = A[boff[j] + row_rel];
    const uint64_t new_ready = (uint64_t)gaps[g].start + (uint64_t)a.dur;
    if (new_ready > 0xFFFFFFFFull) atomicOr(flags, FLAG_OVF_READY);
    awards[g].granted = 1;
    p[j] = a.end_step;
    ready[j] = new_ready > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)new_ready;
    pb[j] = row_rel + 1;
    Dp[j] = r.x;
    Wp[j] = pack64(r.z, r.w);
    winners[atomicAdd(n_granted, 1u)] = j;
}

// Commit, step 3: one warp per granted job rebuilds the running-maximum column from the
// new progress point (the maximum of a window is not derivable from the previous column),
// stopping as soon as the new and the old column agree, and clears the job's vote.
__global__ void __launch_bounds__(256) commit_refresh_kernel(
    const uint32_t* __restrict__ winners, const uint32_t* __restrict__ n_granted, uint32_t G,
    const uint64_t* __restrict__ boff, const uint32_t* __restrict__ pb, uint4* __restrict__ A,
    const uint2* __restrict__ B, unsigned long long* __restrict__ jobwin) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (w >= G || w >= *n_granted) return;
    const uint32_t j = winners[w];
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
}

}  // namespace sja
