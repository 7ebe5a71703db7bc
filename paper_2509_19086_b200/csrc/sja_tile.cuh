// Tile-sweep select kernel (protocol phases two and three, Section 3.5).
//
// Same result as the merge kernel, far fewer instructions per (gap, job) pair.  A warp owns
// 32 jobs (one cursor per lane, as in the merge kernel) but meets the ordered gaps 32 at a
// time, one gap per lane.  Inside a run of gaps of one capacity class with windows
// T_lo <= ... <= T_hi the answer for a gap splits in two parts:
//
//  * base: every row a job's cursor has passed qualifies for ALL gaps of the run (its
//    duration is <= T_lo).  The warp keeps these per-job candidates ordered by the jobs'
//    ready times and prefix-maximised ("PM": entry r = best candidate among the r+1 jobs
//    that become ready first).  A gap's eligible jobs (ready <= start, Section 3.5: the
//    window must not begin before the job can) are a prefix of that order, so its base
//    answer is ONE lookup, PM[#eligible - 1] -- no per-job work at all.
//  * events: rows whose duration lies in (T_lo, T_hi].  The owning lanes step their
//    cursors (all lanes that have one step together) and post (duration, ready, key) to
//    shared memory; every gap lane tests each posted event with two compares and a key
//    comparison.  An event is looked at once, by one warp instruction stream.
//
// The cost is therefore per (warp, 32 gaps) a fixed part (PM rebuild, lookup) plus a part
// proportional to the number of boundary rows the windows actually reach, not to the
// number of pairs.
#pragma once
#include "sja_round.cuh"

namespace sja {

#ifndef SJA_TILE_WARPS
#define SJA_TILE_WARPS 16
#endif
#ifndef SJA_TILE_CTAS_PER_SM
#define SJA_TILE_CTAS_PER_SM 2
#endif
#ifndef SJA_TILE_RING
#define SJA_TILE_RING 4
#endif
#ifndef SJA_TILE_GT
#define SJA_TILE_GT 128
#endif
constexpr int TILE_WARPS = SJA_TILE_WARPS;
constexpr int TILE_CTAS_PER_SM = SJA_TILE_CTAS_PER_SM;
constexpr int TILE_RING = SJA_TILE_RING;     // rows per job ring (power of two)
constexpr int TILE_GT = SJA_TILE_GT;         // gaps per staging tile (multiple of 32)
constexpr int TILE_JOBS = TILE_WARPS * 32;
constexpr int TILE_RING_BYTES = TILE_WARPS * TILE_RING * 32 * 16;
constexpr int TILE_STAGE_BYTES = TILE_WARPS * TILE_GT * 16;
constexpr int TILE_GAP_BYTES = TILE_GT * 16;
constexpr int TILE_EVENT_BYTES = TILE_WARPS * 32 * 16;   // posted events, one slot per lane
constexpr int TILE_ECNT_BYTES = TILE_WARPS * 32 * 4;     // their row counts
constexpr int TILE_PM_BYTES = TILE_WARPS * 32 * 16;      // rank-ordered candidates before the scan
constexpr int TILE_SMEM_BYTES =
    TILE_RING_BYTES + TILE_STAGE_BYTES + TILE_GAP_BYTES + TILE_EVENT_BYTES + TILE_ECNT_BYTES + TILE_PM_BYTES;
static_assert((TILE_RING & (TILE_RING - 1)) == 0, "ring size must be a power of two");
static_assert(TILE_GT % 32 == 0 && TILE_GT <= TILE_JOBS, "one thread per gap of a staging tile");

// Candidate order: larger key first, then the lower job id.
__device__ __forceinline__ bool cand_better(uint64_t ka, uint32_t ja, uint64_t kb, uint32_t jb) {
    return ka > kb || (ka == kb && ja < jb);
}

template <uint32_t KIND, bool BOUNDED>
__global__ void __launch_bounds__(TILE_WARPS * 32, TILE_CTAS_PER_SM) select_tile_kernel(
    JobView jv, const Gap* __restrict__ sgaps, uint32_t G, uint32_t gaps_per_split, Partial* __restrict__ partial_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(smem_raw);
    Partial* stage = reinterpret_cast<Partial*>(smem_raw + TILE_RING_BYTES);                       // [WARPS][GT]
    const uint4* sg = reinterpret_cast<const uint4*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES);
    uint4* sg_w = reinterpret_cast<uint4*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES);
    uint4* ev = reinterpret_cast<uint4*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES + TILE_GAP_BYTES) + wid * 32;
    uint32_t* evc = reinterpret_cast<uint32_t*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES + TILE_GAP_BYTES +
                                                TILE_EVENT_BYTES) + wid * 32;
    uint4* pm_s = reinterpret_cast<uint4*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES + TILE_GAP_BYTES +
                                           TILE_EVENT_BYTES + TILE_ECNT_BYTES) + wid * 32;
    const uint32_t ring_s = smem_s + (wid * TILE_RING * 32 + lane) * 16;   // slot i of the ring: + i * 512

    // ---- the lane's job
    const uint32_t job0 = blockIdx.x * TILE_JOBS + wid * 32;
    const uint32_t j = job0 + lane;
    const uint4* row0 = jv.A;
    const uint4* next_row = jv.A;
    uint64_t Wp = 0, nextW = 0, curKey = 0;
    uint32_t n = 0, Dp = 0, ready = 0xFFFFFFFFu, factor = 0;
    if (j < jv.J) {
        const uint64_t b0 = jv.boff[j], b1 = jv.boff[j + 1];
        const uint32_t pb = jv.pb[j];
        row0 = jv.A + b0 + pb;
        n = (uint32_t)(b1 - b0) - pb;
        if (jv.blocked && jv.blocked[j]) n = 0;
        Dp = jv.Dp[j];
        Wp = jv.Wp[j];
        ready = jv.ready[j];
        factor = policy_factor(jv, KIND, j);
    }
    uint32_t w = 0;                  // rows passed: they satisfy both bounds for every gap from here on
    uint32_t thr = 0xFFFFFFFFu;      // duration of row w relative to the progress point
    bool open = false;               // row w exists and its running maximum fits the current class

    // ---- the warp's jobs in order of their ready times (fixed for the whole kernel)
    uint32_t rank = 0;
#pragma unroll 8
    for (uint32_t l = 0; l < 32; ++l) {
        const uint32_t rl = __shfl_sync(0xFFFFFFFFu, ready, l);
        rank += (rl < ready || (rl == ready && l < lane)) ? 1u : 0u;
    }
    pm_s[rank] = make_uint4(ready, j, 0u, 0u);
    __syncwarp();
    const uint32_t sready = pm_s[lane].x;   // ready time of the job of rank `lane`
    const uint32_t sjob = pm_s[lane].y;     // and its id
    __syncwarp();
    const uint32_t sready_last = __shfl_sync(0xFFFFFFFFu, sready, 31);
    uint64_t pk = 0;                 // PM entry of rank `lane`: key, job, row count
    uint32_t pj = 0xFFFFFFFFu, pc = 0;

    const uint32_t g_begin = blockIdx.y * gaps_per_split;
    const uint32_t g_end = min(G, g_begin + gaps_per_split);
    bool have_class = false, dirty = true;
    uint32_t curC = 0;

    // One cursor step of this lane: row w becomes the job's candidate, row w + 1 is fetched.
    auto step_cursor = [&](uint32_t C) {
        curKey = (!BOUNDED || thr >= jv.tau_min) ? policy_key(KIND, nextW - Wp, factor) : 0ull;
        if (w + TILE_RING < n) mg_cp_async16(ring_s + (w & (TILE_RING - 1)) * 512, next_row);
        mg_commit();
        ++next_row;
        ++w;
        open = false;
        thr = 0xFFFFFFFFu;
        if (w < n) {
            mg_wait<TILE_RING - 1>();
            const uint4 row = mg_lds128(ring_s + (w & (TILE_RING - 1)) * 512);
            nextW = pack64(row.z, row.w);
            if (row.y <= C) { open = true; thr = row.x - Dp; }
        }
    };

    for (uint32_t g0 = g_begin; g0 < g_end; g0 += TILE_GT) {
        const uint32_t gt = min((uint32_t)TILE_GT, g_end - g0);
        if (threadIdx.x < gt) sg_w[threadIdx.x] = __ldg(reinterpret_cast<const uint4*>(sgaps) + g0 + threadIdx.x);
        __syncthreads();
        for (uint32_t sub = 0; sub < gt; sub += 32) {
            const bool in = sub + lane < gt;
            uint4 gq = make_uint4(0u, 0u, 0u, 0u);
            if (in) gq = sg[sub + lane];
            const uint32_t start = gq.y, C = gq.w;
            const uint32_t T = BOUNDED ? min(gq.z, jv.tau_max) : gq.z;
            uint64_t bk = 0;                 // this gap's best candidate of the warp
            uint32_t bj = 0xFFFFFFFFu, bc = 0;
            uint32_t todo = __ballot_sync(0xFFFFFFFFu, in);
            while (todo) {
                // the next run of gaps of one capacity (the list is ordered by capacity, then T)
                const uint32_t first = (uint32_t)__ffs((int)todo) - 1u;
                const uint32_t Cc = __shfl_sync(0xFFFFFFFFu, C, first);
                const uint32_t run = __ballot_sync(0xFFFFFFFFu, in && C == Cc) & todo;
                todo &= ~run;
                const uint32_t last = 31u - (uint32_t)__clz((int)run);
                const uint32_t T_lo = __shfl_sync(0xFFFFFFFFu, T, first);
                const uint32_t T_hi = __shfl_sync(0xFFFFFFFFu, T, last);
                const bool mine = (run >> lane) & 1u;

                if (!have_class || Cc != curC) {
                    // new capacity class: T restarts from its smallest value, so do the cursors
                    have_class = true;
                    curC = Cc;
                    mg_wait<0>();
#pragma unroll
                    for (int i = 0; i < TILE_RING; ++i) {
                        if ((uint32_t)i < n) mg_cp_async16(ring_s + i * 512, row0 + i);
                        mg_commit();
                    }
                    next_row = row0 + TILE_RING;
                    mg_wait<0>();
                    w = 0; curKey = 0; open = false; thr = 0xFFFFFFFFu;
                    if (n) {
                        const uint4 row = mg_lds128(ring_s);
                        nextW = pack64(row.z, row.w);
                        if (row.y <= Cc) { open = true; thr = row.x - Dp; }
                    }
                    dirty = true;
                }
                // catch up: rows no longer than T_lo qualify for every gap of the run
                while (__any_sync(0xFFFFFFFFu, open && thr <= T_lo)) {
                    if (open && thr <= T_lo) step_cursor(Cc);
                    dirty = true;
                }
                if (dirty) {
                    // PM: candidates in ready order, inclusive prefix maximum
                    __syncwarp();
                    pm_s[rank] = make_uint4((uint32_t)curKey, (uint32_t)(curKey >> 32), w, 0u);
                    __syncwarp();
                    const uint4 v = pm_s[lane];
                    pk = pack64(v.x, v.y); pc = v.z; pj = sjob;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint64_t k2 = __shfl_up_sync(0xFFFFFFFFu, pk, o);
                        const uint32_t j2 = __shfl_up_sync(0xFFFFFFFFu, pj, o);
                        const uint32_t c2 = __shfl_up_sync(0xFFFFFFFFu, pc, o);
                        if (lane >= (uint32_t)o && cand_better(k2, j2, pk, pj)) { pk = k2; pj = j2; pc = c2; }
                    }
                    dirty = false;
                }
                // base answer: number of jobs of the warp that are ready by this gap's start
                uint32_t e = 0;
#pragma unroll
                for (uint32_t s = 16; s >= 1; s >>= 1) {
                    const uint32_t v = __shfl_sync(0xFFFFFFFFu, sready, (e + s - 1u) & 31u);
                    if (v <= start) e += s;
                }
                if (e == 31u && sready_last <= start) e = 32u;
                {
                    const uint32_t src = (e ? e - 1u : 0u) & 31u;
                    const uint64_t k0 = __shfl_sync(0xFFFFFFFFu, pk, src);
                    const uint32_t j0 = __shfl_sync(0xFFFFFFFFu, pj, src);
                    const uint32_t c0 = __shfl_sync(0xFFFFFFFFu, pc, src);
                    if (mine && e) { bk = k0; bj = j0; bc = c0; }
                }
                // events: rows with a duration in (T_lo, T_hi]
                uint32_t pending;
                while ((pending = __ballot_sync(0xFFFFFFFFu, open && thr <= T_hi)) != 0u) {
                    if (open && thr <= T_hi) {
                        const uint32_t thr_e = thr;
                        step_cursor(Cc);
                        ev[lane] = make_uint4(thr_e, ready, (uint32_t)curKey, (uint32_t)(curKey >> 32));
                        evc[lane] = w;
                    }
                    dirty = true;
                    __syncwarp();
                    uint32_t m = pending;
                    while (m) {
                        const uint32_t b = (uint32_t)__ffs((int)m) - 1u;
                        m &= m - 1u;
                        const uint4 q = ev[b];
                        const uint32_t c = evc[b];
                        const uint64_t k = pack64(q.z, q.w);
                        const uint32_t jb = job0 + b;
                        // a later row of the job that already leads replaces it (jb == bj): the longest subjob
                        const bool take = mine && T >= q.x && start >= q.y && (k > bk || (k == bk && jb <= bj));
                        if (take) { bk = k; bj = jb; bc = c; }
                    }
                    __syncwarp();
                }
            }
            if (in) {
                Partial pr;
                pr.key = bk; pr.job = bk ? bj : 0xFFFFFFFFu; pr.cnt = bk ? bc : 0u;
                stage[wid * TILE_GT + sub + lane] = pr;
            }
        }
        __syncthreads();
        if (threadIdx.x < gt) {
            Partial bestp = stage[threadIdx.x];
#pragma unroll
            for (int ww = 1; ww < TILE_WARPS; ++ww) {
                const Partial c = stage[ww * TILE_GT + threadIdx.x];
                if (cand_better(c.key, c.job, bestp.key, bestp.job)) bestp = c;
            }
            partial_out[(size_t)blockIdx.x * G + g0 + threadIdx.x] = bestp;
        }
        __syncthreads();
    }
    mg_wait<0>();
}

}  // namespace sja
