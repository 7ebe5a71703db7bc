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
//    cursors, all lanes that have steps to do at once.  A step can only matter if its key
//    beats the PM entry at the job's own rank as it stood at the start of the run: every gap
//    that may take the job (rank < #eligible) already holds at least that entry.  Such steps
//    (few: the prefix maxima of a random order of 32 are about 4 jobs) are posted to shared
//    memory as (duration, rank, key); the others are silent.  Every lane then looks at each
//    posted event twice over: as a gap (is the row within my window, is the job among my
//    eligible ones, does it beat my best) and as PM entry (does it raise the prefix maximum
//    at my rank), which leaves the PM ready for the next 32 gaps.
//
// Where the next 64 gaps all belong to the class the cursors are in, a lane takes two of them
// at once (SJA_TILE_MULTI): one set of cursor steps and one pass over the posted events serve
// both, and the bookkeeping of a step is paid once.
//
// The cost is therefore per (warp, 32 gaps) a small fixed part (the lookup) plus the cursor
// steps, not the number of pairs.  The PM is rebuilt by a warp scan only after a restart of
// the cursors (a new capacity class, or the start of a CTA's gap range).
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
#define SJA_TILE_GT 256
#endif
#ifndef SJA_TILE_MULTI
#define SJA_TILE_MULTI 2
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
constexpr int TILE_SMEM_BYTES = TILE_RING_BYTES + TILE_STAGE_BYTES + TILE_GAP_BYTES + TILE_EVENT_BYTES + TILE_ECNT_BYTES;
static_assert((TILE_RING & (TILE_RING - 1)) == 0, "ring size must be a power of two");
static_assert(TILE_GT % 32 == 0 && TILE_GT <= TILE_JOBS, "one thread per gap of a staging tile");

// Candidate order: larger key first, then the lower job id.
__device__ __forceinline__ bool cand_better(uint64_t ka, uint32_t ja, uint64_t kb, uint32_t jb) {
    return ka > kb || (ka == kb && ja < jb);
}

// Inside a warp a candidate is (key, inv) with inv = 31 - owning lane: the larger pair wins
// (larger key, then the lower lane = lower job id).  An equal pair is a later row of the job
// that already leads: it wins too (same score, longer subjob).
__device__ __forceinline__ bool pair_ge(uint64_t ka, uint32_t ia, uint64_t kb, uint32_t ib) {
    return ka > kb || (ka == kb && ia >= ib);
}

template <uint32_t KIND, bool BOUNDED>
__global__ void __launch_bounds__(TILE_WARPS * 32, TILE_CTAS_PER_SM) select_tile_kernel(
    JobView jv, const Gap* __restrict__ sgaps, uint32_t G, uint32_t gaps_per_split, Partial* __restrict__ partial_out,
    LaunchGate gate) {
    dep_wait();
    dep_launch();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // G is the gap count the launch was sized for (and the row length of partial_out); a re-auction hands
    // the count actually left in device memory, so that several passes can be queued without a host wait
    const uint32_t G_now = gate_gaps(gate, G);
    if (blockIdx.y * gaps_per_split >= G_now) return;
    if (!chunk_dirty(gate, blockIdx.x * TILE_JOBS, TILE_JOBS)) return;   // re-auction: its candidate row still stands
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(smem_raw);
    Partial* stage = reinterpret_cast<Partial*>(smem_raw + TILE_RING_BYTES);                       // [WARPS][GT]
    const uint4* sg = reinterpret_cast<const uint4*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES);
    uint4* sg_w = reinterpret_cast<uint4*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES);
    uint4* ev = reinterpret_cast<uint4*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES + TILE_GAP_BYTES) + wid * 32;
    uint32_t* evc = reinterpret_cast<uint32_t*>(smem_raw + TILE_RING_BYTES + TILE_STAGE_BYTES + TILE_GAP_BYTES +
                                                TILE_EVENT_BYTES) + wid * 32;
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
    evc[rank] = lane;
    ev[rank].x = ready;
    __syncwarp();
    const uint32_t sready = ev[lane].x;     // ready time of the job of rank `lane`
    const uint32_t slane = evc[lane];       // and the lane that owns it
    __syncwarp();
    const uint32_t sready_last = __shfl_sync(0xFFFFFFFFu, sready, 31);
    uint64_t pk = 0;                 // PM entry of rank `lane`: key and 31 - owning lane
    uint32_t pi = 0;

    const uint32_t g_begin = blockIdx.y * gaps_per_split;
    const uint32_t g_end = min(G_now, g_begin + gaps_per_split);
    bool have_class = false, dirty = true;
    uint32_t curC = 0;

    // One cursor step of this lane: row w becomes the job's candidate, row w + 1 is fetched.
    auto step_cursor = [&](uint32_t C) {
        curKey = (!BOUNDED || thr >= jv.tau_min) ? policy_key(KIND, nextW, factor) : 0ull;
        if (w + TILE_RING < n) mg_cp_async16(ring_s + (w & (TILE_RING - 1)) * 512, next_row);
        mg_commit();
        ++next_row;
        ++w;
        open = false;
        thr = 0xFFFFFFFFu;
        if (w < n) {
            mg_wait<TILE_RING - 1>();
            const uint4 row = mg_lds128(ring_s + (w & (TILE_RING - 1)) * 512);
            nextW = policy_payload(KIND, row, Wp);
            if (row.y <= C) { open = true; thr = row.x - Dp; }
        }
    };

    for (uint32_t g0 = g_begin; g0 < g_end; g0 += TILE_GT) {
        const uint32_t gt = min((uint32_t)TILE_GT, g_end - g0);
        if (threadIdx.x < gt) sg_w[threadIdx.x] = __ldg(reinterpret_cast<const uint4*>(sgaps) + g0 + threadIdx.x);
        __syncthreads();
        for (uint32_t sub = 0; sub < gt; sub += 32) {
#if SJA_TILE_MULTI > 1
            // Fast path: MULTI x 32 gaps of the class the cursors are in, MULTI per lane.  One set of cursor
            // steps and one pass over the posted events serve all gaps of a lane; the PM is up to date (nothing
            // was restarted), so no run detection, no catch-up and no rebuild are needed.
            bool multi = !dirty && have_class && sub + 32u * SJA_TILE_MULTI <= gt;
            if (multi) {
                bool same = true;
#pragma unroll
                for (int q = 0; q < SJA_TILE_MULTI; ++q) same = same && sg[sub + 32 * q + lane].w == curC;
                multi = __all_sync(0xFFFFFFFFu, same);
            }
            if (multi) {
                uint32_t Tq[SJA_TILE_MULTI], eq[SJA_TILE_MULTI], iq[SJA_TILE_MULTI], cq[SJA_TILE_MULTI];
                uint64_t kq[SJA_TILE_MULTI];
#pragma unroll
                for (int q = 0; q < SJA_TILE_MULTI; ++q) {
                    const uint4 gq = sg[sub + 32 * q + lane];
                    Tq[q] = BOUNDED ? min(gq.z, jv.tau_max) : gq.z;
                    uint32_t e = 0;
#pragma unroll
                    for (uint32_t s = 16; s >= 1; s >>= 1) {
                        const uint32_t v = __shfl_sync(0xFFFFFFFFu, sready, (e + s - 1u) & 31u);
                        if (v <= gq.y) e += s;
                    }
                    if (e == 31u && sready_last <= gq.y) e = 32u;
                    eq[q] = e;
                    // base answer: PM[e - 1]; its row count is the owner's current cursor
                    const uint32_t src = (e ? e - 1u : 0u) & 31u;
                    const uint64_t k0 = __shfl_sync(0xFFFFFFFFu, pk, src);
                    const uint32_t i0 = __shfl_sync(0xFFFFFFFFu, pi, src);
                    const uint32_t c0 = __shfl_sync(0xFFFFFFFFu, w, 31u - i0);
                    kq[q] = e ? k0 : 0ull; iq[q] = e ? i0 : 0u; cq[q] = e ? c0 : 0u;
                }
                const uint64_t pmr_k = __shfl_sync(0xFFFFFFFFu, pk, rank);
                const uint32_t pmr_i = __shfl_sync(0xFFFFFFFFu, pi, rank);
                const uint32_t T_hi = __shfl_sync(0xFFFFFFFFu, Tq[SJA_TILE_MULTI - 1], 31);
                while (__any_sync(0xFFFFFFFFu, open && thr <= T_hi)) {
                    bool post = false;
                    if (open && thr <= T_hi) {
                        uint32_t thr_e;
                        do {
                            thr_e = thr;
                            step_cursor(curC);
                            post = pair_ge(curKey, 31u - lane, pmr_k, pmr_i);
                        } while (!post && open && thr <= T_hi);
                        if (post) {
                            ev[lane] = make_uint4(thr_e, rank, (uint32_t)curKey, (uint32_t)(curKey >> 32));
                            evc[lane] = w;
                        }
                    }
                    uint32_t m = __ballot_sync(0xFFFFFFFFu, post);
                    if (m == 0u) continue;
                    __syncwarp();
                    while (m) {
                        const uint32_t b = (uint32_t)__ffs((int)m) - 1u;
                        m &= m - 1u;
                        const uint4 q4 = ev[b];           // duration, rank of the job, key
                        const uint32_t c = evc[b];
                        const uint64_t k = pack64(q4.z, q4.w);
                        const uint32_t ib = 31u - b;
#pragma unroll
                        for (int q = 0; q < SJA_TILE_MULTI; ++q)
                            if (Tq[q] >= q4.x && q4.y < eq[q] && pair_ge(k, ib, kq[q], iq[q])) { kq[q] = k; iq[q] = ib; cq[q] = c; }
                        if (lane >= q4.y && pair_ge(k, ib, pk, pi)) { pk = k; pi = ib; }
                    }
                    __syncwarp();
                }
#pragma unroll
                for (int q = 0; q < SJA_TILE_MULTI; ++q) {
                    Partial pr;
                    pr.key = kq[q]; pr.job = kq[q] ? job0 + 31u - iq[q] : 0xFFFFFFFFu; pr.cnt = kq[q] ? cq[q] : 0u;
                    stage[wid * TILE_GT + sub + 32 * q + lane] = pr;
                }
                sub += 32u * (SJA_TILE_MULTI - 1);
                continue;
            }
#endif
            const bool in = sub + lane < gt;
            uint4 gq = make_uint4(0u, 0u, 0u, 0u);
            if (in) gq = sg[sub + lane];
            const uint32_t start = gq.y, C = gq.w;
            const uint32_t T = BOUNDED ? min(gq.z, jv.tau_max) : gq.z;
            // number of jobs of the warp that are ready by this gap's start (they are ranks 0 .. e-1)
            uint32_t e = 0;
#pragma unroll
            for (uint32_t s = 16; s >= 1; s >>= 1) {
                const uint32_t v = __shfl_sync(0xFFFFFFFFu, sready, (e + s - 1u) & 31u);
                if (v <= start) e += s;
            }
            if (e == 31u && sready_last <= start) e = 32u;
            uint64_t bk = 0;                 // this gap's best candidate of the warp: key, 31 - lane, rows
            uint32_t bi = 0, bc = 0;
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
                        nextW = policy_payload(KIND, row, Wp);
                        if (row.y <= Cc) { open = true; thr = row.x - Dp; }
                    }
                    dirty = true;
                }
                if (dirty) {
                    // after a restart: catch up without posting (rows no longer than T_lo qualify for
                    // every gap of the run), then PM by a warp scan over the candidates in ready order
                    while (__any_sync(0xFFFFFFFFu, open && thr <= T_lo)) {
                        if (open && thr <= T_lo) step_cursor(Cc);
                    }
                    pk = __shfl_sync(0xFFFFFFFFu, curKey, slane);
                    pi = 31u - slane;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint64_t k2 = __shfl_up_sync(0xFFFFFFFFu, pk, o);
                        const uint32_t i2 = __shfl_up_sync(0xFFFFFFFFu, pi, o);
                        if (lane >= (uint32_t)o && pair_ge(k2, i2, pk, pi)) { pk = k2; pi = i2; }
                    }
                    dirty = false;
                }
                // PM entry at my job's rank as the run starts: what a step of my job has to beat
                const uint64_t pmr_k = __shfl_sync(0xFFFFFFFFu, pk, rank);
                const uint32_t pmr_i = __shfl_sync(0xFFFFFFFFu, pi, rank);
                // base answer: PM[e - 1]; its row count is the owner's current cursor
                {
                    const uint32_t src = (e ? e - 1u : 0u) & 31u;
                    const uint64_t k0 = __shfl_sync(0xFFFFFFFFu, pk, src);
                    const uint32_t i0 = __shfl_sync(0xFFFFFFFFu, pi, src);
                    const uint32_t c0 = __shfl_sync(0xFFFFFFFFu, w, 31u - i0);
                    if (mine && e) { bk = k0; bi = i0; bc = c0; }
                }
                // events: rows with a duration up to T_hi
                while (__any_sync(0xFFFFFFFFu, open && thr <= T_hi)) {
                    bool post = false;
                    if (open && thr <= T_hi) {
                        uint32_t thr_e;
                        do {
                            thr_e = thr;
                            step_cursor(Cc);
                            post = pair_ge(curKey, 31u - lane, pmr_k, pmr_i);
                        } while (!post && open && thr <= T_hi);
                        if (post) {
                            ev[lane] = make_uint4(thr_e, rank, (uint32_t)curKey, (uint32_t)(curKey >> 32));
                            evc[lane] = w;
                        }
                    }
                    uint32_t m = __ballot_sync(0xFFFFFFFFu, post);
                    if (m == 0u) continue;
                    __syncwarp();
                    while (m) {
                        const uint32_t b = (uint32_t)__ffs((int)m) - 1u;
                        m &= m - 1u;
                        const uint4 q = ev[b];           // duration, rank of the job, key
                        const uint32_t c = evc[b];
                        const uint64_t k = pack64(q.z, q.w);
                        const uint32_t ib = 31u - b;
                        // as a gap: row within my window, job among my eligible ones, beats my best
                        if (mine && T >= q.x && q.y < e && pair_ge(k, ib, bk, bi)) { bk = k; bi = ib; bc = c; }
                        // as PM entry `lane`: the job is among the first lane + 1 by ready time
                        if (lane >= q.y && pair_ge(k, ib, pk, pi)) { pk = k; pi = ib; }
                    }
                    __syncwarp();
                }
            }
            if (in) {
                Partial pr;
                pr.key = bk; pr.job = bk ? job0 + 31u - bi : 0xFFFFFFFFu; pr.cnt = bk ? bc : 0u;
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
            partial_out[row_slot(gate, G, blockIdx.x, g0 + threadIdx.x, sg[threadIdx.x].x)] = bestp;
        }
        __syncthreads();
    }
    mg_wait<0>();
}

}  // namespace sja
