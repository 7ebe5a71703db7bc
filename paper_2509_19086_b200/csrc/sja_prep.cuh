// Load preparation kernels: CSR validation and boundary-row counting, row offsets, per-job
// state initialisation.  They run before scan_profiles_kernel (sja_scan.cuh) in sja_load_profiles.
#pragma once
#include "sja_common.cuh"

namespace sja {

// ---------------------------------------------------------------------------------------
// Pass 0: validate the CSR and count the boundary rows of every job (popcount of its safe
// bits above the progress point; the end of a job always counts).  The kernel is bound by
// memory latency, so it wants many warps with several loads in flight each: a CTA of 8
// warps owns 64 consecutive jobs, a warp counts 8 of them, four at a time with eight lanes
// per job (lanes stride over the job's safe words, four independent loads per lane); jobs of
// more than 256 safe words are left to a second phase in which the whole CTA counts them one
// after the other (on a heavy-tailed mix they hold most of the bits, and a warp that met
// several of them would keep the other seven waiting).  The CTA scans its 64 counts and
// writes each job's offset relative to the CTA plus the CTA total.  Two tiny kernels then
// turn CTA totals into global offsets.
constexpr int COUNT_JOBS_PER_CTA = 64;
constexpr int COUNT_JOBS_PER_WARP = 8;
#ifndef SJA_COUNT_COOP_WORDS
#define SJA_COUNT_COOP_WORDS 256
#endif
constexpr uint32_t COUNT_COOP_WORDS = SJA_COUNT_COOP_WORDS;   // jobs of this many safe words or more: whole-CTA pass (swept 16 .. 1024)
constexpr uint32_t COUNT_LONG = 0x80000000u;   // marker: job left to the whole-CTA pass

__global__ void __launch_bounds__(256, 8) count_boundaries_kernel(
    const uint64_t* __restrict__ off, const uint32_t* __restrict__ sbits,
    const uint32_t* __restrict__ p0 /* may be nullptr: all 0 */, uint32_t J, uint64_t* __restrict__ local_off,
    uint64_t* __restrict__ cta_total, uint32_t* __restrict__ flags, uint32_t* __restrict__ long_list) {
    dep_launch();   // the one-CTA offsets kernel may be brought in meanwhile
    __shared__ uint32_t cnts[COUNT_JOBS_PER_CTA];
    __shared__ uint32_t is_long[COUNT_JOBS_PER_CTA];
    __shared__ uint32_t long_cnt[COUNT_JOBS_PER_CTA];   // boundary rows of the jobs the whole CTA counts
    __shared__ uint4 ldesc[COUNT_JOBS_PER_CTA];         // those jobs: {first word lo, hi, last word - first word, first bit | last bit << 8 | slot << 16}
    __shared__ uint32_t n_long_cta;
    __shared__ uint64_t warp_sums[COUNT_JOBS_PER_CTA / 32];
    if (threadIdx.x < COUNT_JOBS_PER_CTA) long_cnt[threadIdx.x] = 0u;
    if (threadIdx.x == 0) n_long_cta = 0u;
    __syncthreads();
    const uint64_t N = __ldg(off + J);   // total step count
    const uint64_t long_thresh = long_job_threshold(N, J);
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    const uint32_t slot0 = wid * COUNT_JOBS_PER_WARP;              // first job slot of this warp in the CTA
    const uint32_t jbase = blockIdx.x * COUNT_JOBS_PER_CTA + slot0;
    const uint32_t grp = lane >> 3, sub = lane & 7u;
#pragma unroll
    for (uint32_t it = 0; it < COUNT_JOBS_PER_WARP / 4; ++it) {
        const uint32_t i = it * 4u + grp;
        const uint32_t j = jbase + i;
        uint32_t cnt = 0;
        bool bad = false, lng = false;
        if (j < J) {
            const uint64_t js = __ldg(off + j), je = __ldg(off + j + 1);
            const uint32_t p = p0 ? __ldg(p0 + j) : 0u;
            bad = (je < js) || (je > N) || (je - js > 0xFFFFFFFFull) || ((uint64_t)p > je - js);
            if (j == 0 && js != 0) bad = true;
            if (!bad) {
                const uint64_t s = js + p, e = je;
                lng = e - s > long_thresh;   // goes on the list the scan works off first
                if (s < e && ((e - 1) >> 5) - (s >> 5) >= COUNT_COOP_WORDS) {
                    cnt = COUNT_LONG;   // long job: counted by the whole CTA below
                    if (sub == 0) {
                        const uint64_t w0 = s >> 5;
                        ldesc[atomicAdd(&n_long_cta, 1u)] =
                            make_uint4((uint32_t)w0, (uint32_t)(w0 >> 32), (uint32_t)(((e - 1) >> 5) - w0),
                                       (uint32_t)(s & 31) | ((uint32_t)((e - 1) & 31) << 8) | ((slot0 + i) << 16));
                    }
                } else if (s < e) {
                    const uint64_t w0 = s >> 5, w1 = (e - 1) >> 5;
                    const uint32_t m0 = 0xFFFFFFFFu << (uint32_t)(s & 31);
                    const uint32_t m1 = 0xFFFFFFFFu >> (31u - (uint32_t)((e - 1) & 31));
                    uint64_t w = w0 + sub;
                    // four independent loads in flight per lane
                    for (; w + 24 <= w1; w += 32) {
                        uint32_t x0 = __ldg(sbits + w), x1 = __ldg(sbits + w + 8);
                        uint32_t x2 = __ldg(sbits + w + 16), x3 = __ldg(sbits + w + 24);
                        if (w == w0) x0 &= m0;
                        if (w + 24 == w1) x3 &= m1;
                        cnt += __popc(x0) + __popc(x1) + __popc(x2) + __popc(x3);
                    }
                    for (; w <= w1; w += 8) {
                        uint32_t x = __ldg(sbits + w);
                        if (w == w0) x &= m0;
                        if (w == w1) x &= m1;
                        cnt += __popc(x);
                    }
                    if (sub == 0) cnt += 1u - ((__ldg(sbits + w1) >> (uint32_t)((e - 1) & 31)) & 1u);
                }
            }
        }
        if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(flags, FLAG_BAD_PROFILE);
        if (cnt != COUNT_LONG) {   // (uniform within the eight lanes of a job)
            cnt += __shfl_xor_sync(0xFFu << (lane & 24u), cnt, 1);
            cnt += __shfl_xor_sync(0xFFu << (lane & 24u), cnt, 2);
            cnt += __shfl_xor_sync(0xFFu << (lane & 24u), cnt, 4);
        }
        if (sub == 0) { cnts[slot0 + i] = cnt; is_long[slot0 + i] = lng ? 1u : 0u; }
    }
    __syncthreads();
    // long jobs (more than 256 safe words), by the whole CTA: every thread takes up to eight words of a job, 256
    // apart, and two jobs are under way at a time (sixteen independent loads in flight per thread), so that all
    // warps of the CTA carry the long jobs of any one of them and a job costs about half a memory round trip.
    // A warp adds its part to the job's counter in shared memory.  The thread that holds a job's last word also
    // counts the end of the job where its bit is not set.
    {
        const uint32_t n_long = n_long_cta;
        // words [base, base + 8 * 256) of the job, relative to its first word
        auto load8 = [&](const uint4& dsc, uint32_t base, uint32_t (&x)[8]) {
            const uint64_t w0 = pack64(dsc.x, dsc.y);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t r = base + threadIdx.x + 256u * u;
                x[u] = r <= dsc.z ? __ldg(sbits + w0 + r) : 0u;
            }
        };
        auto tally8 = [&](const uint4& dsc, uint32_t base, uint32_t (&x)[8]) -> uint32_t {
            const uint32_t first_bit = dsc.w & 31u, last_bit = (dsc.w >> 8) & 31u;
            uint32_t cnt = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t r = base + threadIdx.x + 256u * u;
                if (r == 0u) x[u] &= 0xFFFFFFFFu << first_bit;
                if (r == dsc.z) {
                    cnt += 1u - ((x[u] >> last_bit) & 1u);
                    x[u] &= 0xFFFFFFFFu >> (31u - last_bit);
                }
                cnt += __popc(x[u]);
            }
            return cnt;
        };
        auto add = [&](const uint4& dsc, uint32_t cnt) {
            cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
            if (lane == 0 && cnt) atomicAdd(&long_cnt[dsc.w >> 16], cnt);
        };
        for (uint32_t q = 0; q < n_long; q += 2) {
            const bool two = q + 1 < n_long;
            const uint4 da = ldesc[q];
            const uint4 db = two ? ldesc[q + 1] : make_uint4(0u, 0u, 0u, 0u);
            uint32_t xa[8], xb[8];
            load8(da, 0u, xa);
            if (two) load8(db, 0u, xb);
            uint32_t ca = tally8(da, 0u, xa);
            uint32_t cb = two ? tally8(db, 0u, xb) : 0u;
            // jobs of more than 2048 words: the rest, one job at a time
            for (uint32_t base = 8u * 256u; base <= da.z; base += 8u * 256u) {
                load8(da, base, xa);
                ca += tally8(da, base, xa);
            }
            if (two)
                for (uint32_t base = 8u * 256u; base <= db.z; base += 8u * 256u) {
                    load8(db, base, xb);
                    cb += tally8(db, base, xb);
                }
            add(da, ca);
            if (two) add(db, cb);
        }
    }
    __syncthreads();
    // exclusive scan of the CTA's counts by its first warps, one job per thread
    uint32_t mine = 0;
    uint64_t inc = 0;
    if (threadIdx.x < COUNT_JOBS_PER_CTA) {
        // the list of long jobs (flags[1] counts them): one atomic per warp of 32 jobs, not one per job --
        // on a heavy-tailed mix every eighth job is long, and that many atomics on one word take longer than the count
        const bool lng = is_long[threadIdx.x] != 0u;
        const uint32_t lb = __ballot_sync(0xFFFFFFFFu, lng);
        if (lb) {
            uint32_t base = 0;
            if (lane == 0) base = atomicAdd(flags + 1, (uint32_t)__popc(lb));
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            if (lng) long_list[base + __popc(lb & ((1u << lane) - 1u))] = blockIdx.x * COUNT_JOBS_PER_CTA + threadIdx.x;
        }
        mine = cnts[threadIdx.x];
        if (mine == COUNT_LONG) mine = long_cnt[threadIdx.x];
        inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= (uint32_t)o) inc += y;
        }
        if (lane == 31) warp_sums[wid] = inc;
    }
    __syncthreads();
    if (threadIdx.x < COUNT_JOBS_PER_CTA) {
        uint64_t before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < COUNT_JOBS_PER_CTA / 32; ++w) {
            const uint64_t v = warp_sums[w];
            if ((uint32_t)w < wid) before += v;
            total += v;
        }
        const uint32_t j = blockIdx.x * COUNT_JOBS_PER_CTA + threadIdx.x;
        if (j < J) local_off[j] = before + inc - mine;
        if (threadIdx.x == 0) cta_total[blockIdx.x] = total;
    }
}

// Exclusive prefix sum of the per-CTA totals -> base[P+1].  One CTA of 1024 threads walks the
// array in tiles of 8192 with a running carry.
__global__ void __launch_bounds__(1024) cta_offsets_kernel(const uint64_t* __restrict__ totals, uint32_t P,
                                                           uint64_t* __restrict__ base_out) {
    dep_wait();
    dep_launch();
    __shared__ uint64_t warp_sums[32];
    __shared__ uint64_t warp_excl[32];
    __shared__ uint64_t tile_total;
    const uint32_t t = threadIdx.x, lane = t & 31u, wid = t >> 5;
    uint64_t carry = 0;  // same value in every thread
    for (uint64_t base = 0; base < P; base += 8192) {
        uint64_t v[8];
        uint64_t local = 0;
        const uint64_t i0 = base + (uint64_t)t * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            v[i] = (i0 + i < P) ? totals[i0 + i] : 0ull;
            local += v[i];
        }
        uint64_t inc = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= (uint32_t)o) inc += y;
        }
        if (lane == 31) warp_sums[wid] = inc;
        __syncthreads();
        if (wid == 0) {
            const uint64_t ws = warp_sums[lane];
            uint64_t wi = ws;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, wi, o);
                if (lane >= (uint32_t)o) wi += y;
            }
            warp_excl[lane] = wi - ws;
            if (lane == 31) tile_total = wi;
        }
        __syncthreads();
        uint64_t run = carry + warp_excl[wid] + (inc - local);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (i0 + i < P) base_out[i0 + i] = run;
            run += v[i];
        }
        carry += tile_total;
        __syncthreads();  // warp_sums / tile_total are rewritten by the next tile
    }
    if (t == 0) base_out[P] = carry;
}

// Last preparation step of a load, one thread per job:
//  * boff[j] = base of the job's counting CTA + offset inside it; boff[J] = total row count.  A total above
//    `cap_rows` (what the table buffers handed to the scan can hold) raises FLAG_NEED_ROWS.
//  * If the load stands (CSR valid, table fits): per-job state of a fresh load -- progress and attributes
//    copied, cursors and commit votes cleared, the scan's job counter reset.  Otherwise nothing of the
//    previously loaded state is touched.
// Source pointers may be nullptr (attribute not given; progress = 0).
__global__ void __launch_bounds__(256) finish_load_kernel(
    uint32_t J, uint32_t P, const uint64_t* __restrict__ local_off, const uint64_t* __restrict__ cta_base,
    uint64_t* __restrict__ boff, uint64_t cap_rows, const uint32_t* __restrict__ p_src,
    const uint32_t* __restrict__ ready_src, const uint32_t* __restrict__ wait_src,
    const uint8_t* __restrict__ prio_src, uint32_t* __restrict__ p, uint32_t* __restrict__ ready,
    uint32_t* __restrict__ wait, uint8_t* __restrict__ prio, uint32_t* __restrict__ pb, uint32_t* __restrict__ Dp,
    uint64_t* __restrict__ Wp, unsigned long long* __restrict__ jobwin, uint32_t* __restrict__ counter,
    uint32_t* __restrict__ flags) {
    dep_wait();
    dep_launch();
    const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t total = cta_base[P];
    if (j < J) boff[j] = cta_base[j / COUNT_JOBS_PER_CTA] + local_off[j];
    if (j == 0) {
        boff[J] = total;
        if (total > cap_rows) atomicOr(flags, FLAG_NEED_ROWS);
    }
    if ((*flags & FLAG_BAD_PROFILE) || total > cap_rows) return;     // same verdict in every thread
    if (j == 0) *counter = 0;
    if (j >= J) return;
    p[j] = p_src ? p_src[j] : 0u;
    if (ready_src) ready[j] = ready_src[j];
    if (wait_src) wait[j] = wait_src[j];
    if (prio_src) prio[j] = prio_src[j];
    pb[j] = 0;
    Dp[j] = 0;
    Wp[j] = 0;
    jobwin[j] = 0ull;
}

}  // namespace sja
