// Segmented prefix scan: raw per-step profiles -> per-job boundary table.
//
// The window-max admissibility test (Sections 3.8 / 3.9) and the window-length bound
// (Section 3.1) only ever need to be evaluated at safe boundaries (Section 3.7), because a
// subjob may end nowhere else.  The scan therefore streams every step once (8 B + 1 bit)
// and writes one 24-byte row per safe boundary.
//
// Work split: one warp streams one job (jobs are handed out by an atomic counter, so no
// warp ever waits on another).  A warp moves 512 steps per iteration: coalesced 16-byte
// cp.async copies into a per-warp shared-memory ring (XOR-swizzled at 16-byte granularity),
// then each lane reads its 16 CONSECUTIVE steps back with conflict-free 128-bit shared
// loads, reduces them locally, the warp combines the 32 lane aggregates with shuffles, and
// each lane re-walks its 16 steps to emit rows at its safe bits.
#pragma once
#include "sja_common.cuh"

namespace sja {

#ifndef SJA_SCAN_STAGES
#define SJA_SCAN_STAGES 2
#endif
#ifndef SJA_SCAN_WARPS
#define SJA_SCAN_WARPS 10
#endif
#ifndef SJA_SCAN_CTAS_PER_SM
#define SJA_SCAN_CTAS_PER_SM 2
#endif
constexpr int SCAN_BLK = 512;                       // steps per warp iteration (16 per lane)
constexpr int SCAN_STAGES = SJA_SCAN_STAGES;        // cp.async ring depth per warp
constexpr int SCAN_WARPS = SJA_SCAN_WARPS;          // warps per CTA
constexpr int SCAN_CTAS_PER_SM = SJA_SCAN_CTAS_PER_SM;
constexpr int SCAN_STAGE_BYTES = 2048 + 2048 + 64;  // d, m, 16 safe words
// Per warp, between its two ring slots: 3 KB that belong to the row buffer only.  A consumed slot alone holds the
// rows of a block with boundaries up to one in three steps; with the region next to it (behind slot 0, before
// slot 1: contiguous with either) up to 301 rows, i.e. boundaries denser than one in two, leave through the buffer
// with coalesced stores.  2 CTAs x 10 warps x 11 392 B = 222.5 KB of the SM's 227 KB.
#ifndef SJA_SCAN_EXTRA_BYTES
#define SJA_SCAN_EXTRA_BYTES 3072
#endif
constexpr int SCAN_EXTRA_BYTES = SJA_SCAN_EXTRA_BYTES;
constexpr int SCAN_WARP_BYTES = SCAN_STAGES * SCAN_STAGE_BYTES + SCAN_EXTRA_BYTES;
constexpr int SCAN_SMEM_BYTES = SCAN_WARPS * SCAN_WARP_BYTES;

struct ScanArgs {
    const uint64_t* off;     // [J+1]
    const uint32_t* d;       // [N]
    const uint32_t* m;       // [N]
    const uint32_t* sbits;   // [ceil(N/32)]
    const uint32_t* p0;      // [J] progress at load, or nullptr (all 0)
    const uint32_t* wait;    // [J] or nullptr
    const uint8_t* prio;     // [J] or nullptr
    const uint64_t* boff;    // [J+1] row offsets
    uint4* A;                // rows {D, M, W_lo, W_hi}
    uint2* B;                // rows {k, S}
    uint32_t J;              // N = off[J] is read by the kernel
    uint32_t* counter;       // job hand-out counter (zeroed before launch)
    uint32_t* flags;         // flags[0] status bits, flags[1] number of listed long jobs
    const uint32_t* long_list;   // jobs to scan first (see long_job_threshold)
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// 16-byte chunk c of a 2 KB stage array lives at chunk slot swz(c): lane L reading chunks
// 4L..4L+3 and lane L writing chunks 32r+L both hit 8 distinct bank groups per quarter-warp.
__device__ __forceinline__ uint32_t swz(uint32_t c) { return c ^ ((c >> 3) & 3u); }

// ---------------------------------------------------------------------------------------
// The scan proper.
//
// Per 512-step block a warp knows, after one popcount scan, how many rows the block emits.
// Usual case (at most SCAN_STAGE_ROWS rows): each lane walks its 16 steps ONCE, keeping
// lane-local sums, and drops a lane-relative row into shared memory at every safe bit (the
// just-consumed input slot of the ring, lengthened by the region next to it, is the row buffer).  The warp then scans the
// 32 lane totals and a second, row-indexed phase (32 rows per iteration, i.e. about a tenth of
// the steps) adds each row's lane offset, derives the running maximum as a prefix maximum over
// the rows' segment maxima, and writes the finished rows with fully coalesced 512-byte and
// 256-byte stores.  Blocks with more rows (boundaries denser than about three in five steps)
// take the two-pass route: lane totals first, then a second walk that produces finished rows,
// the first SCAN_STAGE_ROWS through the buffer, the rest stored directly.
constexpr int SCAN_STAGE_ROWS = (SCAN_EXTRA_BYTES ? SCAN_STAGE_BYTES + SCAN_EXTRA_BYTES : 4096) / 24;   // 301 rows of 24 B
#ifndef SJA_SCAN_STAGED_MAX
#define SJA_SCAN_STAGED_MAX SCAN_STAGE_ROWS
#endif
constexpr int SCAN_STAGED_MAX = SJA_SCAN_STAGED_MAX;   // blocks with more rows take the two-pass route
static_assert(SCAN_STAGED_MAX <= SCAN_STAGE_ROWS, "staged rows must fit the row buffer");
static_assert(SCAN_EXTRA_BYTES == 0 || SCAN_STAGES == 2, "the extra region sits between two slots");
static_assert(SCAN_EXTRA_BYTES % 16 == 0, "row buffer alignment");

__global__ void __launch_bounds__(SCAN_WARPS * 32, SCAN_CTAS_PER_SM) scan_profiles_kernel(ScanArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t wid = threadIdx.x >> 5;
    unsigned char* wbase = smem_raw + (size_t)wid * SCAN_WARP_BYTES;
    const uint32_t wbase_s = (uint32_t)__cvta_generic_to_shared(wbase);
    // a load that was rejected by the validation pass, or whose table does not fit the buffers, is not scanned
    if (*reinterpret_cast<volatile const uint32_t*>(a.flags) & (FLAG_BAD_PROFILE | FLAG_NEED_ROWS)) return;
    const uint64_t N_total = __ldg(a.off + a.J);
    const uint32_t n_long = a.flags[1];
    const uint64_t long_thresh = long_job_threshold(N_total, a.J);
    const uint32_t lane_sw = (lane ^ ((lane >> 3) & 3u)) * 16u;   // swz(32 r + lane) * 16 - 512 r
    const uint32_t rd_x = (lane >> 1) & 3u;                        // swz(4 lane + r) = 4 lane + (r ^ rd_x)

    // hand-out order: the listed long jobs first, then all jobs in id order (neighbouring warps stream
    // neighbouring memory), the long ones skipped.  A warp draws its next number when it starts on a job, so
    // that the counter's round trip is over by the time the job is done.
    uint32_t drawn = 0;
    if (lane == 0) drawn = atomicAdd(a.counter, 1u);
    for (;;) {
        const uint32_t c = __shfl_sync(0xFFFFFFFFu, drawn, 0);
        if (lane == 0) drawn = atomicAdd(a.counter, 1u);
        uint32_t j;
        if (c < n_long) {
            j = __ldg(a.long_list + c);
        } else {
            j = c - n_long;
            if (j >= a.J) break;
        }

        const uint64_t js = __ldg(a.off + j), je = __ldg(a.off + j + 1);
        const uint32_t p = a.p0 ? __ldg(a.p0 + j) : 0u;
        const uint64_t s = js + p, e = je;
        if (s >= e) continue;
        if (c >= n_long && e - s > long_thresh) continue;   // scanned in the first phase
        const uint64_t blk0 = s & ~31ull;
        const uint64_t nblk = (e - blk0 + (SCAN_BLK - 1)) / SCAN_BLK;
        const uint64_t out_base = __ldg(a.boff + j);
        const uint64_t out_end = __ldg(a.boff + j + 1);   // rows are never written past this

        // issue the async copies of block t into ring slot t % STAGES
        auto issue = [&](uint64_t t) {
            if (t < nblk) {
                const uint64_t bs = blk0 + t * SCAN_BLK;
                const uint32_t st = wbase_s + (uint32_t)(t % SCAN_STAGES) * (SCAN_STAGE_BYTES + SCAN_EXTRA_BYTES);
                if (bs >= s && bs + SCAN_BLK <= e) {
                    // block entirely inside the job: plain 16-byte copies, no clipping
                    const uint32_t* dp = a.d + bs + 4u * lane;
                    const uint32_t* mp = a.m + bs + 4u * lane;
                    const uint32_t dst = st + lane_sw;
#pragma unroll
                    for (uint32_t r = 0; r < 4; ++r) {
                        cp_async16(dst + r * 512u, dp + r * 128u, 16u);
                        cp_async16(dst + r * 512u + 2048u, mp + r * 128u, 16u);
                    }
                    if (lane < 16) cp_async4(st + 4096u + lane * 4u, a.sbits + (bs >> 5) + lane, 4u);
                } else {
#pragma unroll
                    for (uint32_t r = 0; r < 4; ++r) {
                        const uint32_t c = r * 32u + lane;
                        const uint64_t step = bs + 4ull * c;
                        uint32_t bytes = 0;
                        if (step + 4 > s && step < e) {
                            const uint64_t left = (N_total - step) * 4ull;
                            bytes = left < 16 ? (uint32_t)left : 16u;
                        }
                        const uint64_t src = bytes ? step : 0ull;
                        const uint32_t dst = st + swz(c) * 16u;
                        cp_async16(dst, a.d + src, bytes);
                        cp_async16(dst + 2048u, a.m + src, bytes);
                    }
                    if (lane < 16) {
                        const uint64_t w = (bs >> 5) + lane;
                        const bool ok = (w << 5) < e && ((w << 5) + 32) > s;
                        cp_async4(st + 4096u + lane * 4u, a.sbits + (ok ? w : 0ull), ok ? 4u : 0u);
                    }
                }
            }
            cp_async_commit();
        };

        uint32_t carryD = 0;     // cumulative duration mod 2^32
        uint64_t tot64 = 0;      // exact cumulative duration (overflow check)
        uint64_t carryW = 0;     // cumulative work
        uint32_t carrySeg = 0;   // max m since the last boundary
        uint32_t carryRun = 0;   // max m over all finished segments since the progress point
        uint32_t outpos = 0;     // rows written so far

#pragma unroll
        for (int t = 0; t < SCAN_STAGES - 1; ++t) issue((uint64_t)t);

        for (uint64_t t = 0; t < nblk; ++t) {
            issue(t + SCAN_STAGES - 1);
            cp_async_wait<SCAN_STAGES - 1>();
            __syncwarp();

            unsigned char* st = wbase + (size_t)(t % SCAN_STAGES) * (SCAN_STAGE_BYTES + SCAN_EXTRA_BYTES);
            const uint4* sd = reinterpret_cast<const uint4*>(st);
            const uint4* sm = reinterpret_cast<const uint4*>(st + 2048);
            const uint32_t* ss = reinterpret_cast<const uint32_t*>(st + 4096);
            uint32_t dv[16], mv[16];
#pragma unroll
            for (uint32_t r = 0; r < 4; ++r) {
                const uint32_t ph = 4u * lane + (r ^ rd_x);
                const uint4 qd = sd[ph];
                const uint4 qm = sm[ph];
                dv[4 * r + 0] = qd.x; dv[4 * r + 1] = qd.y; dv[4 * r + 2] = qd.z; dv[4 * r + 3] = qd.w;
                mv[4 * r + 0] = qm.x; mv[4 * r + 1] = qm.y; mv[4 * r + 2] = qm.z; mv[4 * r + 3] = qm.w;
            }
            uint32_t bits = (ss[lane >> 1] >> ((lane & 1u) * 16u)) & 0xFFFFu;
            __syncwarp();  // every lane has read the slot: it may now be reused as the row buffer

            const uint64_t bs = blk0 + t * SCAN_BLK;
            const uint64_t lane_base = bs + 16ull * lane;
            if (!(bs >= s && bs + SCAN_BLK < e)) {
                // first / last block of the job: clip to [s, e), force the end-of-job boundary
                uint32_t lo = 0, hi = 16;
                if (s > lane_base) lo = (s - lane_base) >= 16 ? 16u : (uint32_t)(s - lane_base);
                if (e < lane_base + 16) hi = (e <= lane_base) ? 0u : (uint32_t)(e - lane_base);
                const uint32_t vm = (hi > lo) ? (((1u << hi) - 1u) & ~((1u << lo) - 1u)) : 0u;
                if (vm != 0xFFFFu) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (!((vm >> i) & 1u)) { dv[i] = 0; mv[i] = 0; }
                }
                bits &= vm;
                if (e - 1 >= lane_base && e - 1 < lane_base + 16) bits |= 1u << (uint32_t)(e - 1 - lane_base);
            }
            const uint32_t k0 = (uint32_t)(lane_base - js);   // steps of the job before this lane

            // rows of this block: exclusive count per lane, total
            const uint32_t cnt = __popc(bits);
            uint32_t incC = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t yc = __shfl_up_sync(0xFFFFFFFFu, incC, o);
                if (lane >= (uint32_t)o) incC += yc;
            }
            const uint32_t c_total = __shfl_sync(0xFFFFFFFFu, incC, 31);
            const bool staged = c_total <= (uint32_t)SCAN_STAGED_MAX;   // warp-uniform

            // the row buffer: the consumed slot, plus the extra region next to it (behind slot 0, before slot 1)
            unsigned char* rbuf = (SCAN_EXTRA_BYTES && (t % SCAN_STAGES)) ? st - SCAN_EXTRA_BYTES : st;
            uint4* rowA = reinterpret_cast<uint4*>(rbuf);
            uint2* rowB = reinterpret_cast<uint2*>(rbuf + 16 * SCAN_STAGE_ROWS);

            // ---- walk the 16 steps: lane totals, and (staged route) lane-relative rows
            uint32_t td = 0, tail = 0, orv = 0;
            uint64_t tw = 0;
            if (staged) {
                uint32_t lpos = incC - cnt;
                uint32_t meta = lane | 256u;   // bit 8: first row of this lane (takes the carried-in segment)
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    td += dv[i];
                    tw += (uint64_t)dv[i] * (uint64_t)mv[i];
                    tail = max(tail, mv[i]);
                    orv |= dv[i];
                    if ((bits >> i) & 1u) {
                        rowA[lpos] = make_uint4(td, meta, (uint32_t)tw, (uint32_t)(tw >> 32));
                        rowB[lpos] = make_uint2(k0 + (uint32_t)i + 1u, tail);
                        ++lpos;
                        tail = 0;
                        meta = lane;
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    td += dv[i];
                    tw += (uint64_t)dv[i] * (uint64_t)mv[i];
                    tail = max(tail, mv[i]);
                    orv |= dv[i];
                    if ((bits >> i) & 1u) tail = 0;
                }
            }

            // ---- warp combine of the lane totals
            uint32_t incD = td;
            uint64_t incW = tw;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t yd = __shfl_up_sync(0xFFFFFFFFu, incD, o);
                const uint64_t yw = __shfl_up_sync(0xFFFFFFFFu, incW, o);
                if (lane >= (uint32_t)o) { incD += yd; incW += yw; }
            }
            // exact block duration for the overflow check.  If every d < 2^22 the 32-bit block
            // sum cannot wrap (512 * 2^22 = 2^31); otherwise sum the lanes exactly in 64 bits.
            uint64_t blockD = __shfl_sync(0xFFFFFFFFu, incD, 31);
            if (__reduce_or_sync(0xFFFFFFFFu, orv) >= (1u << 22)) {
                uint64_t t64 = 0;
#pragma unroll
                for (int i = 0; i < 16; ++i) t64 += dv[i];
                const uint32_t sum_lo = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)(t64 & 0xFFFFu));
                const uint32_t sum_hi = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)(t64 >> 16));
                blockD = ((uint64_t)sum_hi << 16) + sum_lo;
            }
            // segmented max of the lane tails: a lane with a safe bit starts a new segment
            const uint32_t hm = __ballot_sync(0xFFFFFFFFu, bits != 0u);
            const uint32_t below = hm & (0xFFFFFFFFu >> (31u - lane));   // lanes 0..lane
            const int head = below ? (31 - __clz((int)below)) : -1;
            uint32_t x = tail;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                if ((int)lane - o >= head && (int)lane >= o) x = max(x, y);
            }
            uint32_t seg_in = __shfl_up_sync(0xFFFFFFFFu, x, 1);
            const bool none_before = (hm & ((1u << lane) - 1u)) == 0u;   // no boundary in lanes < lane
            if (lane == 0) seg_in = carrySeg;
            else if (none_before) seg_in = max(seg_in, carrySeg);
            const uint32_t baseD = carryD + (incD - td);     // duration before this lane's first step
            const uint64_t baseW = carryW + (incW - tw);
            const uint64_t out0 = out_base + outpos;

            if (staged) {
                __syncwarp();   // all lanes' rows are in the buffer
                uint32_t runc = carryRun;
                for (uint32_t rb = 0; rb < c_total; rb += 32) {
                    const uint32_t idx = rb + lane;
                    const bool ok = idx < c_total;
                    uint4 ra = make_uint4(0, 0, 0, 0);
                    uint2 rbv = make_uint2(0, 0);
                    if (ok) { ra = rowA[idx]; rbv = rowB[idx]; }
                    const uint32_t src = ra.y & 31u;
                    const uint32_t sD = __shfl_sync(0xFFFFFFFFu, baseD, src);
                    const uint64_t sW = __shfl_sync(0xFFFFFFFFu, baseW, src);
                    const uint32_t sS = __shfl_sync(0xFFFFFFFFu, seg_in, src);
                    const uint32_t segr = (ra.y & 256u) ? max(rbv.y, sS) : rbv.y;
                    uint32_t v = ok ? segr : 0u;      // running max = prefix max over the rows' segment maxima
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, v, o);
                        if (lane >= (uint32_t)o) v = max(v, y);
                    }
                    v = max(v, runc);
                    const uint64_t W = pack64(ra.z, ra.w) + sW;
                    const uint64_t pos = out0 + idx;
                    if (ok && pos < out_end) {
                        a.A[pos] = make_uint4(ra.x + sD, v, (uint32_t)W, (uint32_t)(W >> 32));
                        a.B[pos] = make_uint2(rbv.x, segr);
                    }
                    runc = __shfl_sync(0xFFFFFFFFu, v, 31);
                }
                carryRun = runc;
            } else {
                // two-pass route: per-lane running maximum needs the exclusive prefix max of the
                // lane maxima (everything before this lane counts, finished segment or not)
                uint32_t lmax = 0;
#pragma unroll
                for (int i = 0; i < 16; ++i) lmax = max(lmax, mv[i]);
                uint32_t incR = lmax;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t yr = __shfl_up_sync(0xFFFFFFFFu, incR, o);
                    if (lane >= (uint32_t)o) incR = max(incR, yr);
                }
                const uint32_t before = max(carryRun, carrySeg);
                uint32_t run = __shfl_up_sync(0xFFFFFFFFu, incR, 1);
                run = (lane == 0) ? before : max(run, before);
                uint32_t D = baseD;
                uint64_t W = baseW;
                uint32_t seg = seg_in;
                // finished rows: the first SCAN_STAGE_ROWS go through the row buffer and leave with
                // coalesced stores, the rest is stored directly
                uint32_t lpos = incC - cnt;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    D += dv[i];
                    W += (uint64_t)dv[i] * (uint64_t)mv[i];
                    seg = max(seg, mv[i]);
                    run = max(run, mv[i]);
                    if ((bits >> i) & 1u) {
                        const uint4 ra = make_uint4(D, run, (uint32_t)W, (uint32_t)(W >> 32));
                        const uint2 rb = make_uint2(k0 + (uint32_t)i + 1u, seg);
                        if (lpos < (uint32_t)SCAN_STAGE_ROWS) {
                            rowA[lpos] = ra;
                            rowB[lpos] = rb;
                        } else if (out0 + lpos < out_end) {
                            a.A[out0 + lpos] = ra;
                            a.B[out0 + lpos] = rb;
                        }
                        ++lpos;
                        seg = 0;
                    }
                }
                __syncwarp();
                for (uint32_t idx = lane; idx < (uint32_t)SCAN_STAGE_ROWS; idx += 32) {
                    if (out0 + idx < out_end) {
                        a.A[out0 + idx] = rowA[idx];
                        a.B[out0 + idx] = rowB[idx];
                    }
                }
                carryRun = max(before, __shfl_sync(0xFFFFFFFFu, incR, 31));
            }

            // ---- carries for the next block
            carryD += __shfl_sync(0xFFFFFFFFu, incD, 31);
            carryW += __shfl_sync(0xFFFFFFFFu, incW, 31);
            outpos += c_total;
            const uint32_t x31 = __shfl_sync(0xFFFFFFFFu, x, 31);
            carrySeg = hm ? x31 : max(x31, carrySeg);
            tot64 += blockD;
            __syncwarp();   // the row buffer is read out before the next copies land in this slot
        }

        if (lane == 0) {
            uint32_t f = 0;
            if (tot64 > 0xFFFFFFFFull) f |= FLAG_OVF_DURATION;
            if (carryW >= (1ull << 63)) f |= FLAG_OVF_WORK;
            if (carryW >= (1ull << KEY_SLA_SHIFT)) f |= FLAG_OVF_SLA;
            if (a.wait) {
                const uint64_t fac = 1ull + (uint64_t)(__ldg(a.wait + j) / 1000u);
                if (__umul64hi(carryW, fac) != 0ull || carryW * fac >= (1ull << 63)) f |= FLAG_OVF_FAIR;
            }
            if ((uint64_t)outpos != out_end - out_base) f |= FLAG_INTERNAL;
            if (f) atomicOr(a.flags, f);
        }
    }
}

}  // namespace sja
