// Second resource envelope: predicted power per step (Section 4.4, item 1).  Offers may carry a
// power cap; a subjob is admissible only if the maximum of its power trace stays below it.
// The per-row data mirrors the memory columns of the boundary table: for every boundary row
// the maximum over the segment since the previous boundary (Ps) and the running maximum from
// the job's progress point (Pm).
#pragma once
#include "sja_common.cuh"

namespace sja {

constexpr int POWER_WARPS = 8;          // warps per CTA, each streaming one job at a time
#ifndef SJA_POWER_GROUP
#define SJA_POWER_GROUP 1
#endif
constexpr uint32_t POWER_GROUP = SJA_POWER_GROUP;   // jobs a warp looks at per draw of the long-job pass (at most 32)
constexpr int POWER_BLK = 512;          // steps per warp iteration (16 per lane)
constexpr int POWER_BUF_BYTES = POWER_BLK * 4 + 64;    // a block's trace values + one boundary bit per step
constexpr int POWER_WARP_BYTES = 2 * POWER_BUF_BYTES;  // two blocks in flight per warp

// One warp per job streams the job's part of the trace from its progress point on, 512 steps at a time:
// coalesced 16-byte cp.async copies into one of the warp's two shared-memory blocks (the next block is under way
// while the current one is worked on; chunks XOR-swizzled so that the lanes' 128-bit reads of their 16
// CONSECUTIVE steps are conflict-free), boundary bits of the block from the end indices of the table rows that
// end in it (the next 64 row ends are fetched one block ahead), then the same two-level scheme as the profile
// scan: every lane reduces its 16 steps, the warp combines the lane results with shuffles (running maximum =
// plain prefix maximum, segment maximum = prefix maximum that restarts at every boundary), and every lane walks
// its steps again to emit {Pm, Ps} for the rows that end there.  Rows below the progress point are left alone
// (nothing reads them).  A job whose length in `off` differs from the loaded one raises FLAG_BAD_PROFILE.
#ifndef SJA_POWER_MIN_CTAS
#define SJA_POWER_MIN_CTAS 4
#endif
template <bool DYNAMIC>
__global__ void __launch_bounds__(POWER_WARPS * 32, SJA_POWER_MIN_CTAS) scan_power_kernel(
    const uint64_t* __restrict__ off, const uint32_t* __restrict__ power, uint32_t J,
    const uint64_t* __restrict__ boff, const uint32_t* __restrict__ pb, const uint32_t* __restrict__ p,
    const uint2* __restrict__ B, uint2* __restrict__ PW, uint32_t* __restrict__ flags,
    uint32_t* __restrict__ counters) {
    __shared__ __align__(16) unsigned char smem[POWER_WARPS * POWER_WARP_BYTES];
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    unsigned char* wbase = smem + wid * POWER_WARP_BYTES;
    const uint32_t wbase_s = (uint32_t)__cvta_generic_to_shared(wbase);
    const uint64_t N_total = off[J];
    const uint64_t long_thresh = long_job_threshold(N_total, J);
    // Jobs are handed out by two counters (zeroed before the launch), so that no warp waits on another.  First the
    // jobs with many steps left, so that none of them starts late: a warp draws a small group of jobs, its lanes look
    // at one job each, and the warp streams the long ones among them.  Then all jobs one by one, the long ones
    // skipped; the number of the next job is drawn when the warp starts on one.
    // Without DYNAMIC (no long jobs in the load) the counters are not used: warp w of CTA b takes job 8 b + w.
    uint32_t phase = DYNAMIC ? 0u : 2u, grp = 0, pending = 0;
    uint32_t drawn = 0;
    if (DYNAMIC && lane == 0) drawn = atomicAdd(counters + 1, 1u);
    {
        for (;;) {
            uint32_t j;
            if (!DYNAMIC) {
                if (phase == 3u) break;
                phase = 3u;
                j = blockIdx.x * POWER_WARPS + wid;
                if (j >= J) break;
            } else if (phase == 0u) {
                if (pending == 0u) {
                    uint32_t c = 0;
                    if (lane == 0) c = atomicAdd(counters, 1u);
                    c = __shfl_sync(0xFFFFFFFFu, c, 0);
                    if ((uint64_t)c * POWER_GROUP >= (uint64_t)J) { phase = 1u; continue; }
                    grp = c * POWER_GROUP;
                    const uint32_t jj = grp + lane;
                    bool lng = false;
                    if (lane < POWER_GROUP && jj < J) {
                        const uint64_t l = off[jj + 1] - off[jj];
                        const uint32_t pp = p[jj];
                        lng = l >= (uint64_t)pp && l - pp > long_thresh;
                    }
                    pending = __ballot_sync(0xFFFFFFFFu, lng);
                    if (pending == 0u) continue;
                }
                j = grp + (uint32_t)__ffs((int)pending) - 1u;
                pending &= pending - 1u;
            } else {
                j = __shfl_sync(0xFFFFFFFFu, drawn, 0);
                if (j >= J) break;
                if (lane == 0) drawn = atomicAdd(counters + 1, 1u);
            }
            const uint64_t b1 = boff[j + 1], base = boff[j] + pb[j];
            const uint32_t R = (uint32_t)(b1 - base), pj = p[j];
            const uint64_t s0 = off[j], len = off[j + 1] - s0;
            const uint64_t len_loaded = R ? (uint64_t)B[b1 - 1].x : (uint64_t)pj;   // the last row ends with the job
            if (len != len_loaded) {
                if (lane == 0) atomicOr(flags, FLAG_BAD_PROFILE);
                continue;
            }
            if (R == 0) continue;
            if (DYNAMIC && (len - pj > long_thresh) != (phase == 0u)) continue;
            const uint64_t first = s0 + pj, end = s0 + len;       // global steps [first, end) are scanned
            const uint64_t bs0 = first & ~3ull;                   // blocks start 16-byte aligned
            // everything below counts steps from bs0 in 32 bits (a job has fewer than 2^32 steps)
            const uint32_t lead = (uint32_t)(first - bs0);        // 0..3 steps of the first block precede the scan
            const uint32_t span = (uint32_t)(end - bs0);          // steps from bs0 to the end of the job
            const uint32_t nblk = (span + POWER_BLK - 1) / POWER_BLK;
            const uint32_t* src0 = power + bs0;
            const uint64_t room = N_total - bs0;                  // steps of the trace from bs0 on
            // block t into buffer t & 1: chunk c = steps 4c .. 4c + 3 of the block at swizzled slot c ^ ((c >> 3) & 3);
            // bytes beyond the end of the trace are filled with zeros
            auto stage = [&](uint32_t t) {
                if (t < nblk) {
                    const uint32_t dst = wbase_s + (t & 1u) * POWER_BUF_BYTES;
                    const uint32_t* src = src0 + (size_t)t * POWER_BLK + 4u * lane;
                    if ((uint64_t)(t + 1u) * POWER_BLK <= room) {
                        // the whole block lies inside the trace: plain copies
#pragma unroll
                        for (uint32_t r = 0; r < 4; ++r) {
                            const uint32_t c = r * 32u + lane;
                            cp_async16(dst + (c ^ ((c >> 3) & 3u)) * 16u, src + r * 128u, 16u);
                        }
                    } else {
#pragma unroll
                        for (uint32_t r = 0; r < 4; ++r) {
                            const uint32_t c = r * 32u + lane;
                            const uint64_t g = (uint64_t)t * POWER_BLK + 4ull * c;      // steps from bs0
                            uint32_t bytes = 0;
                            if (g < room) bytes = (room - g) >= 4ull ? 16u : (uint32_t)(room - g) * 4u;
                            cp_async16(dst + (c ^ ((c >> 3) & 3u)) * 16u, bytes ? src + r * 128u : power, bytes);
                        }
                    }
                }
                cp_async_commit();
            };
            // end index of table row r of the job (0 beyond its last row: a real end index is at least 1)
            auto row_end = [&](uint32_t r) -> uint32_t { return r < R ? B[base + r].x : 0u; };

            uint32_t row = 0;               // rows emitted so far
            uint32_t carry_run = 0;         // maximum over all steps scanned so far
            uint32_t carry_seg = 0;         // maximum since the last boundary
            stage(0);
            uint32_t k0 = row_end(lane), k1 = row_end(32u + lane);    // ends of rows row + lane and row + 32 + lane
            // a table row with end index k ends at step k - 1 of the job = step k - 1 - pj + lead from bs0
            const uint32_t k_shift = pj + 1u - lead;      // (lead <= 3 and end indices above pj: no wrap for rows that count)
            uint2* out = PW + base;
            for (uint32_t t = 0; t < nblk; ++t) {
                const uint32_t bs = t * POWER_BLK;        // the block's first step, counted from bs0
                unsigned char* buf = wbase + (size_t)(t & 1u) * POWER_BUF_BYTES;
                const uint4* sv = reinterpret_cast<const uint4*>(buf);
                uint32_t* sbits = reinterpret_cast<uint32_t*>(buf + POWER_BLK * 4);
                stage(t + 1);
                if (lane < 16) sbits[lane] = 0u;
                cp_async_wait<1>();
                __syncwarp();
                // ---- boundary bits: the rows (from `row` on) whose last step lies in this block; row ends ascend, so
                // they are a prefix of the rows still to come
                uint32_t in_block = 0;
                {
                    auto mark = [&](uint32_t k) -> uint32_t {
                        const uint32_t o = k - k_shift - bs;          // offset of the row's last step in this block
                        const bool here = k != 0u && o < (uint32_t)POWER_BLK;   // (earlier rows are emitted, later ones wrap or exceed)
                        if (here) atomicOr(&sbits[o >> 5], 1u << (o & 31u));
                        return (uint32_t)__popc(__ballot_sync(0xFFFFFFFFu, here));
                    };
                    uint32_t f = mark(k0);
                    in_block = f;
                    if (f == 32u) {
                        f = mark(k1);
                        in_block += f;
                        for (uint32_t r0 = row + 64u; f == 32u; r0 += 32u) {     // denser than 64 rows per block: fetch on the spot
                            f = mark(row_end(r0 + lane));
                            in_block += f;
                        }
                    }
                }
                // the row ends the next block will want
                const uint32_t k0n = row_end(row + in_block + lane), k1n = row_end(row + in_block + 32u + lane);
                __syncwarp();
                // ---- the lane's 16 consecutive steps
                uint32_t v[16];
#pragma unroll
                for (uint32_t r = 0; r < 4; ++r) {
                    const uint32_t c = 4u * lane + r;
                    const uint4 q = sv[c ^ ((c >> 3) & 3u)];
                    v[4 * r + 0] = q.x; v[4 * r + 1] = q.y; v[4 * r + 2] = q.z; v[4 * r + 3] = q.w;
                }
                uint32_t bits = (sbits[lane >> 1] >> ((lane & 1u) * 16u)) & 0xFFFFu;
                const uint32_t lane_base = bs + 16u * lane;
                if (lane_base < lead || lane_base + 16u > span) {
                    // steps outside the job's part [lead, span) count as 0 and carry no boundary
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (lane_base + i < lead || lane_base + i >= span) { v[i] = 0u; bits &= ~(1u << i); }
                }
                // first walk: maximum of all 16 steps, maximum since the lane's last boundary
                uint32_t lmax = 0, tail = 0;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    lmax = max(lmax, v[i]);
                    tail = max(tail, v[i]);
                    if ((bits >> i) & 1u) tail = 0;
                }
                // running maximum before this lane: exclusive prefix maximum of the lane maxima
                uint32_t inc = lmax;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                    if (lane >= (uint32_t)o) inc = max(inc, y);
                }
                uint32_t run = __shfl_up_sync(0xFFFFFFFFu, inc, 1);
                run = lane == 0 ? carry_run : max(run, carry_run);
                // maximum since the last boundary before this lane: prefix maximum of the tails that restarts at
                // every lane holding a boundary
                const uint32_t hm = __ballot_sync(0xFFFFFFFFu, bits != 0u);
                const uint32_t below = hm & (0xFFFFFFFFu >> (31u - lane));   // lanes 0..lane
                const int head = below ? (31 - __clz((int)below)) : -1;
                uint32_t x = tail;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                    if ((int)lane - o >= head && (int)lane >= o) x = max(x, y);
                }
                uint32_t seg = __shfl_up_sync(0xFFFFFFFFu, x, 1);
                const bool none_before = (hm & ((1u << lane) - 1u)) == 0u;   // no boundary in lanes < lane
                if (lane == 0) seg = carry_seg;
                else if (none_before) seg = max(seg, carry_seg);
                // rows this lane emits start at: rows of earlier blocks + boundaries of lower lanes
                const uint32_t cnt = __popc(bits);
                uint32_t pos = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, pos, o);
                    if (lane >= (uint32_t)o) pos += y;
                }
                pos = row + pos - cnt;
                // second walk: emit {running maximum, segment maximum} at every boundary (lanes without one skip it)
                if (bits) {
                    uint2* o = out + pos;
                    const uint2* o_end = out + R;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        seg = max(seg, v[i]);
                        run = max(run, v[i]);
                        if ((bits >> i) & 1u) {
                            if (o < o_end) *o = make_uint2(run, seg);
                            ++o;
                            seg = 0;
                        }
                    }
                }
                // carries for the next block
                carry_run = max(carry_run, __shfl_sync(0xFFFFFFFFu, inc, 31));
                const uint32_t x31 = __shfl_sync(0xFFFFFFFFu, x, 31);
                carry_seg = hm ? x31 : max(x31, carry_seg);
                row += in_block;
                k0 = k0n;
                k1 = k1n;
                __syncwarp();   // everybody is done with the block before the one after the next overwrites it
            }
            cp_async_wait<0>();
            __syncwarp();
        }   // jobs of a pass
    }
}

}  // namespace sja
