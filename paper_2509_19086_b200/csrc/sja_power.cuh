// Second resource envelope: predicted power per step (Section 4.4, item 1).  Offers may carry a
// power cap; a subjob is admissible only if the maximum of its power trace stays below it.
// The per-row data mirrors the memory columns of the boundary table: for every boundary row
// the maximum over the segment since the previous boundary (Ps) and the running maximum from
// the job's progress point (Pm).
#pragma once
#include "sja_common.cuh"

namespace sja {

// One warp per job: 32 rows at a time, each lane walks the steps of its row's segment, then a
// warp max-scan with a carry turns segment maxima into running maxima.  Rows below the
// progress point are left alone (nothing reads them).  A job whose length in `off` differs
// from the loaded one raises FLAG_BAD_PROFILE.
__global__ void __launch_bounds__(256) scan_power_kernel(
    const uint64_t* __restrict__ off, const uint32_t* __restrict__ power, uint32_t J,
    const uint64_t* __restrict__ boff, const uint32_t* __restrict__ pb, const uint32_t* __restrict__ p,
    const uint2* __restrict__ B, uint2* __restrict__ PW, uint32_t* __restrict__ flags) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (j >= J) return;
    const uint64_t b1 = boff[j + 1], base = boff[j] + pb[j];
    const uint32_t R = (uint32_t)(b1 - base), pj = p[j];
    const uint64_t s0 = off[j], len = off[j + 1] - s0;
    const uint64_t len_loaded = R ? (uint64_t)B[b1 - 1].x : (uint64_t)pj;   // the last row ends with the job
    if (len != len_loaded) {
        if (lane == 0) atomicOr(flags, FLAG_BAD_PROFILE);
        return;
    }
    uint32_t carry = 0;
    for (uint32_t r0 = 0; r0 < R; r0 += 32) {
        const uint32_t r = r0 + lane;
        uint32_t seg = 0;
        if (r < R) {
            const uint32_t a = r ? B[base + r - 1].x : pj, b = B[base + r].x;
            for (uint32_t i = a; i < b; ++i) seg = max(seg, __ldg(power + s0 + i));
        }
        uint32_t run = seg;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, run, o);
            if (lane >= (uint32_t)o) run = max(run, y);
        }
        run = max(run, carry);
        if (r < R) PW[base + r] = make_uint2(run, seg);
        carry = __shfl_sync(0xFFFFFFFFu, run, 31);
    }
}

}  // namespace sja
