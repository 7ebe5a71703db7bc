// Re-profiling of one job (Section 3.9: segmentation is done at offer time because a job's envelope U(t)
// can change between offers as its predictions improve).  The caller hands in new per-step
// durations and memory values for the steps the job has not been granted yet; its safe
// boundaries stay where they are, so the job keeps its rows of the boundary table and only
// their contents are recomputed: cumulative duration, running maximum from the progress
// point, segment maximum and prefix work.
#pragma once
#include "sja_common.cuh"

namespace sja {

enum : uint32_t { UPD_OK = 0, UPD_BAD_SIZE = 1, UPD_OVERFLOW = 2 };

struct UpdateArgs {
    uint32_t j, n;              // job, number of steps handed in (must equal len_j - p_j)
    const uint32_t* d;          // [n] new durations of steps p_j .. len_j - 1
    const uint32_t* m;          // [n] new memory envelope of the same steps
    const uint64_t* boff;
    const uint32_t* pb;
    const uint32_t* p;
    const uint32_t* Dp;
    const uint64_t* Wp;
    const uint32_t* wait;       // may be nullptr
    uint4* A;
    uint2* B;
    uint4* scratch;             // [>= rows of the job] segment values before anything is written
    uint32_t* flags;            // context flag word (score overflow bits are added)
    uint32_t* status;           // UPD_*
};

constexpr int UPDATE_THREADS = 256;

__device__ __forceinline__ uint64_t sat_add_u64(uint64_t a, uint64_t b) {
    const uint64_t s = a + b;
    return s < a ? ~0ull : s;
}

// One CTA.  Phase 1: one thread per row walks the row's segment of steps.  Phase 2: the totals are
// checked (size, overflow) before a single table entry changes.  Phase 3: inclusive scans over the
// rows in tiles of 256 with running carries, and the rows are rewritten.
__global__ void __launch_bounds__(UPDATE_THREADS) update_profile_kernel(UpdateArgs a) {
    __shared__ uint64_t red_d[UPDATE_THREADS / 32], red_w[UPDATE_THREADS / 32];
    __shared__ uint32_t red_m[UPDATE_THREADS / 32];
    __shared__ uint64_t carry_d, carry_w;
    __shared__ uint32_t carry_m, verdict;
    const uint32_t t = threadIdx.x, lane = t & 31u, wid = t >> 5;
    const uint64_t b0 = a.boff[a.j], b1 = a.boff[a.j + 1];
    const uint32_t pbj = a.pb[a.j], pj = a.p[a.j];
    const uint64_t base = b0 + pbj;
    const uint32_t R = (uint32_t)(b1 - base);                  // rows above the progress point
    const uint32_t len = R ? a.B[b1 - 1].x : pj;               // the last row ends with the job
    if (len - pj != a.n) {
        if (t == 0) *a.status = UPD_BAD_SIZE;
        return;
    }
    // ---- phase 1: per-row segment sums
    uint64_t my_d = 0, my_w = 0;
    for (uint32_t r = t; r < R; r += UPDATE_THREADS) {
        const uint32_t s0 = (r ? a.B[base + r - 1].x : pj) - pj, s1 = a.B[base + r].x - pj;
        uint64_t sd = 0, sw = 0;
        uint32_t mx = 0;
        for (uint32_t i = s0; i < s1; ++i) {
            const uint32_t d = a.d[i], m = a.m[i];
            sd += d;
            sw = sat_add_u64(sw, (uint64_t)d * (uint64_t)m);
            mx = max(mx, m);
        }
        a.scratch[r] = make_uint4((uint32_t)min(sd, (uint64_t)0xFFFFFFFFull), mx, (uint32_t)sw, (uint32_t)(sw >> 32));
        my_d = sat_add_u64(my_d, sd);
        my_w = sat_add_u64(my_w, sw);
    }
    // ---- phase 2: totals and the verdict
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        my_d = sat_add_u64(my_d, __shfl_xor_sync(0xFFFFFFFFu, my_d, o));
        my_w = sat_add_u64(my_w, __shfl_xor_sync(0xFFFFFFFFu, my_w, o));
    }
    if (lane == 0) { red_d[wid] = my_d; red_w[wid] = my_w; }
    __syncthreads();
    if (t == 0) {
        uint64_t td = 0, tw = 0;
        for (int w = 0; w < UPDATE_THREADS / 32; ++w) { td = sat_add_u64(td, red_d[w]); tw = sat_add_u64(tw, red_w[w]); }
        const uint64_t D_end = sat_add_u64(td, a.Dp[a.j]), W_end = sat_add_u64(tw, a.Wp[a.j]);
        uint32_t v = UPD_OK;
        if (D_end > 0xFFFFFFFFull || W_end >= (1ull << 63)) v = UPD_OVERFLOW;
        if (v == UPD_OK) {
            uint32_t f = 0;
            if (W_end >= (1ull << KEY_SLA_SHIFT)) f |= FLAG_OVF_SLA;
            if (a.wait) {
                const uint64_t fac = 1ull + (uint64_t)(a.wait[a.j] / 1000u);
                if (__umul64hi(W_end, fac) != 0ull || W_end * fac >= (1ull << 63)) f |= FLAG_OVF_FAIR;
            }
            if (f) atomicOr(a.flags, f);
        }
        verdict = v;
        *a.status = v;
        carry_d = a.Dp[a.j];
        carry_w = a.Wp[a.j];
        carry_m = 0;
    }
    __syncthreads();
    if (verdict != UPD_OK) return;
    // ---- phase 3: scans over the rows, table rewritten
    for (uint32_t r0 = 0; r0 < R; r0 += UPDATE_THREADS) {
        const uint32_t r = r0 + t;
        uint4 s = make_uint4(0u, 0u, 0u, 0u);
        if (r < R) s = a.scratch[r];
        uint64_t d = s.x, w = pack64(s.z, s.w);
        uint32_t m = s.y;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint64_t d2 = __shfl_up_sync(0xFFFFFFFFu, d, o), w2 = __shfl_up_sync(0xFFFFFFFFu, w, o);
            const uint32_t m2 = __shfl_up_sync(0xFFFFFFFFu, m, o);
            if (lane >= (uint32_t)o) { d += d2; w += w2; m = max(m, m2); }
        }
        if (lane == 31) { red_d[wid] = d; red_w[wid] = w; red_m[wid] = m; }
        __syncthreads();
        uint64_t pd = carry_d, pw = carry_w;
        uint32_t pm = carry_m;
        for (uint32_t q = 0; q < wid; ++q) { pd += red_d[q]; pw += red_w[q]; pm = max(pm, red_m[q]); }
        d += pd; w += pw; m = max(m, pm);
        if (r < R) {
            a.A[base + r] = make_uint4((uint32_t)d, m, (uint32_t)w, (uint32_t)(w >> 32));
            a.B[base + r].y = s.y;
        }
        __syncthreads();
        if (t == UPDATE_THREADS - 1) { carry_d = d; carry_w = w; carry_m = m; }
        __syncthreads();
    }
}

}  // namespace sja
