// One scheduler over several GPUs: the jobs are sharded (contiguous id ranges), the gaps are
// replicated, every GPU selects among its own jobs, and the only exchange of a round is one
// bid per gap and GPU.  A bid carries the local winner with its totally ordered policy key;
// the global winner of a gap is the largest key, ties to the lowest global job id, exactly
// the rule of the single-GPU select.  These kernels build the bids and fold the gathered ones.
#pragma once
#include "sja_round.cuh"

namespace sja {

struct Bid { uint64_t key; uint32_t job, end_step, dur, rank; uint64_t score; };   // same layout as sja_bid

// bid[g] of this GPU from its award of gap g: key 0 = no interested job here.
__global__ void __launch_bounds__(256) make_bids_kernel(const Award* __restrict__ awards, uint32_t G, uint32_t kind,
                                                        const uint8_t* __restrict__ prio, uint32_t job_base,
                                                        uint32_t rank, Bid* __restrict__ bids) {
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= G) return;
    const Award a = awards[g];
    Bid b;
    b.key = 0; b.job = 0xFFFFFFFFu; b.end_step = 0; b.dur = 0; b.rank = rank; b.score = 0;
    if (a.job != 0xFFFFFFFFu) {
        // the reported score is the work (SLA), the peak (tight fit) or the weighted work: key as in select
        const uint32_t factor = kind == 2 ? (uint32_t)prio[a.job] : 1u;
        b.key = kind == 2 ? policy_key(2, a.score, factor) : a.score + 1ull;
        b.job = job_base + a.job;
        b.end_step = a.end_step; b.dur = a.dur; b.score = a.score;
    }
    bids[g] = b;
}

// Fold the bids of all GPUs (all[r * G + g]): accept[g] = 1 iff GPU `my_rank` holds the global winner of gap g;
// global[g] (optional) = the winning award with the global job id.
__global__ void __launch_bounds__(256) reduce_bids_kernel(const Bid* __restrict__ all, uint32_t n_ranks, uint32_t G,
                                                          uint32_t my_rank, uint8_t* __restrict__ accept,
                                                          Award* __restrict__ global) {
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= G) return;
    Bid best = all[g];
    for (uint32_t r = 1; r < n_ranks; ++r) {
        const Bid b = all[(size_t)r * G + g];
        if (b.key > best.key || (b.key == best.key && b.job < best.job)) best = b;
    }
    accept[g] = (best.key != 0ull && best.rank == my_rank) ? 1 : 0;
    if (global) {
        Award a;
        a.job = best.key ? best.job : 0xFFFFFFFFu;
        a.end_step = best.end_step; a.dur = best.dur; a.granted = 0; a.score = best.score;
        global[g] = a;
    }
}

}  // namespace sja
