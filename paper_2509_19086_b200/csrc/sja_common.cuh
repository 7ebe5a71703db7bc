// Shared device-side definitions of libsja (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace sja {

// Device error / status bits (one u32 word per context, set with atomicOr, read by the host).
enum : uint32_t {
    FLAG_BAD_PROFILE = 1u << 0,   // CSR offsets / progress invalid
    FLAG_OVF_DURATION = 1u << 1,  // a job's total duration does not fit in 32 bits
    FLAG_OVF_WORK = 1u << 2,      // a job's total work >= 2^63
    FLAG_OVF_FAIR = 1u << 3,      // total work * (1 + wait/1000) >= 2^63 for some job
    FLAG_OVF_SLA = 1u << 4,       // total work >= 2^55 for some job (SLA key packing)
    FLAG_OVF_READY = 1u << 5,     // start + dur >= 2^32 at commit
    FLAG_INTERNAL = 1u << 6,      // self-check failed (boundary count mismatch)
    FLAG_NEED_ROWS = 1u << 7,     // the boundary table of this load needs more rows than the buffers given hold
};

constexpr uint32_t SJA_NO_JOB_DEV = 0xFFFFFFFFu;

// Programmatic dependent launch (griddepcontrol, sm_90 and later).  The small kernels of a round follow one another
// in one stream, each reading what the one before wrote, and the gap between two such launches is longer than most
// of them run.  A kernel launched with the programmatic-stream-serialization attribute may be made resident while
// the kernel before it is still running: dep_wait() then holds it until that grid has completed and its writes are
// visible, and dep_launch() tells the hardware that the NEXT kernel in the stream may be brought in.  Every kernel
// that is launched with the attribute calls dep_wait() as its first statement, before any early return (a kernel
// that left without waiting could complete before its predecessor, and release its own successor too early); in a
// kernel launched without the attribute both calls do nothing.
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// A job counts as "long" for the scan's hand-out order when it has more steps left than twice the
// mean job length (and at least 8192): such jobs are scanned first, so that none of them starts late and
// stretches the kernel's tail.  The row-counting kernel lists them, the scan kernel skips them later.
#ifndef SJA_LONG_FACTOR
#define SJA_LONG_FACTOR 2
#endif
__host__ __device__ inline uint64_t long_job_threshold(uint64_t n_steps, uint32_t n_jobs) {
    const uint64_t above = (uint64_t)SJA_LONG_FACTOR * (n_steps / (n_jobs ? n_jobs : 1u));
    return above > 8192ull ? above : 8192ull;
}

// One row of the boundary table, "search" half: everything a feasibility probe reads.
// D = cumulative duration of [p_load, k), M = max m over [p_now, k), W = sum d*m over [p_load, k).
// Stored as uint4 {D, M, W_lo, W_hi}.
// "Aux" half, uint2 {k, S}: k = safe end index (steps from the job's first step),
// S = max m over the segment since the previous boundary.

__device__ __forceinline__ uint64_t pack64(uint32_t lo, uint32_t hi) {
    return (uint64_t)lo | ((uint64_t)hi << 32);
}

// Warp-wide maximum of a u64 (all lanes get the result).
__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
    uint32_t hi = (uint32_t)(v >> 32), lo = (uint32_t)v;
    uint32_t mhi = __reduce_max_sync(0xFFFFFFFFu, hi);
    uint32_t mlo = __reduce_max_sync(0xFFFFFFFFu, hi == mhi ? lo : 0u);
    return pack64(mlo, mhi);
}

constexpr uint64_t KEY_SLA_SHIFT = 55;  // SLA key = 1 + (prio << 55) + work, work < 2^55

// Policy key of an interested job: 0 is reserved for "no candidate".
// kind 0 efficiency, 1 fairness (factor = 1 + wait/1000), 2 SLA (factor = prio): payload = work of the subjob;
// kind 3 tight fit: payload = peak memory of the subjob (the running maximum of its last row).
__device__ __forceinline__ uint64_t policy_key(uint32_t kind, uint64_t payload, uint32_t factor) {
    if (kind == 1) return payload * (uint64_t)factor + 1ull;
    if (kind == 2) return ((uint64_t)factor << KEY_SLA_SHIFT) + payload + 1ull;
    return payload + 1ull;
}

// What policy_key wants from a boundary row {D, M, W_lo, W_hi}: the work above the progress point, or the peak.
__device__ __forceinline__ uint64_t policy_payload(uint32_t kind, const uint4& row, uint64_t Wp) {
    return kind == 3 ? (uint64_t)row.y : pack64(row.z, row.w) - Wp;
}

__device__ __forceinline__ uint64_t key_to_score(uint32_t kind, uint64_t key) {
    uint64_t v = key - 1ull;
    if (kind == 2) v &= (1ull << KEY_SLA_SHIFT) - 1ull;
    return v;
}

}  // namespace sja
