// libsja: C-ABI entry points and host-side orchestration (see include/sja.h).
#include "../../include/sja.h"

#include <cuda_runtime.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "sja_common.cuh"
#include "sja_prep.cuh"
#include "sja_round.cuh"
#include "sja_scan.cuh"
#include "sja_tile.cuh"
#include "sja_update.cuh"
#include "sja_power.cuh"
#include "sja_shard.cuh"

using namespace sja;

// Passes of a re-auction queued between two host waits (four words of the pinned read-back area each).
#ifndef REAUCTION_BATCH
#define REAUCTION_BATCH 16
#endif
// Select grids aim at this many CTAs per SM (several waves even out the tail).
#ifndef SJA_SELECT_CTAS_PER_SM
#define SJA_SELECT_CTAS_PER_SM 8
#endif

namespace {

struct DevBuf {
    void* p = nullptr;
    size_t cap = 0;
    template <class T> T* as() const { return static_cast<T*>(p); }
};

enum ProfCat { CAT_SCAN = 0, CAT_PREP, CAT_ADVERTISE, CAT_SELECT, CAT_COMMIT, CAT_COUNT };

struct ProfSpan { cudaEvent_t a, b; int cat; };

}  // namespace

struct sja_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    char err[320] = {0};
    bool poisoned = false;
    int n_sm = 148;
    int fail_alloc_in = 0;             // sja_debug_fail_alloc: the n-th growing allocation from now fails (0 = off)

    // profiles / scan
    bool loaded = false;
    uint32_t J = 0;
    uint64_t N = 0, n_rows = 0;
    uint32_t n_long = 0;               // jobs the load listed as long (many more steps than the mean)
    bool reauction_later_pass = false; // set by sja_round_reauction around the select of its passes after the first
    bool have_wait = false, have_prio = false;
    uint32_t load_flags = 0;
    DevBuf st_off, st_d, st_m, st_s, st_p, st_ready, st_wait, st_prio;   // staging for host inputs
    DevBuf p, ready, pb, Dp, Wp, wait, prio;          // per-job state and attributes
    DevBuf nbj, cta_tot, cta_base, boff, boff_next, A, B, jobwin;   // row counting scratch, boundary table
    DevBuf flags, counter, n_granted;                 // small device words
    DevBuf long_list;                                 // jobs the scan of a load takes first
    uint32_t* h_words = nullptr;                      // pinned host scratch (128 words)

    // gaps / awards
    bool advertised = false, selected = false, committed = false;
    uint32_t G = 0, last_policy = 0;
    uint32_t tau_min = 0, tau_max = 0xFFFFFFFFu;   // subjob duration thresholds for select
    bool late_start = false, have_deadline = false;   // window options (sja_set_window_options)
    DevBuf deadline;
    uint32_t min_gain = 0;                             // hysteresis threshold (sja_set_hysteresis); 0 = off
    bool have_locality = false;                        // checkpoint sizes and last slices loaded (sja_set_locality)
    uint32_t loc_weight = 0;
    DevBuf ckpt, last_slice;
    bool have_power = false, have_caps = false;        // power envelope (sja_load_power, sja_advertise_power_caps)
    DevBuf PW, caps, st_power;
    DevBuf st_bids, st_accept, st_global;              // sharded rounds: staging for host-side callers
    DevBuf upd_d, upd_m, upd_scratch, upd_status;   // sja_update_profile: staged inputs, segment values, verdict
    bool gaps_sorted = false;          // sgaps is ordered by (C, T); else it is the caller's order
    DevBuf gaps, sgaps, gap_info, gap_rank, awards, widx, partial, winners;
    DevBuf sgaps_alt, blocked, n_active, accept;   // re-auction: second ordered gap list, per-job block flags, gap counter
    DevBuf dirty;                                  // re-auction: job chunks whose candidate rows have to be found again

    // profiling
    int prof = 0;                      // 0 off, 1 every phase, 2 the scan kernel only
    std::vector<ProfSpan> spans;
    std::vector<cudaEvent_t> free_events;
    float acc_ms[CAT_COUNT] = {0};
    uint32_t acc_n[CAT_COUNT] = {0};
};

namespace {

sja_status fail(sja_ctx* c, sja_status st, const char* fmt, ...) {
    if (c) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->err, sizeof(c->err), fmt, ap);
        va_end(ap);
    }
    return st;
}

sja_status cuda_fail(sja_ctx* c, cudaError_t e, const char* what) {
    if (e == cudaErrorMemoryAllocation) {
        cudaGetLastError();
        return fail(c, SJA_ERR_OOM, "%s: out of memory", what);
    }
    if (c) c->poisoned = true;
    return fail(c, SJA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define CU(call)                                                        \
    do {                                                                \
        cudaError_t e__ = (call);                                       \
        if (e__ != cudaSuccess) return cuda_fail(c, e__, #call);        \
    } while (0)

#define TRY(call)                                   \
    do {                                            \
        sja_status s__ = (call);                    \
        if (s__ != SJA_OK) return s__;              \
    } while (0)

// Makes the context's device current for the duration of a call.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; cudaGetLastError(); }
        if (prev != dev) ok = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

// Grow a context buffer (contents are not kept).  The new block is allocated before the old one is let go, so
// a failed allocation leaves the buffer as it was.  `fail_alloc_in` is the host-side fault injector of
// sja_debug_fail_alloc: when it counts down to zero the allocation is reported as failed without being tried.
sja_status reserve(sja_ctx* c, DevBuf& b, size_t bytes) {
    if (bytes <= b.cap) return SJA_OK;
    const size_t want = (bytes + 255) & ~(size_t)255;
    void* fresh = nullptr;
    cudaError_t e = cudaSuccess;
    if (c->fail_alloc_in > 0 && --c->fail_alloc_in == 0) e = cudaErrorMemoryAllocation;
    else e = cudaMalloc(&fresh, want);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMalloc");
    if (b.p) {
        e = cudaStreamSynchronize(c->stream);   // a kernel in flight may still use the old buffer
        if (e == cudaSuccess) e = cudaFree(b.p);
        if (e != cudaSuccess) { cudaFree(fresh); return cuda_fail(c, e, "cudaFree"); }
    }
    b.p = fresh;
    b.cap = want;
    return SJA_OK;
}

void release(DevBuf& b) {
    if (b.p) cudaFree(b.p);
    b.p = nullptr;
    b.cap = 0;
}

struct ProfScope {
    sja_ctx* c;
    ProfSpan sp;
    bool on;
    ProfScope(sja_ctx* ctx, int cat) : c(ctx), on(ctx->prof == 1 || (ctx->prof == 2 && cat == CAT_SCAN)) {
        if (!on) return;
        sp.cat = cat;
        sp.a = take();
        sp.b = take();
        if (!sp.a || !sp.b) { on = false; return; }
        cudaEventRecord(sp.a, c->stream);
    }
    ~ProfScope() {
        if (!on) return;
        cudaEventRecord(sp.b, c->stream);
        c->spans.push_back(sp);
    }
    cudaEvent_t take() {
        if (!c->free_events.empty()) {
            cudaEvent_t e = c->free_events.back();
            c->free_events.pop_back();
            return e;
        }
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return e;
    }
};

sja_status collect_spans(sja_ctx* c) {
    if (c->spans.empty()) return SJA_OK;
    CU(cudaStreamSynchronize(c->stream));
    for (ProfSpan& s : c->spans) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, s.a, s.b) == cudaSuccess) {
            c->acc_ms[s.cat] += ms;
            c->acc_n[s.cat] += 1;
        } else {
            cudaGetLastError();
        }
        c->free_events.push_back(s.a);
        c->free_events.push_back(s.b);
    }
    c->spans.clear();
    return SJA_OK;
}

sja_status check_ctx(sja_ctx* c) {
    if (!c) return SJA_ERR_INVALID_ARG;
    if (c->poisoned) return fail(c, SJA_ERR_CUDA, "context unusable after an earlier CUDA error");
    return SJA_OK;
}

sja_status copy_in(sja_ctx* c, void* dst, const void* src, size_t bytes, sja_memspace where) {
    if (bytes == 0) return SJA_OK;
    CU(cudaMemcpyAsync(dst, src, bytes, where == SJA_MEM_HOST ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice,
                       c->stream));
    return SJA_OK;
}

sja_status copy_out(sja_ctx* c, void* dst, const void* src, size_t bytes, sja_memspace where) {
    if (bytes == 0) return SJA_OK;
    CU(cudaMemcpyAsync(dst, src, bytes, where == SJA_MEM_HOST ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice,
                       c->stream));
    return SJA_OK;
}

// Read the device flag word (waits for the stream).
sja_status read_flags(sja_ctx* c, uint32_t* out) {
    CU(cudaMemcpyAsync(c->h_words, c->flags.p, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    *out = c->h_words[0];
    return SJA_OK;
}

JobView job_view(const sja_ctx* c) {
    JobView v;
    v.boff = c->boff.as<uint64_t>();
    v.pb = c->pb.as<uint32_t>();
    v.Dp = c->Dp.as<uint32_t>();
    v.Wp = c->Wp.as<uint64_t>();
    v.ready = c->ready.as<uint32_t>();
    v.wait = c->have_wait ? c->wait.as<uint32_t>() : nullptr;
    v.prio = c->have_prio ? c->prio.as<uint8_t>() : nullptr;
    v.A = c->A.as<uint4>();
    v.B = c->B.as<uint2>();
    v.blocked = nullptr;
    v.tau_min = c->tau_min;
    v.tau_max = c->tau_max;
    v.deadline = c->have_deadline ? c->deadline.as<uint32_t>() : nullptr;
    v.late_start = c->late_start ? 1u : 0u;
    v.PW = (c->have_power && c->have_caps) ? c->PW.as<uint2>() : nullptr;
    v.caps = (c->have_power && c->have_caps) ? c->caps.as<uint32_t>() : nullptr;
    v.min_gain = c->min_gain;
    v.ckpt = c->have_locality ? c->ckpt.as<uint32_t>() : nullptr;
    v.last_slice = c->have_locality ? c->last_slice.as<uint32_t>() : nullptr;
    v.loc_weight = c->loc_weight;
    v.gaps_orig = c->gaps.as<uint4>();
    v.J = c->J;
    return v;
}

// De-interleave the boundary table for sja_get_scan.
__global__ void export_rows_kernel(const uint4* __restrict__ A, const uint2* __restrict__ B, uint64_t n,
                                   uint32_t* k, uint32_t* D, uint32_t* M, uint32_t* S, uint64_t* W) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint4 a = A[i];
    const uint2 b = B[i];
    if (k) k[i] = b.x;
    if (D) D[i] = a.x;
    if (M) M[i] = a.y;
    if (S) S[i] = b.y;
    if (W) W[i] = pack64(a.z, a.w);
}

// Launch a kernel of the round so that it may be brought onto the GPU while the kernel before it in the stream is
// still running (programmatic dependent launch): all kernels launched here begin with dep_wait(), which holds them
// until that kernel has completed and its writes are visible.  The launch gap between two small dependent
// kernels shrinks to what the hardware needs to hand over.
#ifndef SJA_DEP_LAUNCH
#define SJA_DEP_LAUNCH 1
#endif
template <typename... P, typename... A>
void launch_dep(void (*kernel)(P...), dim3 grid, uint32_t threads, size_t smem, cudaStream_t stream, A&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = SJA_DEP_LAUNCH ? 1u : 0u;
    (void)cudaLaunchKernelEx(&cfg, kernel, P(args)...);   // a failure stays in the runtime's last-error slot
}

// The merge and tile kernels are templated on the policy and on whether the subjob duration
// thresholds are in force; these helpers pick the instance.
enum SelectKernel { SEL_TILE = 0, SEL_MERGE = 1, SEL_SEARCH = 2 };

template <uint32_t KIND, bool BOUNDED>
void launch_sorted_kb(SelectKernel which, dim3 grid, cudaStream_t stream, const JobView& jv, const Gap* sgaps,
                      uint32_t G, uint32_t per_split, Partial* partial, const LaunchGate& gate) {
    if (which == SEL_TILE)
        launch_dep(select_tile_kernel<KIND, BOUNDED>, grid, TILE_WARPS * 32, TILE_SMEM_BYTES, stream, jv, sgaps, G,
                   per_split, partial, gate);
    else
        launch_dep(select_merge_kernel<KIND, BOUNDED>, grid, MERGE_WARPS * 32, MERGE_SMEM_BYTES, stream, jv, sgaps, G,
                   per_split, partial, gate);
}

template <bool BOUNDED>
void launch_sorted_b(SelectKernel which, uint32_t kind, dim3 grid, cudaStream_t stream, const JobView& jv,
                     const Gap* sgaps, uint32_t G, uint32_t per_split, Partial* partial, const LaunchGate& gate) {
    if (kind == SJA_POLICY_FAIRNESS)
        launch_sorted_kb<1, BOUNDED>(which, grid, stream, jv, sgaps, G, per_split, partial, gate);
    else if (kind == SJA_POLICY_SLA)
        launch_sorted_kb<2, BOUNDED>(which, grid, stream, jv, sgaps, G, per_split, partial, gate);
    else if (kind == SJA_POLICY_TIGHT_FIT)
        launch_sorted_kb<3, BOUNDED>(which, grid, stream, jv, sgaps, G, per_split, partial, gate);
    else
        launch_sorted_kb<0, BOUNDED>(which, grid, stream, jv, sgaps, G, per_split, partial, gate);
}

void launch_sorted(SelectKernel which, uint32_t kind, dim3 grid, cudaStream_t stream, const JobView& jv,
                   const Gap* sgaps, uint32_t G, uint32_t per_split, Partial* partial, const LaunchGate& gate) {
    if (jv.tau_min != 0u || jv.tau_max != 0xFFFFFFFFu)
        launch_sorted_b<true>(which, kind, grid, stream, jv, sgaps, G, per_split, partial, gate);
    else
        launch_sorted_b<false>(which, kind, grid, stream, jv, sgaps, G, per_split, partial, gate);
}

template <uint32_t KIND, bool BOUNDED>
cudaError_t sorted_smem_attr() {
    cudaError_t e = cudaFuncSetAttribute(select_merge_kernel<KIND, BOUNDED>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, MERGE_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(select_tile_kernel<KIND, BOUNDED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                TILE_SMEM_BYTES);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

// Policy argument checks shared by the select entry points.
sja_status check_policy(sja_ctx* c, const sja_policy* policy, const char* who) {
    if (!policy) return fail(c, SJA_ERR_INVALID_ARG, "%s: policy is NULL", who);
    const uint32_t kind = policy->kind;
    if (kind > SJA_POLICY_TIGHT_FIT) return fail(c, SJA_ERR_INVALID_ARG, "%s: unknown policy %u", who, kind);
    if (!c->loaded || !c->advertised) return fail(c, SJA_ERR_STATE, "%s before load / advertise", who);
    if (kind == SJA_POLICY_FAIRNESS && !c->have_wait)
        return fail(c, SJA_ERR_INVALID_ARG, "fairness policy needs wait_ms at load");
    if (kind == SJA_POLICY_SLA && !c->have_prio) return fail(c, SJA_ERR_INVALID_ARG, "SLA policy needs prio at load");
    if (kind == SJA_POLICY_FAIRNESS && (c->load_flags & FLAG_OVF_FAIR))
        return fail(c, SJA_ERR_OVERFLOW, "fairness score may reach 2^63 for some job");
    if (kind == SJA_POLICY_SLA && (c->load_flags & FLAG_OVF_SLA))
        return fail(c, SJA_ERR_OVERFLOW, "SLA key needs work < 2^55 for every job");
    return SJA_OK;
}

// Launch signal + score + select for the first G_act entries of `sgaps` (ordered or not);
// awards and widx are written at the gaps' original indices.  `blocked` may be nullptr.
//
// Which kernel: the per-pair search alone where only it can serve the round (it is asked for, a window option or
// power caps are in force, the batch is not ordered) or where the round is small; else an ordered-gap kernel
// (tile sweep, or the merge kernel on request) AND the search kernel behind it: the number of capacity classes
// of the batch lives in device memory (the host does not wait for sja_advertise), so both are queued and each
// looks at the count -- with very many classes the ordered-gap kernels would pay one cursor restart per class,
// and the search serves the round instead.
struct KernelPlan { SelectKernel kernel; uint32_t jobs_per_cta, n_chunks, splits, per_split; };
struct SelectPlan { KernelPlan primary, alt; bool have_alt; uint32_t max_classes; uint32_t rows; };

// `fixed`: the passes of a re-auction keep the candidate rows of untouched job chunks from pass to pass, so the
// kernel and its chunk size must not change with the number of gaps left.
#ifndef SJA_REAUC_SPLIT_GAPS
#define SJA_REAUC_SPLIT_GAPS 256
#endif
KernelPlan plan_kernel(const sja_ctx* c, SelectKernel k, uint32_t G_act, bool fixed) {
    KernelPlan p;
    p.kernel = k;
    // the search kernel gives every gap a thread: with few gaps it takes small job chunks, so that many CTAs share the jobs
    p.jobs_per_cta = k == SEL_TILE ? (uint32_t)TILE_JOBS : k == SEL_MERGE ? (uint32_t)MERGE_JOBS
                     : (G_act <= 64u && !fixed) ? 32u : (uint32_t)SEARCH_JOBS;
    p.n_chunks = (c->J + p.jobs_per_cta - 1) / p.jobs_per_cta;
    // granularity of a gap split: a staging tile; the tile kernel also works in 32-gap steps, which a
    // small problem needs to put enough CTAs on the GPU
    uint32_t tile = k == SEL_TILE ? (uint32_t)TILE_GT : k == SEL_MERGE ? (uint32_t)MERGE_GT : (uint32_t)SEARCH_GT;
    if (k == SEL_TILE && (uint64_t)p.n_chunks * ((G_act + tile - 1) / tile) < (uint64_t)SJA_SELECT_CTAS_PER_SM * c->n_sm)
        tile = 32u;
    // split the gaps so that the grid covers the SMs several times over
    uint32_t splits = (uint32_t)(((uint64_t)SJA_SELECT_CTAS_PER_SM * c->n_sm + p.n_chunks - 1) / p.n_chunks);
    const uint32_t max_splits = (G_act + tile - 1) / tile;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
#if SJA_REAUC_SPLIT_GAPS > 0
    // Later passes of a re-auction evaluate a handful of job chunks only (the others keep their candidate rows):
    // the grid is nearly empty and a pass lasts as long as one CTA needs for its gaps, so the gaps are cut finer.
    if (fixed && c->reauction_later_pass && k != SEL_SEARCH)
        splits = std::min(max_splits, std::max(splits, (G_act + SJA_REAUC_SPLIT_GAPS - 1) / SJA_REAUC_SPLIT_GAPS));
#endif
    uint32_t per_split = (G_act + splits - 1) / splits;
    per_split = ((per_split + tile - 1) / tile) * tile;
    p.per_split = per_split;
    p.splits = (G_act + per_split - 1) / per_split;
    return p;
}

// `classes_known` (>= 0): the class count of the batch as read by the host; the choice is then made here and no
// stand-by launch is needed.
SelectPlan plan_select(const sja_ctx* c, uint32_t pflags, uint32_t G_act, bool fixed = false, int64_t classes_known = -1) {
    SelectPlan p;
    const bool forced = (pflags & (SJA_FLAG_FORCE_MERGE | SJA_FLAG_FORCE_TILE)) != 0;
    // A round of a few thousand pairs cannot fill the GPU either way; there the cursors' sequential walk
    // through each capacity class is pure latency and the independent per-pair searches finish sooner.
    // (a later pass of a re-auction with a handful of gaps left is such a round too, whatever J is: below
    // 2^21 pairs the fixed start-up of the ordered-gap kernels outweighs what they save)
    const bool tiny = (uint64_t)c->J * c->G < (1ull << 16) ||
                      (!fixed && G_act < c->G && (uint64_t)c->J * G_act < (1ull << 21));
    // with a window option the usable window differs from pair to pair: only the search kernel does that
    const bool per_pair_window = c->late_start || c->have_deadline || (c->have_power && c->have_caps) ||
                                 c->min_gain != 0u || c->have_locality;
    p.max_classes = std::max<uint32_t>(64u, c->G / 16u);
    const bool search_only = (pflags & SJA_FLAG_FORCE_SEARCH) || per_pair_window || !c->gaps_sorted || (!forced && tiny) ||
                             (classes_known >= 0 && classes_known > (int64_t)p.max_classes);
    p.have_alt = !search_only && classes_known < 0;
    p.primary = plan_kernel(c, search_only ? SEL_SEARCH : (pflags & SJA_FLAG_FORCE_MERGE) ? SEL_MERGE : SEL_TILE, G_act, fixed);
    p.alt = plan_kernel(c, SEL_SEARCH, G_act, fixed);
    p.rows = p.have_alt ? std::max(p.primary.n_chunks, p.alt.n_chunks) : p.primary.n_chunks;
    return p;
}

// `scratch`: candidate rows (plan rows x G entries); nullptr = the context's own buffer, grown on demand.
// `timed`: record profiling events (creates CUDA events on first use).
// `G_dev`: optional device word with the number of gaps actually left (<= G_act, which then only sizes the launch).
// `dirty` (re-auction only): flags of the 128-job blocks whose chunks have to be evaluated again; the candidate
// rows then have the whole batch as their length, are addressed by original gap index, and `classes_known` is the
// batch's class count as read by the host.
sja_status run_select(sja_ctx* c, uint32_t kind, uint32_t pflags, const Gap* sgaps, uint32_t G_act,
                      const uint32_t* blocked, Partial* scratch = nullptr, bool timed = true,
                      const uint32_t* G_dev = nullptr, const uint32_t* dirty = nullptr, int64_t classes_known = -1) {
    const bool reauction = dirty != nullptr;
    const SelectPlan pl = plan_select(c, pflags, G_act, reauction, classes_known);
    Partial* partial = scratch;
    if (!partial) {
        // (a re-auction sizes the rows for the whole batch before its first pass: nothing grows between passes)
        TRY(reserve(c, c->partial, (size_t)pl.rows * (reauction ? c->G : G_act) * sizeof(Partial)));
        partial = c->partial.as<Partial>();
    }
    const int was_on = c->prof;
    if (!timed) c->prof = 0;
    {
        ProfScope ps(c, CAT_SELECT);
        JobView jv = job_view(c);
        jv.blocked = blocked;
        LaunchGate gate;
        gate.gaps_left = G_dev;
        gate.n_classes = pl.have_alt ? &c->gap_info.as<GapInfo>()->n_classes : nullptr;
        gate.max_classes = pl.max_classes;
        gate.run_if_many = 0u;
        gate.dirty = dirty;
        gate.row_len = reauction ? c->G : 0u;
        gate.stable = reauction ? 1u : 0u;
        auto launch_search = [&](const KernelPlan& kp, const LaunchGate& g) {
            const bool opts = jv.late_start != 0u || jv.deadline != nullptr || jv.PW != nullptr || jv.min_gain != 0u ||
                              jv.ckpt != nullptr;
            if (opts)
                launch_dep(select_search_kernel<true>, dim3(kp.n_chunks, kp.splits), SEARCH_THREADS,
                           jv.PW ? SEARCH_SMEM_BYTES_POWER : SEARCH_SMEM_BYTES, c->stream, jv, sgaps, G_act,
                           kp.per_split, kind, partial, g, kp.jobs_per_cta);
            else
                launch_dep(select_search_kernel<false>, dim3(kp.n_chunks, kp.splits), SEARCH_THREADS, SEARCH_SMEM_BYTES,
                           c->stream, jv, sgaps, G_act, kp.per_split, kind, partial, g, kp.jobs_per_cta);
        };
        if (pl.primary.kernel != SEL_SEARCH)
            launch_sorted(pl.primary.kernel, kind, dim3(pl.primary.n_chunks, pl.primary.splits), c->stream, jv, sgaps,
                          G_act, pl.primary.per_split, partial, gate);
        else
            launch_search(pl.primary, gate);
        if (pl.have_alt) {
            LaunchGate many = gate;
            many.run_if_many = 1u;
            launch_search(pl.alt, many);
        }
        launch_dep(finalize_awards_kernel, dim3((G_act + 31) / 32), FINALIZE_WARPS * 32, 0, c->stream, jv, partial,
                   pl.primary.n_chunks, pl.alt.n_chunks, sgaps, G_act, kind, c->awards.as<Award>(),
                   c->widx.as<uint32_t>(), gate);
    }
    c->prof = was_on;
    return SJA_OK;
}

CommitArgs commit_args(sja_ctx* c, uint32_t* blocked, const uint8_t* accept, uint32_t* dirty_next) {
    CommitArgs a;
    a.awards = c->awards.as<Award>(); a.gaps = c->gaps.as<Gap>(); a.widx = c->widx.as<uint32_t>();
    a.jobwin = c->jobwin.as<unsigned long long>(); a.boff = c->boff.as<uint64_t>();
    a.A = c->A.as<uint4>(); a.B = c->B.as<uint2>();
    a.p = c->p.as<uint32_t>(); a.ready = c->ready.as<uint32_t>(); a.pb = c->pb.as<uint32_t>(); a.Dp = c->Dp.as<uint32_t>();
    a.Wp = c->Wp.as<uint64_t>(); a.winners = c->winners.as<uint32_t>(); a.n_granted = c->n_granted.as<uint32_t>();
    a.flags = c->flags.as<uint32_t>(); a.blocked = blocked; a.accept = accept; a.late_start = c->late_start ? 1u : 0u;
    a.last_slice = c->have_locality ? c->last_slice.as<uint32_t>() : nullptr;
    a.dirty_next = dirty_next;
    a.PW = c->have_power ? c->PW.as<uint2>() : nullptr;
    return a;
}

// Launch the three commit kernels over all G awards.  `blocked` may be nullptr.
void run_commit(sja_ctx* c, uint32_t* blocked, const uint8_t* accept = nullptr, uint32_t* dirty_next = nullptr) {
    const uint32_t G = c->G;
    ProfScope ps(c, CAT_COMMIT);
    const uint32_t gb = (G + 255) / 256;
    const CommitArgs a = commit_args(c, blocked, accept, dirty_next);
    launch_dep(commit_vote_kernel, dim3(gb), 256, 0, c->stream, a.awards, G, a.jobwin, a.n_granted, accept);
    launch_dep(commit_apply_kernel, dim3(gb), 256, 0, c->stream, a, G);
    launch_dep(commit_refresh_kernel, dim3((uint32_t)(((uint64_t)G * 32 + 255) / 256)), 256, 0, c->stream, a.winners,
               a.n_granted, G, a.boff, a.pb, a.A, a.B, a.jobwin, a.PW);
}

// ---------------------------------------------------------------------------------------
// Fixed scratch for sja_select_static: the per-CTA candidate rows of one select call.
// It is part of the loaded module, so every GPU that loads this library holds these bytes
// until the process exits.  In host code the name below is only a handle for the runtime,
// never a device address; the address is looked up once per device by static_scratch_for().
static __device__ __align__(256) unsigned char g_select_scratch[SJA_STATIC_SCRATCH_BYTES];

namespace {

constexpr int STATIC_MAX_DEVICES = 64;
void* g_scratch_addr[STATIC_MAX_DEVICES] = {nullptr};
std::mutex g_scratch_mutex;   // contexts on different host threads may reach the set-up together

// Device address of g_select_scratch on `device`, which must be the current device.
// The first call per device asks the runtime (this loads the module on that device);
// later calls return the cached pointer.
sja_status static_scratch_for(sja_ctx* c, int device, Partial** out) {
    if (device < 0 || device >= STATIC_MAX_DEVICES)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_select_static: device index %d not supported", device);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[device]) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_select_scratch);
        if (e != cudaSuccess) return cuda_fail(c, e, "cudaGetSymbolAddress(g_select_scratch)");
        if (!ptr) return fail(c, SJA_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_scratch_addr[device] = ptr;
    }
    *out = static_cast<Partial*>(g_scratch_addr[device]);
    return SJA_OK;
}

}  // namespace

// =======================================================================================
extern "C" {

sja_status sja_create(sja_ctx** out, int device, void* cuda_stream) {
    if (!out) return SJA_ERR_INVALID_ARG;
    *out = nullptr;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess) { cudaGetLastError(); return SJA_ERR_CUDA; }
    if (device < 0 || device >= n_dev) return SJA_ERR_INVALID_ARG;
    sja_ctx* c = new (std::nothrow) sja_ctx();
    if (!c) return SJA_ERR_OOM;
    c->device = device;
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(device);
    sja_status st = SJA_OK;
    do {
        if (!guard.ok) { st = SJA_ERR_CUDA; break; }
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { st = SJA_ERR_CUDA; break; }
        c->n_sm = prop.multiProcessorCount;
        if (cudaMallocHost(reinterpret_cast<void**>(&c->h_words), 512) != cudaSuccess) { st = SJA_ERR_OOM; break; }
        if ((st = reserve(c, c->flags, 8)) != SJA_OK) break;   // [0] status bits, [1] long-job count of a load
        if ((st = reserve(c, c->counter, 8)) != SJA_OK) break;
        if ((st = reserve(c, c->n_granted, 4)) != SJA_OK) break;
        if (cudaMemsetAsync(c->flags.p, 0, 8, c->stream) != cudaSuccess) { st = SJA_ERR_CUDA; break; }
        if (cudaFuncSetAttribute(scan_profiles_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 SCAN_SMEM_BYTES) != cudaSuccess) { st = SJA_ERR_CUDA; break; }
        if (cudaFuncSetAttribute(select_search_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 SEARCH_SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(select_search_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 SEARCH_SMEM_BYTES_POWER) != cudaSuccess) { st = SJA_ERR_CUDA; break; }
        if (sorted_smem_attr<0, false>() != cudaSuccess || sorted_smem_attr<1, false>() != cudaSuccess ||
            sorted_smem_attr<2, false>() != cudaSuccess || sorted_smem_attr<3, false>() != cudaSuccess ||
            sorted_smem_attr<0, true>() != cudaSuccess || sorted_smem_attr<1, true>() != cudaSuccess ||
            sorted_smem_attr<2, true>() != cudaSuccess || sorted_smem_attr<3, true>() != cudaSuccess) {
            st = SJA_ERR_CUDA;
            break;
        }
        if ((st = reserve(c, c->gap_info, sizeof(GapInfo))) != SJA_OK) break;
    } while (0);
    if (st != SJA_OK) {
        cudaGetLastError();
        sja_destroy(c);
        return st;
    }
    *out = c;
    return SJA_OK;
}

sja_status sja_destroy(sja_ctx* c) {
    if (!c) return SJA_OK;
    DeviceGuard guard(c->device);
    cudaStreamSynchronize(c->stream);
    DevBuf* bufs[] = {&c->st_off, &c->st_d, &c->st_m, &c->st_s, &c->st_p, &c->st_ready, &c->st_wait, &c->st_prio, &c->p, &c->ready, &c->pb, &c->Dp,
                      &c->Wp, &c->wait, &c->prio, &c->nbj, &c->cta_tot, &c->cta_base, &c->boff, &c->boff_next, &c->A, &c->B, &c->jobwin,
                      &c->flags, &c->counter, &c->n_granted, &c->long_list, &c->gaps, &c->sgaps, &c->gap_info, &c->gap_rank, &c->sgaps_alt, &c->dirty, &c->blocked, &c->n_active, &c->accept, &c->deadline, &c->ckpt, &c->last_slice, &c->PW, &c->caps, &c->st_power, &c->st_bids, &c->st_accept, &c->st_global, &c->upd_d, &c->upd_m, &c->upd_scratch, &c->upd_status, &c->awards, &c->widx, &c->partial,
                      &c->winners};
    for (DevBuf* b : bufs) release(*b);
    for (ProfSpan& s : c->spans) { cudaEventDestroy(s.a); cudaEventDestroy(s.b); }
    for (cudaEvent_t e : c->free_events) cudaEventDestroy(e);
    if (c->h_words) cudaFreeHost(c->h_words);
    cudaGetLastError();
    delete c;
    return SJA_OK;
}

const char* sja_last_error(const sja_ctx* c) { return c ? c->err : ""; }

sja_status sja_debug_fail_alloc(sja_ctx* c, int nth) {
    TRY(check_ctx(c));
    if (nth < 0) return fail(c, SJA_ERR_INVALID_ARG, "sja_debug_fail_alloc: nth must be >= 0");
    c->fail_alloc_in = nth;
    return SJA_OK;
}

sja_status sja_profile_enable(sja_ctx* c, int on) {
    TRY(check_ctx(c));
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    TRY(collect_spans(c));
    for (int i = 0; i < CAT_COUNT; ++i) { c->acc_ms[i] = 0.f; c->acc_n[i] = 0; }
    if (on < 0 || on > 2) return fail(c, SJA_ERR_INVALID_ARG, "sja_profile_enable: mode must be 0, 1 or 2");
    c->prof = on;
    return SJA_OK;
}

sja_status sja_profile_read(sja_ctx* c, sja_timing* out) {
    TRY(check_ctx(c));
    if (!out) return fail(c, SJA_ERR_INVALID_ARG, "sja_profile_read: out is NULL");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    TRY(collect_spans(c));
    out->scan_ms = c->acc_ms[CAT_SCAN];
    out->prep_ms = c->acc_ms[CAT_PREP];
    out->advertise_ms = c->acc_ms[CAT_ADVERTISE];
    out->select_ms = c->acc_ms[CAT_SELECT];
    out->commit_ms = c->acc_ms[CAT_COMMIT];
    out->scan_launches = c->acc_n[CAT_SCAN];
    out->prep_launches = c->acc_n[CAT_PREP];
    out->advertise_launches = c->acc_n[CAT_ADVERTISE];
    out->select_launches = c->acc_n[CAT_SELECT];
    out->commit_launches = c->acc_n[CAT_COMMIT];
    return SJA_OK;
}

// ---------------------------------------------------------------------------------------
sja_status sja_load_profiles(sja_ctx* c, uint32_t J, const uint64_t* off, const uint32_t* dur_ms,
                             const uint32_t* mem_MiB, const uint32_t* safe_bits, const uint32_t* ready_ms,
                             const uint32_t* progress, const uint32_t* wait_ms, const uint8_t* prio,
                             sja_memspace where) {
    TRY(check_ctx(c));
    if (J == 0 || J == 0xFFFFFFFFu) return fail(c, SJA_ERR_INVALID_ARG, "sja_load_profiles: J out of range");
    if (!off || !ready_ms) return fail(c, SJA_ERR_INVALID_ARG, "sja_load_profiles: off / ready_ms is NULL");
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_load_profiles: bad memspace");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");

    // N = off[J].  Host arrays: read it here.  Device arrays: the kernels read it themselves and the
    // host learns it together with the validation result, so no extra wait is needed -- unless a
    // profile pointer is NULL, which is only legal for N = 0 and must be known before any launch.
    uint64_t N = 0;
    bool n_known = true;
    if (where == SJA_MEM_HOST) {
        if (off[0] != 0) return fail(c, SJA_ERR_BAD_PROFILE, "off[0] != 0");
        N = off[J];
    } else if (!dur_ms || !mem_MiB || !safe_bits) {
        CU(cudaMemcpyAsync(c->h_words, off + J, 8, cudaMemcpyDeviceToHost, c->stream));
        CU(cudaStreamSynchronize(c->stream));
        memcpy(&N, c->h_words, 8);
    } else {
        n_known = false;
    }
    if (N >= (1ull << 40)) return fail(c, SJA_ERR_BAD_PROFILE, "off[J] = %llu is implausible", (unsigned long long)N);
    if (N > 0 && (!dur_ms || !mem_MiB || !safe_bits))
        return fail(c, SJA_ERR_INVALID_ARG, "sja_load_profiles: profile array is NULL");
    const uint64_t n_words = (N + 31) / 32;

    const uint64_t* d_off = off;
    const uint32_t *d_d = dur_ms, *d_m = mem_MiB, *d_s = safe_bits;
    if (where == SJA_MEM_HOST) {
        TRY(reserve(c, c->st_off, (size_t)(J + 1) * 8));
        TRY(reserve(c, c->st_d, (size_t)N * 4 + 16));
        TRY(reserve(c, c->st_m, (size_t)N * 4 + 16));
        TRY(reserve(c, c->st_s, (size_t)n_words * 4 + 16));
        TRY(copy_in(c, c->st_off.p, off, (size_t)(J + 1) * 8, where));
        TRY(copy_in(c, c->st_d.p, dur_ms, (size_t)N * 4, where));
        TRY(copy_in(c, c->st_m.p, mem_MiB, (size_t)N * 4, where));
        TRY(copy_in(c, c->st_s.p, safe_bits, (size_t)n_words * 4, where));
        d_off = c->st_off.as<uint64_t>();
        d_d = c->st_d.as<uint32_t>();
        d_m = c->st_m.as<uint32_t>();
        d_s = c->st_s.as<uint32_t>();
    } else if ((!n_known || N > 0) && (!aligned16(dur_ms) || !aligned16(mem_MiB) || !aligned16(safe_bits))) {
        return fail(c, SJA_ERR_INVALID_ARG, "sja_load_profiles: device profile arrays must be 16-byte aligned");
    }
    const uint32_t n_count_ctas = (J + COUNT_JOBS_PER_CTA - 1) / COUNT_JOBS_PER_CTA;
    // scratch of the preparation pass and staging of host-side per-job inputs (none of it is loaded state)
    TRY(reserve(c, c->nbj, (size_t)J * 8));                       // per-job row offset inside its counting CTA
    TRY(reserve(c, c->cta_tot, (size_t)n_count_ctas * 8));
    TRY(reserve(c, c->cta_base, (size_t)(n_count_ctas + 1) * 8));
    TRY(reserve(c, c->boff_next, (size_t)(J + 1) * 8));
    TRY(reserve(c, c->long_list, (size_t)J * 4));
    const uint32_t *d_p = progress, *d_ready = ready_ms, *d_wait = wait_ms;
    const uint8_t* d_prio = prio;
    if (where == SJA_MEM_HOST) {
        TRY(reserve(c, c->st_ready, (size_t)J * 4));
        TRY(copy_in(c, c->st_ready.p, ready_ms, (size_t)J * 4, where));
        d_ready = c->st_ready.as<uint32_t>();
        if (progress) {
            TRY(reserve(c, c->st_p, (size_t)J * 4));
            TRY(copy_in(c, c->st_p.p, progress, (size_t)J * 4, where));
            d_p = c->st_p.as<uint32_t>();
        }
        if (wait_ms) {
            TRY(reserve(c, c->st_wait, (size_t)J * 4));
            TRY(copy_in(c, c->st_wait.p, wait_ms, (size_t)J * 4, where));
            d_wait = c->st_wait.as<uint32_t>();
        }
        if (prio) {
            TRY(reserve(c, c->st_prio, (size_t)J));
            TRY(copy_in(c, c->st_prio.p, prio, (size_t)J, where));
            d_prio = c->st_prio.as<uint8_t>();
        }
    }

    // The kernels of a load test the verdict of the validation pass on the device: the state kernel and the
    // scan do nothing for a rejected load or for one whose table outgrows the buffers.  Where the context's
    // buffers are large enough for this J they are therefore launched right behind the validation pass, and
    // the host waits once per load; otherwise it waits for the verdict first, so that a rejected load never
    // costs the previous one its buffers.
    const size_t need4 = (size_t)J * 4, need8 = (size_t)J * 8;
    const bool perjob_ready = c->p.cap >= need4 && c->ready.cap >= need4 && c->pb.cap >= need4 && c->Dp.cap >= need4 &&
                              c->Wp.cap >= need8 && c->jobwin.cap >= need8 &&
                              (!wait_ms || c->wait.cap >= need4) && (!prio || c->prio.cap >= (size_t)J);
    const bool speculate = perjob_ready && c->A.cap >= 32 && c->B.cap >= 24;
    const uint64_t cap_now = speculate ? std::min<uint64_t>(c->A.cap / 16 - 1, c->B.cap / 8 - 2) : 0ull;

    // launched once or twice: row offsets and per-job state, then the scan
    auto launch_state_and_scan = [&](uint64_t cap_rows) -> sja_status {
        {
            ProfScope ps(c, CAT_PREP);
            launch_dep(finish_load_kernel, dim3((J + 255) / 256), 256, 0, c->stream,
                J, n_count_ctas, c->nbj.as<uint64_t>(), c->cta_base.as<uint64_t>(), c->boff_next.as<uint64_t>(), cap_rows,
                d_p, d_ready, d_wait, d_prio, c->p.as<uint32_t>(), c->ready.as<uint32_t>(),
                c->wait.as<uint32_t>(), c->prio.as<uint8_t>(), c->pb.as<uint32_t>(), c->Dp.as<uint32_t>(),
                c->Wp.as<uint64_t>(), c->jobwin.as<unsigned long long>(),
                c->counter.as<uint32_t>(), c->flags.as<uint32_t>());
        }
        ScanArgs a;
        a.off = d_off; a.d = d_d; a.m = d_m; a.sbits = d_s;
        a.p0 = d_p;
        a.wait = wait_ms ? c->wait.as<uint32_t>() : nullptr;
        a.prio = prio ? c->prio.as<uint8_t>() : nullptr;
        a.boff = c->boff_next.as<uint64_t>();
        a.A = c->A.as<uint4>();
        a.B = c->B.as<uint2>();
        a.J = J;
        a.counter = c->counter.as<uint32_t>();
        a.flags = c->flags.as<uint32_t>();
        a.long_list = c->long_list.as<uint32_t>();
        if (!n_known || N > 0) {
            ProfScope ps(c, CAT_SCAN);
            const uint32_t ctas_per_sm = SCAN_CTAS_PER_SM;
            const uint32_t want = (J + SCAN_WARPS - 1) / SCAN_WARPS;
            const uint32_t grid = std::min<uint32_t>(want, (uint32_t)c->n_sm * ctas_per_sm);
            scan_profiles_kernel<<<grid, SCAN_WARPS * 32, SCAN_SMEM_BYTES, c->stream>>>(a);
        }
        CU(cudaGetLastError());
        return SJA_OK;
    };

    // pass 0: validate + count rows, offsets of the counting CTAs; nothing of the loaded
    // state is touched yet
    CU(cudaMemsetAsync(c->flags.p, 0, 8, c->stream));
    {
        ProfScope ps(c, CAT_PREP);
        count_boundaries_kernel<<<n_count_ctas, 256, 0, c->stream>>>(
            d_off, d_s, d_p, J, c->nbj.as<uint64_t>(), c->cta_tot.as<uint64_t>(), c->flags.as<uint32_t>(),
            c->long_list.as<uint32_t>());
        launch_dep(cta_offsets_kernel, dim3(1), 1024, 0, c->stream, c->cta_tot.as<uint64_t>(), n_count_ctas,
                   c->cta_base.as<uint64_t>());
    }
    CU(cudaGetLastError());
    if (speculate) TRY(launch_state_and_scan(cap_now));

    // verdict (waits for the stream): flags, row count and, if not known yet, N
    uint64_t n_rows = 0;
    uint32_t flags = 0;
    CU(cudaMemcpyAsync(c->h_words, c->flags.p, 8, cudaMemcpyDeviceToHost, c->stream));   // status, long jobs listed
    CU(cudaMemcpyAsync(c->h_words + 2, c->cta_base.as<uint64_t>() + n_count_ctas, 8, cudaMemcpyDeviceToHost, c->stream));
    if (!n_known) CU(cudaMemcpyAsync(c->h_words + 4, d_off + J, 8, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    flags = c->h_words[0];
    const uint32_t n_long_jobs = c->h_words[1];
    if (!n_known) {
        memcpy(&N, c->h_words + 4, 8);
        n_known = true;
        if (N >= (1ull << 40) && !(flags & FLAG_BAD_PROFILE))
            return fail(c, SJA_ERR_BAD_PROFILE, "off[J] = %llu is implausible", (unsigned long long)N);
    }
    if (flags & FLAG_BAD_PROFILE)     // a rejected load has touched nothing of the previous one
        return fail(c, SJA_ERR_BAD_PROFILE, "profile CSR invalid (offsets not monotone, job too long, or progress > len)");
    memcpy(&n_rows, c->h_words + 2, 8);

    // from here on the previous load is replaced
    c->loaded = false;
    c->have_deadline = false;                // deadlines, power traces, checkpoint sizes belong to the jobs of a load
    c->have_power = false;
    c->have_locality = false;
    c->advertised = c->selected = c->committed = false;
    if (!speculate || n_rows > cap_now) {
        // buffers too small for this load (the kernels above, if launched, stood still): size them and run
        TRY(reserve(c, c->A, (size_t)n_rows * 16 + 16));
        TRY(reserve(c, c->B, (size_t)n_rows * 8 + 16));
        TRY(reserve(c, c->p, need4));
        TRY(reserve(c, c->ready, need4));
        TRY(reserve(c, c->pb, need4));
        TRY(reserve(c, c->Dp, need4));
        TRY(reserve(c, c->Wp, need8));
        TRY(reserve(c, c->jobwin, need8));
        if (wait_ms) TRY(reserve(c, c->wait, need4));
        if (prio) TRY(reserve(c, c->prio, (size_t)J));
        if (flags & FLAG_NEED_ROWS) {
            // clear that bit alone (the counters of the validation pass behind it stay)
            flags &= ~FLAG_NEED_ROWS;
            c->h_words[8] = flags;
            CU(cudaMemcpyAsync(c->flags.p, c->h_words + 8, 4, cudaMemcpyHostToDevice, c->stream));
        }
        TRY(launch_state_and_scan(~0ull));
        TRY(read_flags(c, &flags));
    }
    std::swap(c->boff, c->boff_next);
    c->J = J;
    c->N = N;
    c->n_rows = n_rows;
    c->have_wait = wait_ms != nullptr;
    c->have_prio = prio != nullptr;
    if (flags & FLAG_INTERNAL) return fail(c, SJA_ERR_CUDA, "scan self-check failed (row count mismatch)");
    if (flags & FLAG_OVF_DURATION) return fail(c, SJA_ERR_OVERFLOW, "a job's total duration does not fit in 32 bits");
    if (flags & FLAG_OVF_WORK) return fail(c, SJA_ERR_OVERFLOW, "a job's total work is >= 2^63");
    c->load_flags = flags;
    c->n_long = n_long_jobs;
    c->loaded = true;
    return SJA_OK;
}

// ---------------------------------------------------------------------------------------
sja_status sja_advertise(sja_ctx* c, uint32_t G, const sja_gap* gaps, sja_memspace where) {
    TRY(check_ctx(c));
    if (G == 0 || !gaps) return fail(c, SJA_ERR_INVALID_ARG, "sja_advertise: no gaps");
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_advertise: bad memspace");
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_advertise before sja_load_profiles");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    // From here on the previous batch is gone, whatever happens below: if growing a buffer fails, a later
    // select or commit must find no batch (SJA_ERR_STATE) rather than buffers that belong to two batches.
    c->advertised = c->selected = c->committed = false;
    c->have_caps = false;      // power caps belong to a batch
    TRY(reserve(c, c->gaps, (size_t)G * sizeof(sja_gap)));
    TRY(reserve(c, c->sgaps, (size_t)G * sizeof(sja_gap)));
    // u32 rank[G] (rounded up to 16 bytes), then u64 tile_key and u32 tile_idx, both padded to whole sort tiles
    const size_t rank_bytes = (((size_t)G * 4 + 15) / 16) * 16;
    TRY(reserve(c, c->gap_rank, rank_bytes + (size_t)((G + SORT_TILE - 1) / SORT_TILE) * SORT_TILE * 12));
    TRY(reserve(c, c->awards, (size_t)G * sizeof(sja_award)));
    TRY(reserve(c, c->widx, (size_t)G * 4));
    TRY(reserve(c, c->winners, (size_t)G * 4));
    const bool sortable = G <= SORT_MAX_GAPS;
    {
        ProfScope ps(c, CAT_ADVERTISE);
        // host batches are copied into the context first; device batches are read in place by the first kernel,
        // which also writes the context's copy (the commit needs the start times after the caller's array is gone)
        const bool dev = where == SJA_MEM_DEVICE;
        if (!dev) TRY(copy_in(c, c->gaps.p, gaps, (size_t)G * sizeof(sja_gap), where));
        const Gap* src = dev ? reinterpret_cast<const Gap*>(gaps) : c->gaps.as<Gap>();
        Gap* keep = dev ? c->gaps.as<Gap>() : nullptr;
        if (sortable) {
            // sorted tiles live behind the ranks in one buffer; the sort kernel clears the ranks and the class counter
            const uint32_t n_tiles = (G + SORT_TILE - 1) / SORT_TILE;
            uint32_t* rank = c->gap_rank.as<uint32_t>();
            uint64_t* tile_key = reinterpret_cast<uint64_t*>(c->gap_rank.as<unsigned char>() + rank_bytes);
            uint32_t* tile_idx = reinterpret_cast<uint32_t*>(tile_key + (size_t)n_tiles * SORT_TILE);
            const bool one_tile = n_tiles == 1;
            launch_dep(sort_gap_tiles_kernel, dim3(n_tiles), SORT_TILE, 0, c->stream, src, G, tile_key, tile_idx, rank,
                       c->gap_info.as<GapInfo>(), one_tile ? c->sgaps.as<Gap>() : nullptr, keep);
            if (!one_tile) {
                launch_dep(rank_gap_tiles_kernel, dim3(n_tiles, n_tiles), SORT_TILE, 0, c->stream, tile_key, tile_idx,
                           rank);
                launch_dep(place_gaps_kernel, dim3((G + 255) / 256), 256, 0, c->stream, src, G, rank,
                           c->sgaps.as<Gap>(), c->gap_info.as<GapInfo>());
            }
        } else {
            launch_dep(copy_gaps_kernel, dim3((G + 255) / 256), 256, 0, c->stream, src, G, c->sgaps.as<Gap>(), keep);
        }
    }
    CU(cudaGetLastError());
    // a host array may be reused as soon as the call returns; a device batch is only queued
    if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));
    c->gaps_sorted = sortable;
    c->G = G;
    c->advertised = true;
    return SJA_OK;
}

// ---------------------------------------------------------------------------------------
sja_status sja_select(sja_ctx* c, const sja_policy* policy, sja_award* out, sja_memspace where) {
    TRY(check_ctx(c));
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_select: bad memspace");
    TRY(check_policy(c, policy, "sja_select"));
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    const uint32_t kind = policy->kind;
    TRY(run_select(c, kind, policy->flags, c->sgaps.as<Gap>(), c->G, nullptr));
    CU(cudaGetLastError());
    c->selected = true;
    c->committed = false;
    c->last_policy = kind;
    if (out) {
        TRY(copy_out(c, out, c->awards.p, (size_t)c->G * sizeof(sja_award), where));
        if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));
    }
    return SJA_OK;
}

// ---------------------------------------------------------------------------------------
// Same work as sja_select, but the candidate rows go to the module's fixed scratch array
// instead of a context buffer, so no allocation can happen on this path: no cudaMalloc,
// no cudaFree, no event creation (kernel timing is therefore not recorded here).
sja_status sja_select_static(sja_ctx* c, const sja_policy* policy, sja_award* out, sja_memspace where) {
    TRY(check_ctx(c));
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_select_static: bad memspace");
    TRY(check_policy(c, policy, "sja_select_static"));
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");

    const uint32_t kind = policy->kind, G = c->G, J = c->J;
    const SelectPlan pl = plan_select(c, policy->flags, G);
    const uint64_t need = (uint64_t)pl.rows * G;   // candidate slots: one per (CTA job chunk, gap)
    const uint64_t have = (uint64_t)SJA_STATIC_SCRATCH_BYTES / sizeof(Partial);
    if (need > have)
        return fail(c, SJA_ERR_INVALID_ARG,
                    "sja_select_static: %u jobs x %u gaps need %llu candidate slots (ceil(J/%u) x G), the fixed "
                    "scratch holds %llu; use sja_select for this size",
                    J, G, (unsigned long long)need,
                    pl.have_alt ? std::min(pl.primary.jobs_per_cta, pl.alt.jobs_per_cta) : pl.primary.jobs_per_cta,
                    (unsigned long long)have);
    Partial* scratch = nullptr;
    TRY(static_scratch_for(c, c->device, &scratch));
    // Every slot that finalize_awards_kernel reads is written by the select kernel of this
    // same call (all chunks x all gaps), so nothing left over from an earlier call is ever
    // read and nothing has to be cleared first.  No profiling events on this path.
    TRY(run_select(c, kind, policy->flags, c->sgaps.as<Gap>(), G, nullptr, scratch, /*timed=*/false));
    CU(cudaGetLastError());
    c->selected = true;
    c->committed = false;
    c->last_policy = kind;
    if (out) {
        TRY(copy_out(c, out, c->awards.p, (size_t)G * sizeof(sja_award), where));
        if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));
    }
    return SJA_OK;
}

// ---------------------------------------------------------------------------------------
static sja_status commit_impl(sja_ctx* c, const uint8_t* accept, uint32_t* n_granted, const char* who) {
    if (!c->selected) return fail(c, SJA_ERR_STATE, "%s without a preceding sja_select", who);
    if (c->committed) return fail(c, SJA_ERR_STATE, "%s: this select was already committed", who);
    run_commit(c, nullptr, accept);
    CU(cudaGetLastError());
    c->committed = true;
    c->selected = false;
    c->advertised = false;   // the granted gaps are used up; advertise the next batch
    if (n_granted) {
        CU(cudaMemcpyAsync(c->h_words, c->n_granted.p, 4, cudaMemcpyDeviceToHost, c->stream));
        CU(cudaMemcpyAsync(c->h_words + 1, c->flags.p, 4, cudaMemcpyDeviceToHost, c->stream));
        CU(cudaStreamSynchronize(c->stream));
        *n_granted = c->h_words[0];
        if (c->h_words[1] & FLAG_OVF_READY) {
            CU(cudaMemsetAsync(c->flags.p, 0, 4, c->stream));
            return fail(c, SJA_ERR_OVERFLOW, "start + dur does not fit in 32 bits for a granted job (ready time saturated)");
        }
    }
    return SJA_OK;
}

sja_status sja_commit(sja_ctx* c, uint32_t* n_granted) {
    TRY(check_ctx(c));
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    return commit_impl(c, nullptr, n_granted, "sja_commit");
}

sja_status sja_commit_masked(sja_ctx* c, const uint8_t* accept, sja_memspace where, uint32_t* n_granted) {
    TRY(check_ctx(c));
    if (!accept) return fail(c, SJA_ERR_INVALID_ARG, "sja_commit_masked: accept is NULL");
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_commit_masked: bad memspace");
    if (!c->selected) return fail(c, SJA_ERR_STATE, "sja_commit_masked without a preceding sja_select");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    TRY(reserve(c, c->accept, c->G));
    TRY(copy_in(c, c->accept.p, accept, c->G, where));
    const sja_status st = commit_impl(c, c->accept.as<uint8_t>(), n_granted, "sja_commit_masked");
    if (st == SJA_OK && where == SJA_MEM_HOST && !n_granted) CU(cudaStreamSynchronize(c->stream));
    return st;
}

// ---------------------------------------------------------------------------------------
sja_status sja_round_reauction(sja_ctx* c, const sja_policy* policy, uint32_t max_passes, uint32_t* n_granted,
                               uint32_t* n_passes) {
    TRY(check_ctx(c));
    TRY(check_policy(c, policy, "sja_round_reauction"));
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    const uint32_t kind = policy->kind, G = c->G, J = c->J;
    TRY(reserve(c, c->sgaps_alt, (size_t)G * sizeof(sja_gap)));
    TRY(reserve(c, c->blocked, (size_t)J * 4));
    CU(cudaMemsetAsync(c->blocked.p, 0, (size_t)J * 4, c->stream));
    // Candidate rows are kept from pass to pass: within a round nothing about a job changes except that granted
    // jobs drop out, so the best candidate of a job chunk for a gap stays the best until one of the chunk's jobs is
    // granted.  Two arrays of flags per block of 128 jobs: the select of a pass evaluates the chunks marked in one,
    // the commit marks the chunks of the jobs it grants in the other, for the next pass.  All marked to begin with.
    const uint32_t n_dirty = ((J + 127u) >> 7) + 8u;
    TRY(reserve(c, c->dirty, (size_t)2 * n_dirty * 4));
    uint32_t* dirty_cur = c->dirty.as<uint32_t>();
    uint32_t* dirty_next = dirty_cur + n_dirty;
    CU(cudaMemsetAsync(dirty_cur, 0xFF, (size_t)n_dirty * 4, c->stream));
    CU(cudaMemsetAsync(dirty_next, 0, (size_t)n_dirty * 4, c->stream));
    // the class count of the batch decides the kernel for every pass: read it once (the call waits for the GPU anyway)
    int64_t classes_known = 0;
    if (c->gaps_sorted) {
        CU(cudaMemcpyAsync(c->h_words + 64, c->gap_info.p, 4, cudaMemcpyDeviceToHost, c->stream));
        CU(cudaStreamSynchronize(c->stream));
        classes_known = c->h_words[64];
    }

    // Passes are queued in batches without a host wait in between: the number of gaps a pass starts with lives
    // in device memory (the report of the pass before it), launches are sized for the count at the last wait
    // (it never grows), and a pass that finds nothing left does nothing.  The merge kernel does not take a
    // device-side count: with SJA_FLAG_FORCE_MERGE every pass is waited for.
    const uint32_t batch_max = (policy->flags & SJA_FLAG_FORCE_MERGE) ? 1u : (uint32_t)REAUCTION_BATCH;
    TRY(reserve(c, c->n_active, (size_t)REAUCTION_BATCH * 16));
    uint32_t* reports = c->n_active.as<uint32_t>();        // 4 words per pass of a batch
    const Gap* cur = c->sgaps.as<Gap>();
    Gap* spare = c->sgaps_alt.as<Gap>();
    Gap* const own = c->sgaps.as<Gap>();   // only ever written as the spare of a later pass, after it was read
    uint32_t g_act = G, total = 0, passes = 0;
    bool overflow = false, done = false;
    while (!done && g_act > 0 && (max_passes == 0 || passes < max_passes)) {
        uint32_t batch = batch_max;
        if (max_passes != 0) batch = std::min(batch, max_passes - passes);
        for (uint32_t k = 0; k < batch; ++k) {
            const uint32_t* g_dev = k ? reports + 4 * (k - 1) : nullptr;   // gaps left after the pass before
            c->reauction_later_pass = passes + k > 0;
            TRY(run_select(c, kind, policy->flags, cur, g_act, c->blocked.as<uint32_t>(), nullptr, true, g_dev, dirty_cur,
                           classes_known));
            {
                // commit of the pass and compaction of its gap list: one launch of one CTA
                ProfScope ps(c, CAT_COMMIT);
                launch_dep(reauction_resolve_kernel, dim3(1), 1024, 0, c->stream,
                           commit_args(c, c->blocked.as<uint32_t>(), nullptr, dirty_next), cur, g_act, spare,
                           reports + 4 * k, g_dev, dirty_cur, n_dirty);
            }
            CU(cudaGetLastError());
            std::swap(dirty_cur, dirty_next);
            cur = spare;
            spare = (spare == c->sgaps_alt.as<Gap>()) ? own : c->sgaps_alt.as<Gap>();
        }
        CU(cudaMemcpyAsync(c->h_words, reports, (size_t)batch * 16, cudaMemcpyDeviceToHost, c->stream));
        CU(cudaStreamSynchronize(c->stream));
        for (uint32_t k = 0; k < batch; ++k) {
            const uint32_t* r = c->h_words + 4 * k;        // orphans left, grants, flags, gaps at the start
            ++passes;
            total += r[1];
            if (r[2] & FLAG_OVF_READY) overflow = true;
            g_act = r[0];
            // nothing granted: no orphan has an interested job left (then none is kept either); nothing left
            if (r[1] == 0 || r[0] == 0) { done = true; break; }
        }
    }
    c->selected = false;
    c->committed = true;
    c->advertised = false;   // sgaps may have been overwritten; advertise the next batch
    c->last_policy = kind;
    if (n_granted) *n_granted = total;
    if (n_passes) *n_passes = passes;
    if (overflow) {
        CU(cudaMemsetAsync(c->flags.p, 0, 4, c->stream));
        return fail(c, SJA_ERR_OVERFLOW, "start + dur does not fit in 32 bits for a granted job (ready time saturated)");
    }
    return SJA_OK;
}

// ---------------------------------------------------------------------------------------
sja_status sja_set_duration_bounds(sja_ctx* c, uint32_t tau_min_ms, uint32_t tau_max_ms) {
    TRY(check_ctx(c));
    if (tau_min_ms > tau_max_ms)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_set_duration_bounds: tau_min %u > tau_max %u", tau_min_ms, tau_max_ms);
    c->tau_min = tau_min_ms;
    c->tau_max = tau_max_ms;
    return SJA_OK;
}

sja_status sja_set_hysteresis(sja_ctx* c, uint32_t min_slack_gain_MiB) {
    TRY(check_ctx(c));
    c->min_gain = min_slack_gain_MiB;
    c->selected = false;   // awards chosen under the old threshold must not be committed under the new one
    return SJA_OK;
}

sja_status sja_set_locality(sja_ctx* c, const uint32_t* ckpt_MiB, const uint32_t* last_slice, uint32_t weight,
                            sja_memspace where) {
    TRY(check_ctx(c));
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_set_locality: bad memspace");
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_set_locality before sja_load_profiles");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    if (ckpt_MiB) {
        TRY(reserve(c, c->ckpt, (size_t)c->J * 4));
        TRY(reserve(c, c->last_slice, (size_t)c->J * 4));
        TRY(copy_in(c, c->ckpt.p, ckpt_MiB, (size_t)c->J * 4, where));
        if (last_slice) TRY(copy_in(c, c->last_slice.p, last_slice, (size_t)c->J * 4, where));
        else CU(cudaMemsetAsync(c->last_slice.p, 0xFF, (size_t)c->J * 4, c->stream));   // nobody has run yet
        if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));   // the caller may reuse its buffers
    }
    c->have_locality = ckpt_MiB != nullptr;
    c->loc_weight = weight;
    c->selected = false;   // awards chosen without the penalty must not be committed with it
    return SJA_OK;
}

sja_status sja_get_locality(sja_ctx* c, uint32_t* last_slice, sja_memspace where) {
    TRY(check_ctx(c));
    if (!last_slice) return fail(c, SJA_ERR_INVALID_ARG, "sja_get_locality: out is NULL");
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_get_locality: bad memspace");
    if (!c->loaded || !c->have_locality) return fail(c, SJA_ERR_STATE, "sja_get_locality before sja_set_locality");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    TRY(copy_out(c, last_slice, c->last_slice.p, (size_t)c->J * 4, where));
    if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));
    return SJA_OK;
}

sja_status sja_update_profile(sja_ctx* c, uint32_t job, uint32_t n_steps, const uint32_t* dur_ms,
                              const uint32_t* mem_MiB, sja_memspace where) {
    TRY(check_ctx(c));
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_update_profile: bad memspace");
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_update_profile before sja_load_profiles");
    if (job >= c->J) return fail(c, SJA_ERR_INVALID_ARG, "sja_update_profile: job %u of %u", job, c->J);
    if (n_steps && (!dur_ms || !mem_MiB)) return fail(c, SJA_ERR_INVALID_ARG, "sja_update_profile: array is NULL");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    const uint32_t *d_d = dur_ms, *d_m = mem_MiB;
    if (where == SJA_MEM_HOST && n_steps) {
        TRY(reserve(c, c->upd_d, (size_t)n_steps * 4));
        TRY(reserve(c, c->upd_m, (size_t)n_steps * 4));
        TRY(copy_in(c, c->upd_d.p, dur_ms, (size_t)n_steps * 4, where));
        TRY(copy_in(c, c->upd_m.p, mem_MiB, (size_t)n_steps * 4, where));
        d_d = c->upd_d.as<uint32_t>();
        d_m = c->upd_m.as<uint32_t>();
    }
    TRY(reserve(c, c->upd_scratch, (size_t)std::max<uint32_t>(n_steps, 1u) * 16));   // a job has at most one row per step
    TRY(reserve(c, c->upd_status, 4));
    CU(cudaMemsetAsync(c->upd_status.p, 0, 4, c->stream));
    UpdateArgs a;
    a.j = job; a.n = n_steps; a.d = d_d; a.m = d_m;
    a.boff = c->boff.as<uint64_t>(); a.pb = c->pb.as<uint32_t>(); a.p = c->p.as<uint32_t>();
    a.Dp = c->Dp.as<uint32_t>(); a.Wp = c->Wp.as<uint64_t>();
    a.wait = c->have_wait ? c->wait.as<uint32_t>() : nullptr;
    a.A = c->A.as<uint4>(); a.B = c->B.as<uint2>();
    a.scratch = c->upd_scratch.as<uint4>();
    a.flags = c->flags.as<uint32_t>();
    a.status = c->upd_status.as<uint32_t>();
    update_profile_kernel<<<1, UPDATE_THREADS, 0, c->stream>>>(a);
    CU(cudaGetLastError());
    CU(cudaMemcpyAsync(c->h_words, c->upd_status.p, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaMemcpyAsync(c->h_words + 1, c->flags.p, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    if (c->h_words[0] == UPD_BAD_SIZE)
        return fail(c, SJA_ERR_BAD_PROFILE, "sja_update_profile: n_steps = %u is not the number of steps job %u has left",
                    n_steps, job);
    if (c->h_words[0] == UPD_OVERFLOW)
        return fail(c, SJA_ERR_OVERFLOW, "sja_update_profile: total duration >= 2^32 ms or total work >= 2^63 for job %u", job);
    c->load_flags |= c->h_words[1] & (FLAG_OVF_FAIR | FLAG_OVF_SLA);
    c->selected = false;   // awards chosen from the old profile must not be committed
    return SJA_OK;
}

static_assert(sizeof(sja_bid) == 32 && sizeof(Bid) == 32, "bid layout");

sja_status sja_get_bids(sja_ctx* c, uint32_t job_base, uint32_t rank, sja_bid* out, sja_memspace where) {
    TRY(check_ctx(c));
    if (!out) return fail(c, SJA_ERR_INVALID_ARG, "sja_get_bids: out is NULL");
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE) return fail(c, SJA_ERR_INVALID_ARG, "sja_get_bids: bad memspace");
    if (!c->selected) return fail(c, SJA_ERR_STATE, "sja_get_bids without a preceding sja_select");
    if ((uint64_t)job_base + c->J > 0xFFFFFFFFull)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_get_bids: job_base + J does not fit a 32-bit job id");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    Bid* d_out = reinterpret_cast<Bid*>(out);
    if (where == SJA_MEM_HOST) {
        TRY(reserve(c, c->st_bids, (size_t)c->G * sizeof(Bid)));
        d_out = c->st_bids.as<Bid>();
    }
    make_bids_kernel<<<(c->G + 255) / 256, 256, 0, c->stream>>>(c->awards.as<Award>(), c->G, c->last_policy,
                                                                c->have_prio ? c->prio.as<uint8_t>() : nullptr,
                                                                job_base, rank, d_out);
    CU(cudaGetLastError());
    if (where == SJA_MEM_HOST) {
        TRY(copy_out(c, out, d_out, (size_t)c->G * sizeof(Bid), where));
        CU(cudaStreamSynchronize(c->stream));
    }
    return SJA_OK;
}

sja_status sja_reduce_bids(sja_ctx* c, uint32_t n_ranks, uint32_t my_rank, const sja_bid* all, uint8_t* accept,
                           sja_award* global_awards, sja_memspace where) {
    TRY(check_ctx(c));
    if (!all || !accept || n_ranks == 0 || my_rank >= n_ranks)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_reduce_bids: bad arguments");
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_reduce_bids: bad memspace");
    if (!c->advertised) return fail(c, SJA_ERR_STATE, "sja_reduce_bids before sja_advertise");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    const uint32_t G = c->G;
    const Bid* d_all = reinterpret_cast<const Bid*>(all);
    uint8_t* d_accept = accept;
    Award* d_global = reinterpret_cast<Award*>(global_awards);
    if (where == SJA_MEM_HOST) {
        TRY(reserve(c, c->st_bids, (size_t)n_ranks * G * sizeof(Bid)));
        TRY(reserve(c, c->st_accept, G));
        TRY(copy_in(c, c->st_bids.p, all, (size_t)n_ranks * G * sizeof(Bid), where));
        d_all = c->st_bids.as<Bid>();
        d_accept = c->st_accept.as<uint8_t>();
        if (global_awards) {
            TRY(reserve(c, c->st_global, (size_t)G * sizeof(Award)));
            d_global = c->st_global.as<Award>();
        }
    }
    reduce_bids_kernel<<<(G + 255) / 256, 256, 0, c->stream>>>(d_all, n_ranks, G, my_rank, d_accept, d_global);
    CU(cudaGetLastError());
    if (where == SJA_MEM_HOST) {
        TRY(copy_out(c, accept, d_accept, G, where));
        if (global_awards) TRY(copy_out(c, global_awards, d_global, (size_t)G * sizeof(Award), where));
        CU(cudaStreamSynchronize(c->stream));
    }
    return SJA_OK;
}

sja_status sja_load_power(sja_ctx* c, const uint64_t* off, const uint32_t* power_W, sja_memspace where) {
    TRY(check_ctx(c));
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_load_power: bad memspace");
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_load_power before sja_load_profiles");
    if (!off || (c->N > 0 && !power_W)) return fail(c, SJA_ERR_INVALID_ARG, "sja_load_power: off / power_W is NULL");
    if (where == SJA_MEM_DEVICE && c->N > 0 && !aligned16(power_W))
        return fail(c, SJA_ERR_INVALID_ARG, "sja_load_power: the device trace must be 16-byte aligned");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    const uint64_t* d_off = off;
    const uint32_t* d_pw = power_W;
    if (where == SJA_MEM_HOST) {
        if (off[0] != 0 || off[c->J] != c->N)
            return fail(c, SJA_ERR_BAD_PROFILE, "sja_load_power: off does not describe the loaded profiles");
        TRY(reserve(c, c->st_off, (size_t)(c->J + 1) * 8));
        TRY(reserve(c, c->st_power, (size_t)c->N * 4 + 16));
        TRY(copy_in(c, c->st_off.p, off, (size_t)(c->J + 1) * 8, where));
        TRY(copy_in(c, c->st_power.p, power_W, (size_t)c->N * 4, where));
        d_off = c->st_off.as<uint64_t>();
        d_pw = c->st_power.as<uint32_t>();
    }
    TRY(reserve(c, c->PW, (size_t)c->n_rows * 8 + 16));
    c->have_power = false;
    c->selected = false;       // awards chosen without the trace must not be committed with it
    {
        ProfScope ps(c, CAT_PREP);
        // Jobs of about equal length: a warp per job, as many CTAs as that takes.  A load that listed long jobs:
        // a persistent grid (as many CTAs as the GPU holds at once) whose warps draw jobs from two counters, the
        // long ones first -- with a warp per job the CTA of a long job would hold seven idle warps' places.
        const uint32_t want = (c->J + POWER_WARPS - 1) / POWER_WARPS;
        uint32_t grid = want;
        if (c->n_long) {
            int per_sm = 0;
            CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, scan_power_kernel<true>, POWER_WARPS * 32, 0));
            grid = std::min<uint32_t>(want, (uint32_t)c->n_sm * (uint32_t)std::max(per_sm, 1));
            CU(cudaMemsetAsync(c->counter.p, 0, 8, c->stream));
            scan_power_kernel<true><<<grid, POWER_WARPS * 32, 0, c->stream>>>(
                d_off, d_pw, c->J, c->boff.as<uint64_t>(), c->pb.as<uint32_t>(), c->p.as<uint32_t>(), c->B.as<uint2>(),
                c->PW.as<uint2>(), c->flags.as<uint32_t>(), c->counter.as<uint32_t>());
        } else {
            scan_power_kernel<false><<<grid, POWER_WARPS * 32, 0, c->stream>>>(
                d_off, d_pw, c->J, c->boff.as<uint64_t>(), c->pb.as<uint32_t>(), c->p.as<uint32_t>(), c->B.as<uint2>(),
                c->PW.as<uint2>(), c->flags.as<uint32_t>(), c->counter.as<uint32_t>());
        }
    }
    CU(cudaGetLastError());
    uint32_t flags = 0;
    TRY(read_flags(c, &flags));
    if (flags & FLAG_BAD_PROFILE) {
        CU(cudaMemsetAsync(c->flags.p, 0, 4, c->stream));   // the bit is only ever set by a load and reported at once
        return fail(c, SJA_ERR_BAD_PROFILE, "sja_load_power: off does not describe the loaded profiles");
    }
    c->have_power = true;
    return SJA_OK;
}

sja_status sja_advertise_power_caps(sja_ctx* c, const uint32_t* cap_W, sja_memspace where) {
    TRY(check_ctx(c));
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_advertise_power_caps: bad memspace");
    if (!c->advertised) return fail(c, SJA_ERR_STATE, "sja_advertise_power_caps before sja_advertise");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    if (cap_W) {
        TRY(reserve(c, c->caps, (size_t)c->G * 4));
        TRY(copy_in(c, c->caps.p, cap_W, (size_t)c->G * 4, where));
        if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));   // the caller may reuse its buffer
    }
    c->have_caps = cap_W != nullptr;
    c->selected = false;       // awards chosen under other caps must not be committed
    return SJA_OK;
}

sja_status sja_set_window_options(sja_ctx* c, uint32_t late_start, const uint32_t* deadline_ms, sja_memspace where) {
    TRY(check_ctx(c));
    if (late_start > 1u) return fail(c, SJA_ERR_INVALID_ARG, "sja_set_window_options: late_start must be 0 or 1");
    if (where != SJA_MEM_HOST && where != SJA_MEM_DEVICE)
        return fail(c, SJA_ERR_INVALID_ARG, "sja_set_window_options: bad memspace");
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_set_window_options before sja_load_profiles");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    if (deadline_ms) {
        TRY(reserve(c, c->deadline, (size_t)c->J * 4));
        TRY(copy_in(c, c->deadline.p, deadline_ms, (size_t)c->J * 4, where));
        if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));   // the caller may reuse its buffer
    }
    c->have_deadline = deadline_ms != nullptr;
    c->late_start = late_start != 0u;
    c->selected = false;   // awards chosen under the old options must not be committed under the new ones
    return SJA_OK;
}

// ---------------------------------------------------------------------------------------
sja_status sja_get_awards(sja_ctx* c, sja_award* out, sja_memspace where) {
    TRY(check_ctx(c));
    if (!out) return fail(c, SJA_ERR_INVALID_ARG, "sja_get_awards: out is NULL");
    if (!c->selected && !c->committed) return fail(c, SJA_ERR_STATE, "sja_get_awards before sja_select");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    TRY(copy_out(c, out, c->awards.p, (size_t)c->G * sizeof(sja_award), where));
    if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));
    return SJA_OK;
}

sja_status sja_get_state(sja_ctx* c, uint32_t* progress, uint32_t* ready_ms, sja_memspace where) {
    TRY(check_ctx(c));
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_get_state before sja_load_profiles");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    if (progress) TRY(copy_out(c, progress, c->p.p, (size_t)c->J * 4, where));
    if (ready_ms) TRY(copy_out(c, ready_ms, c->ready.p, (size_t)c->J * 4, where));
    if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));
    return SJA_OK;
}

sja_status sja_scan_size(sja_ctx* c, uint64_t* n_boundaries) {
    TRY(check_ctx(c));
    if (!n_boundaries) return fail(c, SJA_ERR_INVALID_ARG, "sja_scan_size: out is NULL");
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_scan_size before sja_load_profiles");
    *n_boundaries = c->n_rows;
    return SJA_OK;
}

sja_status sja_get_scan(sja_ctx* c, uint64_t* boff, uint32_t* k, uint32_t* D, uint32_t* M, uint32_t* S,
                        uint64_t* W, sja_memspace where) {
    TRY(check_ctx(c));
    if (!c->loaded) return fail(c, SJA_ERR_STATE, "sja_get_scan before sja_load_profiles");
    DeviceGuard guard(c->device);
    if (!guard.ok) return cuda_fail(c, cudaErrorInvalidDevice, "cudaSetDevice");
    const uint64_t n = c->n_rows;
    if (boff) TRY(copy_out(c, boff, c->boff.p, (size_t)(c->J + 1) * 8, where));
    if (n == 0) {
        if (where == SJA_MEM_HOST) CU(cudaStreamSynchronize(c->stream));
        return SJA_OK;
    }
    uint32_t *dk = k, *dD = D, *dM = M, *dS = S;
    uint64_t* dW = W;
    DevBuf tmp[5];
    sja_status st = SJA_OK;
    if (where == SJA_MEM_HOST) {
        void** outs[5] = {(void**)&dk, (void**)&dD, (void**)&dM, (void**)&dS, (void**)&dW};
        const void* hosts[5] = {k, D, M, S, W};
        const size_t esz[5] = {4, 4, 4, 4, 8};
        for (int i = 0; i < 5 && st == SJA_OK; ++i) {
            if (!hosts[i]) continue;
            st = reserve(c, tmp[i], (size_t)n * esz[i]);
            *outs[i] = tmp[i].p;
        }
    }
    if (st == SJA_OK) {
        const uint64_t blocks = (n + 255) / 256;
        export_rows_kernel<<<(uint32_t)blocks, 256, 0, c->stream>>>(c->A.as<uint4>(), c->B.as<uint2>(), n, dk, dD,
                                                                    dM, dS, dW);
        if (cudaGetLastError() != cudaSuccess) st = fail(c, SJA_ERR_CUDA, "export_rows_kernel launch failed");
    }
    if (st == SJA_OK && where == SJA_MEM_HOST) {
        void* hosts[5] = {k, D, M, S, W};
        const size_t esz[5] = {4, 4, 4, 4, 8};
        for (int i = 0; i < 5; ++i)
            if (hosts[i]) cudaMemcpyAsync(hosts[i], tmp[i].p, (size_t)n * esz[i], cudaMemcpyDeviceToHost, c->stream);
    }
    cudaError_t e = cudaStreamSynchronize(c->stream);
    for (DevBuf& b : tmp) release(b);
    if (st == SJA_OK && e != cudaSuccess) return cuda_fail(c, e, "sja_get_scan");
    return st;
}

}  // extern "C"
