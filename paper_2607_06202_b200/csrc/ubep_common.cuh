// Shared device-side definitions of the dispatch / combine kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ubep {

// Error codes mirrored from the public header (kept numerically identical).
constexpr int kErrCapacity = -3;
constexpr int kErrTimeout = -4;
constexpr int kErrBadIndex = -5;

constexpr int kThreads = 512;          // threads per persistent CTA
constexpr int kWarps = kThreads / 32;
constexpr int kMaxTopk = 32;
constexpr int kMaxChunks = 320;        // scan keeps chunks/32 values per lane in registers
constexpr int kMaxStages = 16;         // rows in the shared-memory ring
constexpr int kRankWordsHost = 4;      // the rank-level fast path handles up to 128 ranks
constexpr int kStealBlock = 2;         // tokens handed out per claim
constexpr int kOutStages = 4;          // FP8, quantising after the layout: quantised rows waiting for their stores
constexpr int kMaxOutStages = 24;      // FP8, quantising beside the layout: at most this many quantised rows wait
constexpr int kFastQuantWarps = 5;     // FP8 in the flag-free kernel with rank-level rows: quantising warps (measured per dispatch of
                                       // 512 / 1024 tokens: 15.5 / 24.3 us with 4, 15.5 / 25.3 with 6, 15.7 / 30.7 with 8, 18.0 / 38.2 with 10)
constexpr int kStorePending = 3;       // FP8: rows whose bulk stores may still be reading shared memory
constexpr int kTraceSlots = 16;        // per-CTA phase time stamps (optional tracing)
constexpr int kModePhased = 1, kModeFused = 2, kModeLocal = 3;
// Every wait in the kernels gives up after this many nanoseconds of wall time.
constexpr unsigned long long kWaitLimitNs = 1500000000ull;

// Everything a dispatch kernel needs, passed by value.
struct Params {
    // problem
    int T, H, E, R, L, k, S, cap, payload, dedup;
    int rowB;        // payload bytes per row: 2H (bf16) or H (FP8)
    int G;           // H / 128 scale groups (FP8)
    int B;           // histogram bins: E expert bins followed by R rank bins
    int nchunks;     // token chunks (contiguous, equal to +-1 token)
    int parts;       // column parts per row: CTA c moves part c % parts of chunk c / parts
    int grid;        // CTAs of the dispatch kernel = nchunks * parts
    unsigned L_magic;  // ceil(2^32 / L): e / L == umulhi(e, L_magic) for e < 65536
    int local_fast;    // flag-free kernel: rank-level fast path (dedup, L < 32, R <= 128)
    int er_cap;      // entries per rank in expert_rows
    unsigned* epoch_ctr;    // device word: dispatches completed on this buffer
    unsigned* done_ticket;  // CTAs of the running dispatch kernel that have finished
    int withhold;    // test hook: chunk whose hist flag is not published (-1 = none)
    // inputs
    const uint16_t* x;
    const int32_t* topk_idx;
    const float* topk_w;
    const int32_t* phys;     // replica table [E_log, C] or null
    const int32_t* ncopies;  // [E_log]
    int E_log, C;
    const int32_t* order_pos;  // [R] position of each rank in the destination-ordering table
    int ordered;               // 1 = a table was set (ubep_set_dest_order): copies are issued in its order
    // arena outputs
    uint8_t* recv_x;
    float* recv_scale;
    int32_t* recv_src_idx;
    float* recv_weight;
    int32_t* recv_topk_idx;
    float* recv_topk_w;
    int32_t* expert_rows;
    int32_t* cnt;
    int32_t* src_offset;
    int32_t* expert_offset;
    int32_t* num_tokens_per_expert;
    int32_t* num_rows_per_rank;
    int32_t* num_tokens_per_rank;
    int32_t* slot_row;   // [T, k] region-local row of each slot, -1 if none
    int32_t* slot_pos;   // [T, k] global row (rank * cap + row) of each slot, -1 if none
    // scratch
    int32_t* chunk_hist;  // [B, nchunks] histogram of every chunk, bin-major
    int32_t* partial;     // [S, B] running chunk histogram at each source-rank boundary
    int32_t* chunk_base;  // [B, nchunks] final base of every bin for every chunk, bin-major
    unsigned* hist_flag;  // [nchunks]
    unsigned* scan_flag;  // [R]
    unsigned* arrival;    // [2, R]
    // token stealing (large T): chunk c's tokens are handed out in blocks through cursor[c],
    // to its owner and, once pos_flag[c] holds the epoch, to CTAs that ran out of work
    int steal;            // 1 = on
    int quant_warps;      // FP8: warps that quantise at most (1 .. kWarps - 2)
    int count_warps;      // FP8 with flags or kernel boundaries: warps 1 .. count_warps compute the layout while the
                          // warps after them already quantise the rows the loader has fetched (0 = all 15 warps
                          // compute the layout and quantise afterwards)
    int prefetch_rows;    // FP8: rows the loader may fetch before the layout is done (the rings bound it as well)
    int32_t* copy_pos;    // [T, k] destinations in issue order (-1 = no copy), for thieves
    unsigned* cursor;     // [nchunks] tokens of the chunk handed out so far
    unsigned* pos_flag;   // [nchunks] == epoch: copy_pos of the chunk is final
    unsigned* claimed;    // [2] tokens handed out in this dispatch (half = epoch & 1)
    int32_t* status;
    unsigned long long* trace;  // optional [nchunks, kTraceSlots] phase stamps in ns, or null
    unsigned ns_per_cycle_q20;  // nanoseconds per SM cycle times 2^20 (the clock the stamps are derived with)
    // ranks on different GPUs (sharded use): this GPU is rank my_rank and moves tokens [tok0, tok1)
    int my_rank, tok0, tok1;
    const long long* peer_delta;  // [R] byte distance from this arena to the arena of rank r
    unsigned* shard_arrival;      // [2] rows announced to this rank so far, rows expected so far
};

// ------------------------------------------------------------------ small helpers

__device__ __forceinline__ int64_t chunk_begin(int c, int T, int n) { return (int64_t)c * T / n; }
__device__ __forceinline__ int src_begin(int s, int T, int S) {
    if ((int64_t)S * T < 0x7fffffffLL) return (int)((unsigned)s * (unsigned)T / (unsigned)S);  // the usual case
    return (int)((int64_t)s * T / S);
}
// Chunk that owns token b: the c with chunk_begin(c) <= b < chunk_begin(c + 1).
__device__ __forceinline__ int chunk_of(int b, int T, int n) {
    return (int)((((int64_t)b + 1) * n - 1) / T);
}

// Records the first asynchronous condition of a call.  Out of line on purpose: it is called from
// many places that almost never take it, and the kernels run every piece of their code once per
// launch, so what they execute has to stay small enough for the instruction cache (measured: a few
// hundred instructions more on the way to the first copy cost the decode-sized dispatch microseconds).
static __device__ __noinline__ void report(int32_t* status, int code) { atomicCAS(status, 0, code); }

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Epoch of the running dispatch: one more than the number of dispatches that ran before.
// Flags must hold this value to count as set, so nothing is ever reset between calls, and a
// captured CUDA graph can be replayed because the value lives on the device.  Thread 0 of
// every CTA reads the counter (acquire, so that nothing below is performed before the read)
// and then takes a ticket; the CTA that takes the last ticket knows that every CTA of this
// launch has read the counter and advances it for the next launch.
__device__ __forceinline__ unsigned read_epoch_and_check_in(const Params& p) {
    unsigned e = ld_acquire(p.epoch_ctr) + 1u;
    if (e == 0u) e = 1u;
    if (atomicAdd(p.done_ticket, 1u) == (unsigned)p.grid - 1u) {
        *p.done_ticket = 0u;
        *p.epoch_ctr = e;
    }
    return e;
}


// The flag-free kernel needs the epoch only to pick the half of the arrival counters it adds to at
// its very end, so it splits read_epoch_and_check_in in three: a relaxed load issued early (nothing
// is ordered against it, so it costs the thread nothing until the value is used), the ticket once
// the value has arrived, and the last CTA's update when the ticket's answer is finally looked at.
__device__ __forceinline__ unsigned ld_relaxed(const unsigned* p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned epoch_from_counter(unsigned ctr) {
    const unsigned e = ctr + 1u;
    return e == 0u ? 1u : e;
}
__device__ __forceinline__ void epoch_finish_check_in(const Params& p, unsigned ticket, unsigned e) {
    if (ticket == (unsigned)p.grid - 1u) {
        *p.done_ticket = 0u;
        *p.epoch_ctr = e;
    }
}

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Optional tracing: per-CTA %globaltimer stamp of a phase boundary.
enum TracePhase { kTrStart = 0, kTrCounted, kTrHistSeen, kTrScanned, kTrScanSeen, kTrFinalized, kTrReady,
                  kTrFirstRow, kTrIssued, kTrStored, kTrEnd };
// The stamps are nanoseconds of the device timer.  Reading that timer is slow enough to show in what
// it measures, so a CTA reads it once, when it starts, and derives later stamps from the SM's cycle
// counter (cheap to read) at the SM clock the host passed in -- exact enough for phase budgets.
__device__ __forceinline__ unsigned long long* trace_origin() {
    __shared__ unsigned long long origin[2];   // device timer and cycle counter at the CTA's start
    return origin;
}
__device__ __forceinline__ unsigned long long trace_ns(const Params& p) {
    const unsigned long long* o = trace_origin();
    return o[0] + (((unsigned long long)(clock64() - (long long)o[1]) * (unsigned long long)p.ns_per_cycle_q20) >> 20);
}
// One thread, before the barrier that lets the CTA's roles go.
__device__ __forceinline__ void trace_begin(const Params& p, int cta) {
    if (!p.trace) return;
    unsigned long long* o = trace_origin();
    o[0] = global_ns();
    o[1] = (unsigned long long)clock64();
    p.trace[(size_t)cta * kTraceSlots + kTrStart] = o[0];
}
__device__ __forceinline__ void trace(const Params& p, int cta, int phase) {
    if (p.trace) p.trace[(size_t)cta * kTraceSlots + phase] = trace_ns(p);
}

// Wait until *flag == epoch.  Gives up after kWaitLimitNs (or as soon as *abort is set) and
// returns false; the caller records the timeout and leaves.
__device__ __forceinline__ bool wait_flag(const unsigned* flag, unsigned epoch, volatile int* abort) {
    if (ld_acquire(flag) == epoch) return true;
    const unsigned long long t_end = global_ns() + kWaitLimitNs;
    unsigned ns = 32;
    for (unsigned i = 1;; ++i) {
        if (ld_acquire(flag) == epoch) return true;
        if (abort && *abort) return false;
        if ((i & 63u) == 0 && global_ns() > t_end) return false;
        __nanosleep(ns);
        if (ns < 256) ns <<= 1;
    }
}

// ------------------------------------------------------------ TMA / mbarrier (PTX)

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Non-blocking test of an mbarrier phase.
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Test of an mbarrier phase that may suspend the thread for up to about `hint_ns` while the phase
// is incomplete, instead of spinning in the issue slots other warps of the CTA need.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity, unsigned hint_ns) {
    unsigned ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Bounded wait on an mbarrier phase; false after kWaitLimitNs or on abort.  Spins: the quickest
// to notice the phase, for a warp whose reaction time is on the critical path.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, volatile int* abort) {
    for (unsigned i = 0; i < 128; ++i)
        if (mbar_test_wait(bar, parity)) return true;
    const unsigned long long t_end = global_ns() + kWaitLimitNs;
    for (unsigned i = 1;; ++i) {
        if (mbar_test_wait(bar, parity)) return true;
        if (abort && *abort) return false;
        if ((i & 63u) == 0 && global_ns() > t_end) return false;
        __nanosleep(40);
    }
}
// The same wait for warps that are many and in no hurry (the quantising warps): suspended by the
// hardware while the phase is incomplete, so that they leave the issue slots to the others.
__device__ __forceinline__ bool mbar_wait_idle(uint64_t* bar, unsigned parity, volatile int* abort) {
    if (mbar_test_wait(bar, parity)) return true;
    const unsigned long long t_end = global_ns() + kWaitLimitNs;
    for (;;) {
        if (mbar_try_wait(bar, parity, 1000u)) return true;
        if (abort && *abort) return false;
        if (global_ns() > t_end) return false;
    }
}
// global -> shared bulk copy, completion counted in bytes on `bar`.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// shared -> global bulk copy, tracked by the thread's bulk async-group.
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_all() {
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Where the dispatch kernel keeps things in dynamic shared memory (byte offsets).
struct SmemPlan {
    int stages, stage_bytes;          // input row ring
    int out_stages, out_stage_bytes;  // FP8: ring of quantised rows
    int map_groups, map_wb, map_bp;   // bin bitmaps: 32-token groups, words of bins, padded bins
    int off_out, off_ids, off_mask, off_bm, off_pos, off_key, off_ord, off_w, off_hist, off_arr, off_order;
    int off_item;                     // per ring stage: where its token comes from, positions of stolen tokens
    int total;
};

// Programmatic dependent launch: a kernel launched with the programmatic-serialization
// attribute may be scheduled while its predecessor in the stream still runs; it must not
// touch anything the predecessor produces before griddep_wait() returns (which is when the
// predecessor has completed and its writes are visible).  griddep_launch() tells the
// scheduler that the next kernel in the stream may start being placed.  Both are no-ops for
// a kernel launched the ordinary way.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Barrier among a subset of the CTA's warps (id 1..15), `nthreads` a multiple of 32.
__device__ __forceinline__ void group_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// The same barrier with an OR-reduction: every thread of the group gets the same answer.
__device__ __forceinline__ bool group_or(int id, int nthreads, bool pred) {
    unsigned r;
    asm volatile(
        "{\n .reg .pred p, q;\n setp.ne.u32 q, %3, 0;\n bar.red.or.pred p, %1, %2, q;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(r)
        : "r"(id), "r"(nthreads), "r"((unsigned)pred)
        : "memory");
    return r != 0;
}

}  // namespace ubep
