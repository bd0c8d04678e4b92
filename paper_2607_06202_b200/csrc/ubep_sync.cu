// Dispatch with a selectable readiness protocol (Sec. 3.4 of the paper, "Data-as-Flag
// Synchronization"): stop-and-wait counters, Token-Flag Fusion, Data-for-Checksum and
// Sentinel Polling.  One persistent kernel; every CTA is first a sender (the rows of its
// token chunk) and then a receiver (a slice of one receive region), so the waits of the
// receivers are satisfied by CTAs that never wait themselves.  All CTAs must be resident
// (grid <= number of SMs, one CTA per SM).
//
// The layout (TokenCnt, CalCumSum, slot -> row) is derived by every CTA alone from the
// whole routing table, with the same device functions and in the same order as the
// flag-free instance of the main dispatch kernel, so the two paths leave identical
// metadata in the arena.
//
// A DataBlock is the 16 bytes one thread stores with a single 128-bit access.
#include "ubep_layout.cuh"
#include "ubep_quant.cuh"
#include "ubep_sync.h"

namespace ubep {

namespace {

constexpr int kSW = 0, kTFF = 1, kDC = 2, kSP = 3;
constexpr int kDcBlockVecs = 32;    // 512-byte checksum block = 32 vectors of 16 bytes
constexpr int kDcMarkerVecs = 2;    // its leading 32 bytes are the marker

__device__ __forceinline__ uint4 ld_relaxed_v4(const void* ptr) {
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(ptr)
                 : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_v4(void* ptr, const uint4 v) {
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(ptr), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* ptr) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ bool is_sentinel(const uint4 v) { return (v.x & v.y & v.z & v.w) == 0xffffffffu; }
__device__ __forceinline__ unsigned long long marker_words(const uint4 v) {
    return ((unsigned long long)v.x | ((unsigned long long)v.y << 32)) +
           ((unsigned long long)v.z | ((unsigned long long)v.w << 32));
}

__device__ __forceinline__ unsigned long long warp_sum64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sequence number of the running call, kept on the device like the dispatch epoch: every
// CTA reads the counter and takes a ticket, the last ticket advances the counter.
__device__ __forceinline__ unsigned read_seq_and_check_in(const SyncParams& sp, int grid) {
    unsigned s = ld_acquire(sp.seq_ctr) + 1u;
    if (s == 0u) s = 1u;   // 0 is what a never-written flag holds
    if (atomicAdd(sp.seq_ticket, 1u) == (unsigned)grid - 1u) {
        *sp.seq_ticket = 0u;
        *sp.seq_ctr = s;
    }
    return s;
}

// Bounded polling: give up after kWaitLimitNs or when another thread of the CTA has.
struct Waiter {
    volatile int* abort;
    unsigned long long t_end;
    int32_t* status;
    unsigned* dirty;   // Sentinel Polling: word that tells the next call that this one gave up (else null)
    __device__ __forceinline__ bool keep_waiting(unsigned& spins) {
        __nanosleep(32);
        if ((++spins & 127u) != 0) return true;
        if (*abort) return false;
        if (global_ns() > t_end) {
            *abort = 1;
            report(status, kErrTimeout);
            if (dirty) *dirty = 1u;
            return false;
        }
        return true;
    }
};

__device__ __forceinline__ bool wait_count(const unsigned* ctr, unsigned want, Waiter& wt) {
    unsigned spins = 0;
    while (ld_acquire(ctr) != want)
        if (!wt.keep_waiting(spins)) return false;
    return true;
}

// kFp8: rows travel quantised (e4m3 payload, then the fp32 scales of the row's 128-channel groups, as one
// wire row of H + 4 * H / 128 bytes); the sender quantises a row once into shared memory and sends from
// there; what arrives goes to the payload and the scale array of the receive region.  The checksum
// markers of Data-for-Checksum are taken from the payload bytes.
// kTable: the layout is derived here from the whole routing table in shared memory (small tables).
// Otherwise it comes from count_kernel / scan_kernel, launched before over the same chunks: the CTA stages
// only its own tokens and reads the rows of earlier chunks, the expert offsets and the region sizes.
template <int kProto, bool kFp8, bool kTable>
__global__ void __launch_bounds__(kThreads, 1) sync_dispatch_kernel(const Params p, const SmemPlan pl,
                                                                   const SyncParams sp) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ unsigned seq_sm;
    __shared__ int abort_flag;
    __shared__ unsigned long long wsum[2][kWarps];   // DC: per-warp marker sums (two tokens in flight)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = blockIdx.x;
    const int k = p.k, R = p.R;
    unsigned long long* times = sp.times + (size_t)c * kSyncTimeSlots;
    if (tid == 0) times[0] = global_ns();

    int* ids_sm = reinterpret_cast<int*>(smem + pl.off_ids);
    int* pos = reinterpret_cast<int*>(smem + pl.off_pos);
    int* key = reinterpret_cast<int*>(smem + pl.off_key);
    float* w_sm = reinterpret_cast<float*>(smem + pl.off_w);
    int* hist = reinterpret_cast<int*>(smem + pl.off_hist);
    int* nrows = reinterpret_cast<int*>(smem + pl.off_arr);     // rows every region receives
    int* order_sm = reinterpret_cast<int*>(smem + pl.off_order);
    unsigned long long* chk_sm = reinterpret_cast<unsigned long long*>(smem + pl.total);   // DC: [R]
    uint8_t* qrow = smem + pl.total + (((size_t)p.R * 8 + 15) & ~(size_t)15);              // FP8: the quantised row
    const BinMaps bmaps{reinterpret_cast<unsigned*>(smem + pl.off_mask), reinterpret_cast<unsigned*>(smem + pl.off_bm),
                        pl.map_wb, pl.map_bp, pl.map_groups};
    const int t0 = (int)chunk_begin(c, p.T, p.nchunks), t1 = (int)chunk_begin(c + 1, p.T, p.nchunks);
    const int ntok = t1 - t0;

    if (tid == 0) {
        seq_sm = read_seq_and_check_in(sp, p.grid);
        abort_flag = 0;
        // Sentinel Polling after a call that gave up: blocks of that call may still sit in the wire and
        // would be taken for this call's.  Nothing is sent or received then; the call reports the
        // condition again, and the library re-fills the wire once it has learnt of it (ubep_status).
        if (kProto == kSP && ld_relaxed(sp.sp_dirty) != 0u) {
            abort_flag = 1;
            report(p.status, kErrTimeout);
        }
    }
    if (kProto == kDC)
        for (int r = tid; r < R; r += kThreads) chk_sm[r] = 0ull;

    // ---- layout: bitmaps of every bin over the whole routing table -> totals, the rows
    // before this CTA's tokens, expert offsets, rows of this CTA's slots
    int* tot = hist;
    int* pre = hist + p.B;
    int* eo = hist + 2 * p.B;
    if (kTable) stage_ids(p, 0, p.T, ids_sm, tid, kThreads);
    else stage_ids(p, t0, t1, ids_sm, tid, kThreads);
    for (int r = tid; r < R; r += kThreads) order_sm[r] = __ldg(p.order_pos + r);
    for (int i = tid; i < ntok * k; i += kThreads) w_sm[i] = __ldg(p.topk_w + (size_t)t0 * k + i);
    __syncthreads();
    const unsigned seq = seq_sm;
    const int par = (int)(seq & 1u);
    if (kTable) {
        local_counts_all_bins(p, ids_sm, bmaps, t0, tot, pre, eo, tid, kThreads, warp, kWarps, lane, 0);
        for (int r = tid; r < R; r += kThreads) nrows[r] = rows_of_rank(p, tot, r);
        __syncthreads();
        finalize_chunk(p, t0, t1, ids_sm + (size_t)t0 * k, w_sm,
                       [&](int e, int tl) { return eo[e] + pre[e] + bits_in_range(bmaps, e, t0, t0 + tl); },
                       [&](int r, int tl) { return pre[p.E + r] + bits_in_range(bmaps, p.E + r, t0, t0 + tl); },
                       true, c, order_sm, pos, key, nullptr, tid, kThreads);
    } else {
        build_bin_maps(p, ids_sm, ntok, bmaps, warp, kWarps, lane);
        int* base_sm = hist;   // per bin: rows of all earlier chunks (+ the expert's offset in its region)
        for (int b = tid; b < p.B; b += kThreads)
            base_sm[b] = __ldcg(p.chunk_base + (size_t)b * p.nchunks + c) + (b < p.E ? __ldcg(p.expert_offset + b) : 0);
        for (int r = tid; r < R; r += kThreads) nrows[r] = __ldcg(p.num_rows_per_rank + r);
        __syncthreads();
        finalize_chunk(p, t0, t1, ids_sm, w_sm,
                       [&](int e, int tl) { return base_sm[e] + bits_in_range(bmaps, e, 0, tl); },
                       [&](int r, int tl) { return base_sm[p.E + r] + bits_in_range(bmaps, p.E + r, 0, tl); },
                       true, c, order_sm, pos, key, nullptr, tid, kThreads);
    }
    __syncthreads();
    if (tid == 0) times[1] = global_ns();
    if (kTable) {
        // counts and offsets nobody inside this kernel waits for (the launches before wrote them otherwise)
        if (c == 0) write_totals(p, tot, eo, tid, kThreads);
        for (int s = c; s < p.S; s += p.grid) write_source_from_maps(p, s, bmaps, eo, tid, kThreads);
    }

    // ---- sender: the rows of tokens [t0, t1), one token at a time, all threads on a row
    const int wbytes = kFp8 ? p.H + 4 * p.G : p.rowB;   // bytes of one row on the wire
    const int nvec = (wbytes + 15) / 16;                // its 16-byte blocks (FP8: the last may be cut short)
    const int pvec = p.rowB / 16;                       // blocks of the payload (all of them for bf16 rows)
    const int nwords = wbytes / 4;
    const int pwords = p.rowB / 4;
    const size_t wire_row = (size_t)sp.tff_blocks * 16;
    const size_t sp_row = (size_t)nvec * 16;
    const bool wire_unusable = kProto == kSP && abort_flag != 0;   // (set before the barriers above, uniform in the CTA)
    // word w of the wire row of global row `where` lands in the payload or, beyond it, in the scales
    auto put_word = [&](size_t where, int w, uint32_t val) {
        if (!kFp8 || w < pwords) reinterpret_cast<uint32_t*>(p.recv_x + where * p.rowB)[w] = val;
        else reinterpret_cast<uint32_t*>(p.recv_scale + where * p.G)[w - pwords] = val;
    };
    for (int tl = 0; tl < ntok && !wire_unusable; ++tl) {
        const int* ps = pos + tl * k;
        const uint4* xrow = reinterpret_cast<const uint4*>(p.x + (size_t)(t0 + tl) * p.H);
        if (kFp8) {
            // quantise the row once (every copy carries the same bytes)
            const int xvec = p.H / 8;
            for (int v0 = 0; v0 < xvec; v0 += kThreads) {   // same trip count for every thread (the quantiser shuffles)
                const int v = v0 + tid;
                const bool in = v < xvec;
                const uint4 d = in ? __ldg(xrow + v) : make_uint4(0, 0, 0, 0);
                uint2 q;
                float scale;
                quantize8(d, in, q, scale);
                if (in) {
                    *reinterpret_cast<uint2*>(qrow + (size_t)v * 8) = q;
                    if ((v & 15) == 0) reinterpret_cast<float*>(qrow + p.H)[v >> 4] = scale;
                }
            }
            for (int w = nwords + tid; w < nvec * 4; w += kThreads) reinterpret_cast<uint32_t*>(qrow)[w] = 0u;   // padding
            __syncthreads();
        }
        if (kProto == kTFF) {
            const uint32_t* xw = kFp8 ? reinterpret_cast<const uint32_t*>(qrow) : reinterpret_cast<const uint32_t*>(xrow);
            for (int g = tid; g < sp.tff_blocks; g += kThreads) {
                const int w0 = 3 * g;
                uint4 blk;
                blk.x = seq;   // the flag leads the block
                blk.y = w0 < nwords ? (kFp8 ? xw[w0] : __ldg(xw + w0)) : 0u;
                blk.z = w0 + 1 < nwords ? (kFp8 ? xw[w0 + 1] : __ldg(xw + w0 + 1)) : 0u;
                blk.w = w0 + 2 < nwords ? (kFp8 ? xw[w0 + 2] : __ldg(xw + w0 + 2)) : 0u;
                for (int j = 0; j < k; ++j) {
                    const int where = ps[j];
                    if (where >= 0) st_relaxed_v4(sp.tff_wire + (size_t)where * wire_row + (size_t)g * 16, blk);
                }
            }
        } else {
            unsigned long long mine = 0ull;
            for (int v = tid; v < nvec; v += kThreads) {
                const uint4 d = kFp8 ? reinterpret_cast<const uint4*>(qrow)[v] : __ldg(xrow + v);
                if (kProto == kDC && v < pvec && (v % kDcBlockVecs) < kDcMarkerVecs) mine += marker_words(d);
                for (int j = 0; j < k; ++j) {
                    const int where = ps[j];
                    if (where < 0) continue;
                    if (kProto == kSP) {
                        st_relaxed_v4(sp.sp_wire + (size_t)where * sp_row + (size_t)v * 16, d);
                    } else if (!kFp8 || v < pvec) {
                        *reinterpret_cast<uint4*>(p.recv_x + (size_t)where * p.rowB + (size_t)v * 16) = d;
                    } else {
                        const uint32_t dw[4] = {d.x, d.y, d.z, d.w};
                        for (int i = 0; i < 4; ++i)
                            if (4 * v + i < nwords) put_word((size_t)where, 4 * v + i, dw[i]);
                    }
                }
            }
            if (kProto == kDC) {
                // marker sum of this row, added to the running sum of every region it goes to
                // (the slot of the token after next is written only after the next barrier)
                mine = warp_sum64(mine);
                if (lane == 0) wsum[tl & 1][warp] = mine;
                __syncthreads();
                if (tid < k && ps[tid] >= 0) {
                    unsigned long long row_sum = 0ull;
                    for (int q = 0; q < kWarps; ++q) row_sum += wsum[tl & 1][q];
                    atomicAdd(&chk_sm[ps[tid] / p.cap], row_sum);
                }
            }
            if (kProto == kSW) {
                // stop-and-wait: the row's stores are fenced before its flag is raised
                __threadfence();
                __syncthreads();
                if (tid < k && ps[tid] >= 0) red_release_add(sp.sw_rows + par * R + ps[tid] / p.cap, 1u);
            }
        }
        if (kFp8) __syncthreads();   // the quantised row is reused for the next token
    }
    if (kProto == kDC) {
        // one fence per sender and batch, then the checksum packet of every region
        __threadfence();
        __syncthreads();
        for (int r = tid; r < R; r += kThreads) {
            if (chk_sm[r]) atomicAdd(sp.checksum + par * R + r, chk_sm[r]);
            red_release_add(sp.announced + par * R + r, 1u);
        }
    }
    if (tid == 0) times[2] = global_ns();

    // ---- receiver: region u / Q, slice u % Q of its rows
    Waiter wt{&abort_flag, global_ns() + kWaitLimitNs, p.status, kProto == kSP ? sp.sp_dirty : nullptr};
    const int Q = p.grid / R > 1 ? p.grid / R : 1;
    bool duty = false;
    for (int u = c; u < R * Q; u += p.grid) {
        const int r = u / Q, q = u % Q;
        const int n_r = nrows[r] < p.cap ? nrows[r] : p.cap;
        if (kProto == kTFF || kProto == kSP) {
            const int lo = (int)((long long)n_r * q / Q), hi = (int)((long long)n_r * (q + 1) / Q);
            duty = duty || hi > lo;
            // The slice's DataBlocks as one index space; every thread keeps kBatch loads in
            // flight and only then looks at what they brought (a block that has not arrived
            // is polled on its own).
            constexpr int kBatch = 4;
            const int per_row = kProto == kTFF ? sp.tff_blocks : nvec;
            const size_t row_stride = kProto == kTFF ? wire_row : sp_row;
            uint8_t* const wire = (kProto == kTFF ? sp.tff_wire : sp.sp_wire) + ((size_t)r * p.cap + lo) * row_stride;
            const size_t row0 = (size_t)r * p.cap + lo;   // global row of the slice's first row
            const int items = (hi - lo) * per_row;
            const uint4 sentinel = make_uint4(0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu);
            bool ok = true;
            for (int i0 = tid; ok && i0 < items && !*wt.abort; i0 += kBatch * kThreads) {
                uint4 blk[kBatch];
                int row[kBatch], g[kBatch];
#pragma unroll
                for (int b = 0; b < kBatch; ++b) {
                    const int i = i0 + b * kThreads;
                    row[b] = i / per_row;
                    g[b] = i - row[b] * per_row;
                    if (i < items) blk[b] = ld_relaxed_v4(wire + row[b] * row_stride + (size_t)g[b] * 16);
                }
#pragma unroll
                for (int b = 0; b < kBatch; ++b) {
                    if (i0 + b * kThreads >= items) break;
                    uint8_t* const src = wire + row[b] * row_stride + (size_t)g[b] * 16;
                    unsigned spins = 0;
                    while (kProto == kTFF ? blk[b].x != seq : is_sentinel(blk[b])) {
                        if (!wt.keep_waiting(spins)) { ok = false; break; }
                        blk[b] = ld_relaxed_v4(src);
                    }
                    if (!ok) break;
                    const size_t grow = row0 + row[b];
                    if (kProto == kTFF) {
                        const int w0 = 3 * g[b];
                        if (w0 < nwords) put_word(grow, w0, blk[b].y);
                        if (w0 + 1 < nwords) put_word(grow, w0 + 1, blk[b].z);
                        if (w0 + 2 < nwords) put_word(grow, w0 + 2, blk[b].w);
                    } else {
                        if (!kFp8 || g[b] < pvec) {
                            *reinterpret_cast<uint4*>(p.recv_x + grow * p.rowB + (size_t)g[b] * 16) = blk[b];
                        } else {
                            const uint32_t dw[4] = {blk[b].x, blk[b].y, blk[b].z, blk[b].w};
                            for (int i = 0; i < 4; ++i)
                                if (4 * g[b] + i < nwords) put_word(grow, 4 * g[b] + i, dw[i]);
                        }
                        st_relaxed_v4(src, sentinel);   // consumed: ready for the next call
                    }
                }
            }
        } else if (q == 0) {
            duty = true;
            if (kProto == kSW) {
                if (tid == 0) (void)wait_count(sp.sw_rows + par * R + r, (unsigned)n_r, wt);
            } else {
                if (tid == 0) (void)wait_count(sp.announced + par * R + r, (unsigned)p.grid, wt);
                __syncthreads();
                if (!abort_flag) {
                    const int nblk = (pvec + kDcBlockVecs - 1) / kDcBlockVecs;
                    const int per_row = nblk * kDcMarkerVecs;
                    unsigned long long mine = 0ull;
                    for (int i = tid; i < n_r * per_row; i += kThreads) {
                        const int row = i / per_row, rem = i - row * per_row;
                        const int v = (rem / kDcMarkerVecs) * kDcBlockVecs + rem % kDcMarkerVecs;
                        if (v < pvec)
                            mine += marker_words(__ldcg(
                                reinterpret_cast<const uint4*>(p.recv_x + ((size_t)r * p.cap + row) * p.rowB) + v));
                    }
                    mine = warp_sum64(mine);
                    if (lane == 0) wsum[0][warp] = mine;
                    __syncthreads();
                    if (tid == 0) {
                        unsigned long long found = 0ull;
                        for (int q = 0; q < kWarps; ++q) found += wsum[0][q];
                        if (found != ld_relaxed_u64(sp.checksum + par * R + r)) report(p.status, kErrChecksum);
                    }
                }
                __syncthreads();
            }
        }
    }
    __syncthreads();
    if (tid == 0) times[3] = (duty && !abort_flag) ? global_ns() : times[2];
    // the counters of the next call live in the other half: clear them now
    if (c == 0)
        for (int r = tid; r < R; r += kThreads) {
            sp.checksum[(par ^ 1) * R + r] = 0ull;
            sp.announced[(par ^ 1) * R + r] = 0u;
            sp.sw_rows[(par ^ 1) * R + r] = 0u;
        }
    if (tid == 0) times[4] = global_ns();
}

__global__ void __launch_bounds__(256) sentinel_scan_kernel(const uint4* __restrict__ x, long long n_vec,
                                                            unsigned long long* count) {
    unsigned long long mine = 0ull;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec;
         i += (long long)gridDim.x * blockDim.x)
        mine += is_sentinel(__ldg(x + i)) ? 1ull : 0ull;
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(count, mine);
}

template <int kProto>
cudaError_t launch_one(const Params& p, const SmemPlan& pl, const SyncParams& sp, bool whole_table, cudaStream_t st) {
    auto kern = whole_table ? (p.payload ? sync_dispatch_kernel<kProto, true, true> : sync_dispatch_kernel<kProto, false, true>)
                            : (p.payload ? sync_dispatch_kernel<kProto, true, false> : sync_dispatch_kernel<kProto, false, false>);
    const int smem = pl.total + sync_extra_smem(p);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    // Receivers wait for senders that are other CTAs of this grid: a cooperative launch, which the
    // runtime refuses when the grid cannot be resident at once and starts only when it is.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3((unsigned)kThreads);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p, pl, sp);
}

}  // namespace

int sync_extra_smem(const Params& p) {
    const int qrow = p.payload ? ((p.H + 4 * p.G + 15) / 16) * 16 : 0;   // FP8: the quantised row of the token being sent
    return p.R * 8 + 128 + qrow + 16;
}

cudaError_t launch_sync_dispatch(const Params& p, const SmemPlan& pl, const SyncParams& sp, bool whole_table,
                                 cudaStream_t st) {
    switch (sp.protocol) {
        case kSW: return launch_one<kSW>(p, pl, sp, whole_table, st);
        case kTFF: return launch_one<kTFF>(p, pl, sp, whole_table, st);
        case kDC: return launch_one<kDC>(p, pl, sp, whole_table, st);
        case kSP: return launch_one<kSP>(p, pl, sp, whole_table, st);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_sentinel_scan(const void* x, long long n_vec, unsigned long long* count, int num_sms,
                                 cudaStream_t st) {
    long long blocks = (n_vec + 255) / 256;
    if (blocks > (long long)num_sms * 8) blocks = (long long)num_sms * 8;
    if (blocks < 1) blocks = 1;
    sentinel_scan_kernel<<<(int)blocks, 256, 0, st>>>(static_cast<const uint4*>(x), n_vec, count);
    return cudaGetLastError();
}

}  // namespace ubep
