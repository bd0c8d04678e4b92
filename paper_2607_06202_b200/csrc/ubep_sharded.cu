// Dispatch and combine with the ranks on different GPUs (Sec. 2.3 and Sec. 4 of the paper,
// "Global Load/Store for Point-to-Point Synchronization"): rank r = GPU r, every GPU holds an
// arena of the same layout that its peers address over NVLink, rows and their metadata are
// stored straight into the receiving rank's arena, expert outputs are loaded straight from the
// producing rank's buffer.  Plain loads and stores only: no TMA, no multicast, no collective.
// FP8 rows are quantised by the sender, payload and scales go to the receiver's arrays.  No kernel here waits for another rank except wait_arrivals_kernel.
//
// Every rank derives the whole layout from the all-gathered routing table, alone, so all ranks
// agree on every row without exchanging a count: for a small table inside the sender kernel, with
// the same device functions and in the same order as the flag-free instance of the main dispatch
// kernel; for a large one with the count and prefix-sum launches of the three-launch pipeline,
// over chunks that do not straddle ranks.
#include "ubep_layout.cuh"
#include "ubep_quant.cuh"
#include "ubep_sharded.h"

namespace ubep {

namespace {

__device__ __forceinline__ void red_release_sys_add(unsigned* ptr, unsigned v) {
    asm volatile("red.release.sys.global.add.u32 [%0], %1;" ::"l"(ptr), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_sys(const unsigned* ptr) {
    unsigned v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

// kTable: the layout is derived here from the whole routing table in shared memory (small tables).
// Otherwise it comes from count_kernel / scan_kernel, run before over the whole table with chunks that
// do not straddle ranks: CTA c then owns chunk my_rank * grid + c of them and only stages its own tokens.
template <bool kTable>
__global__ void __launch_bounds__(kThreads, 1) sharded_dispatch_kernel(const Params p, const SmemPlan pl) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = blockIdx.x;
    const int k = p.k, R = p.R;
    int* ids_sm = reinterpret_cast<int*>(smem + pl.off_ids);
    int* pos = reinterpret_cast<int*>(smem + pl.off_pos);
    int* key = reinterpret_cast<int*>(smem + pl.off_key);
    float* w_sm = reinterpret_cast<float*>(smem + pl.off_w);
    int* hist = reinterpret_cast<int*>(smem + pl.off_hist);
    int* nrows = reinterpret_cast<int*>(smem + pl.off_arr);      // rows every region receives
    int* order_sm = reinterpret_cast<int*>(smem + pl.off_order);
    long long* delta = reinterpret_cast<long long*>(smem + pl.total);   // [R] byte distance to rank r's arena
    int* sent = reinterpret_cast<int*>(delta + R);                       // [R] rows this CTA stores to rank r
    const BinMaps bmaps{reinterpret_cast<unsigned*>(smem + pl.off_mask), reinterpret_cast<unsigned*>(smem + pl.off_bm),
                        pl.map_wb, pl.map_bp, pl.map_groups};
    // this CTA's share of the rank's own tokens [tok0, tok1)
    const int nloc = p.tok1 - p.tok0;
    const int gch = p.my_rank * p.grid + c;   // (large tables) its chunk among the nchunks = R * grid chunks of all tokens
    const int t0 = kTable ? p.tok0 + (int)chunk_begin(c, nloc, p.nchunks) : (int)chunk_begin(gch, p.T, p.nchunks);
    const int t1 = kTable ? p.tok0 + (int)chunk_begin(c + 1, nloc, p.nchunks) : (int)chunk_begin(gch + 1, p.T, p.nchunks);
    const int ntok = t1 - t0;

    for (int r = tid; r < R; r += kThreads) {
        delta[r] = p.peer_delta[r];
        sent[r] = 0;
        order_sm[r] = __ldg(p.order_pos + r);
    }
    if (kTable) {
        // ---- layout over the table of all T tokens (identical on every rank)
        int* tot = hist;
        int* pre = hist + p.B;
        int* eo = hist + 2 * p.B;
        stage_ids(p, 0, p.T, ids_sm, tid, kThreads);
        for (int i = tid; i < ntok * k; i += kThreads) w_sm[i] = __ldg(p.topk_w + (size_t)t0 * k + i);
        __syncthreads();
        local_counts_all_bins(p, ids_sm, bmaps, t0, tot, pre, eo, tid, kThreads, warp, kWarps, lane, 0);
        for (int r = tid; r < R; r += kThreads) nrows[r] = rows_of_rank(p, tot, r);
        __syncthreads();
        // rows of this CTA's slots; the metadata of every row goes to the arena of the rank that receives it
        finalize_chunk<true>(p, t0, t1, ids_sm + (size_t)t0 * k, w_sm,
                             [&](int e, int tl) { return eo[e] + pre[e] + bits_in_range(bmaps, e, t0, t0 + tl); },
                             [&](int r, int tl) { return pre[p.E + r] + bits_in_range(bmaps, p.E + r, t0, t0 + tl); },
                             true, c, order_sm, pos, key, sent, tid, kThreads, delta);
        __syncthreads();
        // counts and offsets: every rank keeps the whole set in its own arena
        if (c == 0) {
            write_totals(p, tot, eo, tid, kThreads);
            // what the local receiver has to wait for (read by wait_arrivals_kernel, later in this stream)
            if (tid == 0) atomicAdd(p.shard_arrival + 1, (unsigned)(nrows[p.my_rank] < p.cap ? nrows[p.my_rank] : p.cap));
        }
        for (int s = c; s < p.S; s += p.grid) write_source_from_maps(p, s, bmaps, eo, tid, kThreads);
    } else {
        // ---- layout from the launches before: bitmaps of this CTA's own tokens, and per bin the rows of
        // all earlier chunks (+ the expert's offset in its region) that the prefix-sum launch left
        stage_ids(p, t0, t1, ids_sm, tid, kThreads);
        for (int i = tid; i < ntok * k; i += kThreads) w_sm[i] = __ldg(p.topk_w + (size_t)t0 * k + i);
        __syncthreads();
        build_bin_maps(p, ids_sm, ntok, bmaps, warp, kWarps, lane);
        int* base_sm = hist;
        for (int b = tid; b < p.B; b += kThreads)
            base_sm[b] = __ldcg(p.chunk_base + (size_t)b * p.nchunks + gch) + (b < p.E ? __ldcg(p.expert_offset + b) : 0);
        __syncthreads();
        finalize_chunk<true>(p, t0, t1, ids_sm, w_sm,
                             [&](int e, int tl) { return base_sm[e] + bits_in_range(bmaps, e, 0, tl); },
                             [&](int r, int tl) { return base_sm[p.E + r] + bits_in_range(bmaps, p.E + r, 0, tl); },
                             true, c, order_sm, pos, key, sent, tid, kThreads, delta);
        __syncthreads();
        if (c == 0 && tid == 0) {
            const int n_mine = __ldcg(p.num_rows_per_rank + p.my_rank);
            atomicAdd(p.shard_arrival + 1, (unsigned)(n_mine < p.cap ? n_mine : p.cap));
        }
    }

    // ---- sender: one token at a time, all threads on its row, one store per copy and vector
    const int nvec = p.H / 8;   // 16-byte vectors of the bf16 input row
    for (int tl = 0; tl < ntok; ++tl) {
        const int* ps = pos + tl * k;
        const uint4* src = reinterpret_cast<const uint4*>(p.x + (size_t)(t0 + tl - p.tok0) * p.H);
        for (int v0 = 0; v0 < nvec; v0 += kThreads) {   // same trip count for every thread (the quantiser shuffles)
            const int v = v0 + tid;
            const bool in = v < nvec;
            const uint4 d = in ? __ldg(src + v) : make_uint4(0, 0, 0, 0);
            uint2 q = make_uint2(0, 0);
            float scale = 0.0f;
            if (p.payload) quantize8(d, in, q, scale);
            if (!in) continue;
            for (int j = 0; j < k; ++j) {
                const int where = ps[j];
                if (where < 0) continue;
                const long long pd = delta[where / p.cap];
                uint8_t* row = p.recv_x + pd + (size_t)where * p.rowB;
                if (p.payload) {
                    *reinterpret_cast<uint2*>(row + (size_t)v * 8) = q;
                    if ((v & 15) == 0) toward_peer<true>(p.recv_scale, pd)[(size_t)where * p.G + (v >> 4)] = scale;
                } else {
                    *reinterpret_cast<uint4*>(row + (size_t)v * 16) = d;
                }
            }
        }
    }
    // ---- announce: everything above is fenced at system scope once, then one release-add per rank
    __threadfence_system();
    __syncthreads();
    for (int r = tid; r < R; r += kThreads)
        if (sent[r]) red_release_sys_add(toward_peer<true>(p.shard_arrival, delta[r]), (unsigned)sent[r]);
}

__global__ void wait_arrivals_kernel(const unsigned* arrival, int32_t* status) {
    if (threadIdx.x != 0) return;
    const unsigned want = arrival[1];
    const unsigned long long t_end = global_ns() + kWaitLimitNs;
    for (unsigned i = 1;; ++i) {
        if ((int)(ld_acquire_sys(arrival) - want) >= 0) return;   // counters only grow (modulo 2^32)
        if ((i & 63u) == 0 && global_ns() > t_end) {
            report(status, kErrTimeout);
            return;
        }
        __nanosleep(64);
    }
}

// One thread per 16-byte vector of the output rows of tokens [tok0, tok1): k gathers from the
// buffers of the ranks that hold the rows, fp32 fused multiply-adds in slot order, one
// round-to-nearest-even pack to bf16 (the arithmetic of combine_kernel).
__global__ void __launch_bounds__(256) sharded_combine_kernel(const uint16_t* const* __restrict__ y_peers,
                                                             const int32_t* __restrict__ slot_pos,
                                                             const float* __restrict__ topk_w, int tok0, int tok1,
                                                             int H, int k, int cap, uint16_t* __restrict__ out) {
    const int nvec = H / 8;
    const int64_t total = (int64_t)(tok1 - tok0) * nvec;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total;
         u += (int64_t)gridDim.x * blockDim.x) {
        const int tl = (int)(u / nvec), v = (int)(u - (int64_t)tl * nvec);
        const int t = tok0 + tl;
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
        for (int j = 0; j < k; ++j) {
            const int where = __ldg(slot_pos + (size_t)t * k + j);
            if (where < 0) continue;
            const float w = __ldg(topk_w + (size_t)t * k + j);
            const uint16_t* y = y_peers[where / cap];
            const uint4 q = *(reinterpret_cast<const uint4*>(y + (size_t)where * H) + v);
            const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                acc[2 * i] = __fmaf_rn(w, __uint_as_float(ww[i] << 16), acc[2 * i]);
                acc[2 * i + 1] = __fmaf_rn(w, __uint_as_float(ww[i] & 0xffff0000u), acc[2 * i + 1]);
            }
        }
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
            o[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        reinterpret_cast<uint4*>(out + (size_t)tl * H)[v] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

}  // namespace

int sharded_extra_smem(const Params& p) { return p.R * 12 + 128; }

cudaError_t launch_sharded_dispatch(const Params& p, const SmemPlan& pl, bool whole_table, cudaStream_t st) {
    const int smem = pl.total + sharded_extra_smem(p);
    auto kern = whole_table ? sharded_dispatch_kernel<true> : sharded_dispatch_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kern<<<p.grid, kThreads, smem, st>>>(p, pl);
    return cudaGetLastError();
}

cudaError_t launch_wait_arrivals(const unsigned* arrival, int32_t* status, cudaStream_t st) {
    wait_arrivals_kernel<<<1, 32, 0, st>>>(arrival, status);
    return cudaGetLastError();
}

cudaError_t launch_sharded_combine(const uint16_t* const* y_peers, const int32_t* slot_pos, const float* topk_w,
                                   int tok0, int tok1, int H, int k, int cap, uint16_t* out_local, int num_sms,
                                   cudaStream_t st) {
    const int64_t total = (int64_t)(tok1 - tok0) * (H / 8);
    int64_t blocks = (total + 255) / 256;
    if (blocks > (int64_t)num_sms * 8) blocks = (int64_t)num_sms * 8;
    if (blocks < 1) blocks = 1;
    sharded_combine_kernel<<<(int)blocks, 256, 0, st>>>(y_peers, slot_pos, topk_w, tok0, tok1, H, k, cap, out_local);
    return cudaGetLastError();
}

}  // namespace ubep
