// Kernels of the dispatch / combine hot path for sm_100a.
//
//   count_kernel / scan_kernel        TokenCnt and CalCumSum as separate launches (the
//                                     bulk-synchronous pipeline; kernel boundaries = barriers)
//   dispatch_kernel<mode, fp8>        persistent CTA per work slice: layout warps plus a mover
//                                     warp that streams rows with TMA bulk copies.  FUSED: the
//                                     layout steps of different CTAs are ordered by
//                                     release/acquire flags instead of launches (kernel
//                                     decomposition).  LOCAL: every CTA derives its offsets
//                                     from the whole routing table (small T*k, no flags).
//   combine_kernel<K>                 gather + fp32 weighted sum + one bf16 rounding
//   layout_kernel                     counts only (ubep_get_dispatch_layout)
#include <atomic>

#include "ubep_kernels.h"
#include "ubep_layout.cuh"
#include "ubep_quant.cuh"

namespace ubep {

// --------------------------------------------------------------- phased: count / scan

// TokenCnt of one token chunk per CTA: bin bitmaps -> chunk histogram and boundary snapshots.
__global__ void __launch_bounds__(256) count_kernel(const Params p, const SmemPlan pl) {
    extern __shared__ __align__(16) uint8_t sm_c[];
    const int c = blockIdx.x, tid = threadIdx.x;
    const int t0 = (int)chunk_begin(c, p.T, p.nchunks), t1 = (int)chunk_begin(c + 1, p.T, p.nchunks);
    int* ids = reinterpret_cast<int*>(sm_c);
    BinMaps bmaps{reinterpret_cast<unsigned*>(sm_c + (pl.off_mask - pl.off_ids)),
                  reinterpret_cast<unsigned*>(sm_c + (pl.off_bm - pl.off_ids)), pl.map_wb, pl.map_bp,
                  pl.map_groups};
    stage_ids(p, t0, t1, ids, tid, 256);
    __syncthreads();
    build_bin_maps(p, ids, t1 - t0, bmaps, tid / 32, 8, tid % 32);
    __syncthreads();
    publish_chunk_counts(p, c, t0, t1, bmaps, tid, 256);
}

__global__ void __launch_bounds__(256) scan_kernel(const Params p) {
    extern __shared__ int sm_i[];
    scan_rank_publish(p, blockIdx.x, sm_i, threadIdx.x / 32, 8, threadIdx.x % 32, 1);
    scan_rank_sources(p, blockIdx.x, sm_i, threadIdx.x, 256);
}

// Everything the roles of one dispatch CTA share.
struct Cta {
    const Params& p;
    const SmemPlan& pl;
    uint8_t* smem;
    uint64_t *full_bar, *empty_bar, *out_full, *out_empty, *ready_bar, *epoch_bar, *staged_bar;
    int* abort_flag;
    int tid, lane, warp, c, part, ch, t0, t1, ntok, stages, nq;
    int gn, nw;        // layout (count) group: warps 1 .. nw, gn = 32 * nw threads
    int out_stages;    // FP8: depth of the ring of quantised rows
    int qwarp0;        // FP8: first quantising warp (warps qwarp0 .. qwarp0 + nq - 1 quantise)
    bool beside;       // FP8: the quantising warps are not layout warps and run beside the layout
    int *ids_sm, *pos, *pos_raw, *key;
    float* w_sm;
    BinMaps bmaps;
    int *hist, *arr, *order_sm;
    unsigned epoch, in_bytes, out_bytes;   // (epoch: 0 until the role that needs it has learnt it from *epoch_late)
    unsigned* epoch_late;
    size_t in_off, out_off;
    bool fast_local;
    bool early0;  // flag-free kernel: the copies of the CTA's first row are issued by the warp that assigns the rows
    int issued;   // rows whose load the mover has started (thread 0's copy is used when leaving early)
};

// The role functions below keep the names the kernel uses for these.
#define UBEP_CTA_LOCALS(x, all15)                                                                              \
    [[maybe_unused]] const Params& p = (x).p;                                                                \
    [[maybe_unused]] const SmemPlan& pl = (x).pl;                                                            \
    [[maybe_unused]] uint8_t* const smem = (x).smem;                                                         \
    [[maybe_unused]] uint64_t* const full_bar = (x).full_bar;                                                \
    [[maybe_unused]] uint64_t* const empty_bar = (x).empty_bar;                                              \
    [[maybe_unused]] uint64_t* const out_full = (x).out_full;                                                \
    [[maybe_unused]] uint64_t* const out_empty = (x).out_empty;                                              \
    [[maybe_unused]] uint64_t& ready_bar = *(x).ready_bar;                                                   \
    [[maybe_unused]] int& abort_flag = *(x).abort_flag;                                                      \
    [[maybe_unused]] volatile int* const abortp = (x).abort_flag;                                            \
    [[maybe_unused]] const int tid = (x).tid, lane = (x).lane, warp = (x).warp, c = (x).c;                   \
    [[maybe_unused]] const int part = (x).part, ch = (x).ch, t0 = (x).t0, t1 = (x).t1, ntok = (x).ntok;     \
    [[maybe_unused]] const int stages = (x).stages, nq = (x).nq;                                             \
    [[maybe_unused]] int* const ids_sm = (x).ids_sm;                                                         \
    [[maybe_unused]] int* const pos = (x).pos;                                                               \
    [[maybe_unused]] int* const pos_raw = (x).pos_raw;                                                       \
    [[maybe_unused]] int* const key = (x).key;                                                               \
    [[maybe_unused]] float* const w_sm = (x).w_sm;                                                           \
    [[maybe_unused]] const BinMaps& bmaps = (x).bmaps;                                                       \
    [[maybe_unused]] int* const hist = (x).hist;                                                             \
    [[maybe_unused]] int* const arr = (x).arr;                                                               \
    [[maybe_unused]] int* const order_sm = (x).order_sm;                                                     \
    [[maybe_unused]] const unsigned epoch = (x).epoch, in_bytes = (x).in_bytes, out_bytes = (x).out_bytes;   \
    [[maybe_unused]] const size_t in_off = (x).in_off, out_off = (x).out_off;                                \
    [[maybe_unused]] const bool fast_local = (x).fast_local;                                                 \
    [[maybe_unused]] int& issued = (x).issued;                                                               \
    /* layout group: warps 1 .. nw; a compile-time constant where it is always all 15 */                    \
    [[maybe_unused]] const int nw = (all15) ? kWarps - 1 : (x).nw;                                           \
    [[maybe_unused]] const int gn = nw * 32;                                                                 \
    [[maybe_unused]] const int out_stages = (x).out_stages;                                                  \
    [[maybe_unused]] const int gtid = (x).tid - 32, gw = (x).warp - 1

// ------------------------------------------------------------------------ mover warp
// Warp 0.  Lane 0 issues the TMA loads; for bf16 rows lane j issues the TMA store of slot j,
// so the k copies of a row are issued side by side; for FP8 rows the warp only loads.
template <int kMode, bool kFp8, bool kSteal>
__device__ __forceinline__ void mover_warp(Cta& x) {
    if (kMode != kModeLocal) {
        // The epoch: one acquire load and one ticket, two round trips to L2.  This warp has nothing
        // urgent to do yet, so it fetches it while the layout group already stages the routing table.
        unsigned ep = 0;
        if (x.lane == 0) {
            ep = read_epoch_and_check_in(x.p);
            *x.epoch_late = ep;
            mbar_arrive(x.epoch_bar);
        }
        x.epoch = __shfl_sync(0xffffffffu, ep, 0);
    }
    UBEP_CTA_LOCALS(x, !kFp8);
    // Lane 0 issues the TMA loads; for bf16 rows lane j issues the TMA store of slot j,
    // so the k copies of a row are issued side by side.  Tokens come from a feeder: the
    // CTA's own chunk first and, when stealing is on, blocks of other chunks afterwards.
    bool ok = true;
    int v = ch, v_t0 = t0, v_ntok = ntok;   // chunk the feeder currently draws from
    int blk_lo = 0, blk_hi = 0;             // tokens of that chunk this CTA may take now
    unsigned pend = 0;                      // lane 0: answer of a claim made ahead of time
    bool pend_valid = false, feeder_done = false;
    int scanned = 0;                        // victims looked at so far
    if (!kSteal) blk_hi = ntok;            // no stealing: the whole chunk, no atomics
    auto pick_victim = [&]() -> int {
        while (scanned < p.nchunks - 1) {
            unsigned done = 0;
            if (lane == 0) done = __ldcg(p.claimed + (epoch & 1));
            if ((int)__shfl_sync(0xffffffffu, done, 0) >= p.T) return -1;   // every token is handed out
            const int idx = scanned + lane;
            int cand = ch + 1 + idx;
            if (cand >= p.nchunks) cand -= p.nchunks;
            int rem = 0;
            if (idx < p.nchunks - 1 && ld_acquire(p.pos_flag + cand) == epoch) {
                const int nt = (int)chunk_begin(cand + 1, p.T, p.nchunks) - (int)chunk_begin(cand, p.T, p.nchunks);
                rem = nt - (int)__ldcg(p.cursor + cand);
            }
            int best = rem > 0 ? (rem << 9) | cand : 0;   // most remaining tokens first (cand < 512)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
            if (best > 0) return best & 511;
            scanned += 32;
        }
        return -1;
    };
    // Next token of the feeder: its index inside chunk v (warp-uniform).  Returns 1 = token,
    // 0 = nothing left anywhere, 2 = only other chunks have work and the caller does not
    // want to take it yet (it still has rows of its own queued).
    bool v_empty = false;   // chunk v has handed out all its tokens
    auto next_token = [&](int& tl, bool allow_steal) -> int {
        while (blk_lo >= blk_hi) {
            if (feeder_done || !kSteal) { feeder_done = true; return 0; }
            if (v_empty) {
                if (!allow_steal) return 2;
                v = pick_victim();
                if (v < 0) { feeder_done = true; return 0; }
                v_t0 = (int)chunk_begin(v, p.T, p.nchunks);
                v_ntok = (int)chunk_begin(v + 1, p.T, p.nchunks) - v_t0;
                v_empty = false;
                pend_valid = false;
            }
            if (v != ch && !allow_steal) return 2;
            if (!pend_valid && lane == 0) pend = atomicAdd(p.cursor + v, (unsigned)kStealBlock);
            const int old = (int)__shfl_sync(0xffffffffu, pend, 0);
            pend_valid = false;
            if (old < v_ntok) {
                blk_lo = old;
                blk_hi = min(old + kStealBlock, v_ntok);
                if (lane == 0) {
                    atomicAdd(p.claimed + (epoch & 1), (unsigned)(blk_hi - blk_lo));
                    pend = atomicAdd(p.cursor + v, (unsigned)kStealBlock);   // answer needed a block later
                }
                pend_valid = true;
            } else {
                v_empty = true;
            }
        }
        tl = blk_lo++;
        return 1;
    };
    int* item_src = reinterpret_cast<int*>(smem + pl.off_item);           // [stages] (chunk << 16 | index), -1 = end
    int* item_pos = item_src + kMaxStages + kMaxOutStages;                // [stages, k] destinations of stolen tokens
    int head = 0, tail = 0;   // rows whose load was issued / whose copies were issued
    // load of the feeder's next token into ring stage head % stages
    auto issue_item = [&](int tl) {
        const int s = head % stages;
        // What travels with the row is written before the load is started: the consumers read it
        // as soon as the row has landed.
        if (kSteal && v != ch) {   // a stolen token: its destinations come from the owner's published list
            for (int j = lane; j < p.k; j += 32)
                item_pos[s * p.k + j] = __ldcg(p.copy_pos + (size_t)(v_t0 + tl) * p.k + j);
            __syncwarp();
        }
        if (lane == 0) {
            if (kSteal) item_src[s] = (v << 16) | tl;
            mbar_arrive_expect_tx(&full_bar[s], in_bytes);
            bulk_load(smem + (size_t)s * pl.stage_bytes,
                      reinterpret_cast<const uint8_t*>(p.x) + (size_t)(v_t0 + tl) * p.H * 2 + in_off, in_bytes,
                      &full_bar[s]);
        }
        if (kSteal) __syncwarp();
        ++head;
    };
    // The first rows of the CTA's own chunk, one load per lane, issued side by side: one lane issuing
    // them one after the other was measured at 0.15 - 0.2 us per load, on the way to the first copy.
    auto issue_first = [&](int n) {   // n <= 32 rows from row `head` on; without stealing
        if (lane < n) {
            const int tl = head + lane, s = tl % stages;
            mbar_arrive_expect_tx(&full_bar[s], in_bytes);
            bulk_load(smem + (size_t)s * pl.stage_bytes,
                      reinterpret_cast<const uint8_t*>(p.x) + (size_t)(t0 + tl) * p.H * 2 + in_off, in_bytes, &full_bar[s]);
        }
        head += n;
    };
    if (kSteal && lane == 0) p.cursor[ch] = 0;   // before anybody can claim from this chunk
    // Rows fetched before the layout is done.  With flags the layout takes many microseconds in which a
    // few small loads and stores of every CTA wait on one another; a ring-full of rows per CTA fetched
    // meanwhile fills the memory system's queues in front of them.  Three rows start the copies, the
    // rest follows once the movers are released.  (Not with stealing: there every block of rows costs a
    // claim, a round trip each, and those are best paid while the layout runs.)
    const int early = (kMode == kModeLocal || kSteal) ? kMaxStages : 3;
    if (!kFp8) {
        // loads run (stages - 3) rows ahead; up to 3 rows' stores stay in flight
        int tl = 0;
        // Flag-free kernel: the routing table first, the rows after it.  The table is the one load the
        // whole layout waits for; the rows of 148 CTAs queued in front of it cost about a microsecond.
        const RankMaps rm{bmaps.bm, bmaps.mask_t, (p.R + 31) / 32, ((p.R + 31) / 32) * 32, (p.T + 31) / 32};
        if (fast_local) {
            // Two rows are asked for at once, so that the first copies find their row in shared memory when
            // the movers are released; then this warp lends a hand with the routing table and asks for the
            // rest of the ring.  (More than two rows in front of the table delay it, 148 CTAs' worth of them
            // queue in front of the one load the layout waits for: measured per layer 25.6 us with one or two
            // rows first, 25.9 with four or with none, 26.5 with the whole ring.)
            if (!kSteal) {
                issue_first(max(min(2, min(stages - 3, ntok)), 0));
                issued = head;
            }
            local_stage_and_rank_maps(p, ids_sm, rm, rm.groups, 0, kWarps, lane);
            group_sync(2, kThreads);
        } else if (kMode == kModeLocal) {
            ok = mbar_wait(x.staged_bar, 0, abortp);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (kSteal) {
            while (head < min(stages - 3, early) && next_token(tl, false) == 1) issue_item(tl);
        } else {
            issue_first(max(min(min(min(stages - 3, early), ntok), 32) - head, 0));
            while (head < min(min(stages - 3, early), ntok)) issue_item(head);
        }
        issued = head;
        ok = mbar_wait(&ready_bar, 0, abortp) && !*abortp;  // no rows without a layout
        ok = __all_sync(0xffffffffu, ok);
        if (kMode != kModeLocal && ok) {   // the rest of the ring
            if (kSteal) {
                while (head < stages - 3 && next_token(tl, false) == 1) issue_item(tl);
            } else {
                while (head < min(stages - 3, ntok)) issue_item(head);
            }
            issued = head;
        }
        if (!kSteal) {
            // the CTA's own rows, in order: row n sits in stage n % stages
            const int n0 = x.early0 ? 1 : 0;   // (the first row's copies may have been issued by the row group)
            for (int n = n0; ok && n < ntok; ++n) {
                const int s = n % stages;
                ok = mbar_wait(&full_bar[s], (n / stages) & 1, abortp);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (n == n0 && lane == 0) trace(p, c, kTrFirstRow);
                const uint8_t* src = smem + (size_t)s * pl.stage_bytes;
                for (int j = lane; j < p.k; j += 32) {
                    const int where = pos[n * p.k + j];
                    if (where >= 0) bulk_store(p.recv_x + (size_t)where * p.rowB + out_off, src, out_bytes);
                }
                bulk_commit();
                if (head < ntok) {
                    bulk_wait_read<3>();     // every lane: its copies of the row 3 back have read the stage
                    __syncwarp();
                    issue_item(head);        // without stealing a row's index in the chunk is its sequence number
                    issued = head;
                }
            }
        }
        while (kSteal && ok) {
            if (tail == head) {
                // nothing queued: take over rows of another chunk, or finish
                if (feeder_done || next_token(tl, true) != 1) break;
                issue_item(tl);
                issued = head;
            }
            const int s = tail % stages;
            ok = mbar_wait(&full_bar[s], (tail / stages) & 1, abortp);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (tail == 0 && lane == 0) trace(p, c, kTrFirstRow);
            const uint8_t* src = smem + (size_t)s * pl.stage_bytes;
            const int from = kSteal ? item_src[s] : ((ch << 16) | tail);   // without stealing: own rows in order
            const bool own = (from >> 16) == ch;
            for (int j = lane; j < p.k; j += 32) {
                const int where = own ? pos[(from & 0xffff) * p.k + j] : item_pos[s * p.k + j];
                if (where >= 0) {
                    bulk_store(p.recv_x + (size_t)where * p.rowB + out_off, src, out_bytes);
                    if (kSteal) atomicAdd(&arr[where / p.cap], 1);   // rows per rank: counted by whoever copies
                }
            }
            bulk_commit();
            ++tail;
            if (!feeder_done && head - tail < stages - 3) {
                bulk_wait_read<3>();     // every lane: its copies of the row 3 back have read the stage
                __syncwarp();
                // own rows first, then rows of other chunks, all loaded as far ahead as the ring allows
                if (next_token(tl, true) == 1) issue_item(tl);
                issued = head;
            }
        }
    } else {
        if (fast_local) {
            const RankMaps rm{bmaps.bm, bmaps.mask_t, (p.R + 31) / 32, ((p.R + 31) / 32) * 32, (p.T + 31) / 32};
            local_stage_and_rank_maps(p, ids_sm, rm, rm.groups, 0, kWarps, lane);   // the table first, the rows after it
            group_sync(2, kThreads);
        } else if (kMode == kModeLocal || x.beside) {
            // the routing table first: it is the one load the layout waits for
            ok = mbar_wait(x.staged_bar, 0, abortp);
            ok = __all_sync(0xffffffffu, ok);
        }
        // loader only; the quantising warps free the stages.  A closing item with no row
        // tells them (and through them the store issuer) that nothing follows.  Rows are fetched as
        // far ahead as the rings allow, at most prefetch_rows of them before the layout is done.
        int tl = 0;
        bool ready_seen = kMode == kModeLocal;   // (the flag-free kernel: its quantisers start after the layout)
        auto wait_ready_at = [&](int n) -> bool {   // warp-uniform
            if (ready_seen || n < p.prefetch_rows) return true;
            bool r = true;
            if (lane == 0) r = mbar_wait(&ready_bar, 0, abortp);
            ready_seen = true;
            return __shfl_sync(0xffffffffu, (int)r, 0) != 0;
        };
        if (!kSteal) {
            // the CTA's own rows only: one thread, as far ahead as the ring allows
            while (ok && head < ntok) {
                ok = wait_ready_at(head);
                if (!ok) break;
                if (head >= stages) {
                    if (lane == 0) ok = mbar_wait(&empty_bar[head % stages], ((head / stages) - 1) & 1, abortp);
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (!ok) break;
                }
                tl = head;
                issue_item(tl);
                issued = head;
            }
        }
        while (kSteal && ok) {
            // rows of other chunks are taken only once all but two queued rows are consumed
            bool drained = head < 3;
            if (!drained) {
                const int hs = head - 3;
                drained = mbar_test_wait(&empty_bar[hs % stages], (hs / stages) & 1);
                drained = __all_sync(0xffffffffu, drained);
            }
            ok = wait_ready_at(head);
            if (!ok) break;
            const int got = feeder_done ? 0 : next_token(tl, drained);
            if (got == 2) {
                const int hs = head - 3;   // wait for the queue to drain, then ask again
                ok = mbar_wait(&empty_bar[hs % stages], (hs / stages) & 1, abortp);
                ok = __all_sync(0xffffffffu, ok);
                continue;
            }
            const int s = head % stages;
            if (head >= stages) {
                ok = mbar_wait(&empty_bar[s], ((head / stages) - 1) & 1, abortp);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
            }
            if (got == 1) {
                issue_item(tl);
                issued = head;
            } else {
                if (lane == 0) {   // (without stealing the consumers know the row count)
                    item_src[s] = -1;
                    mbar_arrive(&full_bar[s]);
                }
                break;
            }
        }
    }
    if (kFp8 && fast_local && ok) {
        // metadata of the CTA's own tokens (see the row group): one warp, no barrier but its own
        ok = mbar_wait(&ready_bar, 0, abortp);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            float* w_own = reinterpret_cast<float*>(key);   // the ordering keys are no longer needed
            if (part == 0)
                for (int i = lane; i < ntok * p.k; i += 32) w_own[i] = __ldg(p.topk_w + (size_t)t0 * p.k + i);
            local_clean_own_duplicates(p, t0, t1, ids_sm, lane, 32);
            __syncwarp();
            if (part == 0) local_meta_dedup(p, t0, t1, ids_sm, pos_raw, reinterpret_cast<int*>(w_sm), w_own, lane, 32);
        }
    }
    if (!ok && lane == 0) {
        report(p.status, kErrTimeout);  // a wait gave up: record it and let everybody leave
        abort_flag = 1;
    }
    if (lane == 0) trace(p, c, kTrIssued);
    bulk_wait_all<0>();
    if (lane == 0) trace(p, c, kTrStored);
}

// ---------------------------------------------------------------------- layout group
// Warps 1..15: TokenCnt, CalCumSum (by exchange or alone), slot -> row assignment; releases
// the movers and then writes what nobody inside the kernel waits for.  Returns 1, 0 if a wait ran
// out, or 2 for a warp that has done its share of the counting and now leaves to quantise.
template <int kMode, bool kFp8, bool kSteal>
__device__ __forceinline__ int layout_group(Cta& x) {
    UBEP_CTA_LOCALS(x, !kFp8);
    bool ok = true;
    const int* ids = ids_sm;  // staged slots of this CTA's tokens
    // Small global reads whose values are needed only after the first barriers: issue the
    // loads now (first trip of each loop), store to shared memory after the ids are staged.
    const int order_r = gtid < p.R ? __ldg(p.order_pos + gtid) : 0;
    const bool stage_w = !(kMode == kModeLocal && p.local_fast);
    const float w_first = (stage_w && gtid < ntok * p.k) ? __ldg(p.topk_w + (size_t)t0 * p.k + gtid) : 0.0f;
    auto stage_small = [&](int n) {   // by n threads
        if (gtid < p.R) order_sm[gtid] = order_r;
        for (int r = gtid + n; r < p.R; r += n) order_sm[r] = __ldg(p.order_pos + r);
        if (stage_w) {
            if (gtid < ntok * p.k) w_sm[gtid] = w_first;
            for (int i = gtid + n; i < ntok * p.k; i += n) w_sm[i] = __ldg(p.topk_w + (size_t)t0 * p.k + i);
        }
    };
    if (kMode == kModeLocal && p.local_fast) {
        // rank-level rows first, movers released, expert-level outputs afterwards
        const RankMaps rm{bmaps.bm, bmaps.mask_t, (p.R + 31) / 32, ((p.R + 31) / 32) * 32, (p.T + 31) / 32};
        int* row_sm = reinterpret_cast<int*>(w_sm);
        local_stage_and_rank_maps(p, ids_sm, rm, rm.groups, warp, kWarps, lane);   // with the mover warp
        stage_small(gn);
        group_sync(2, kThreads);
        if (gtid == 0) trace(p, c, kTrCounted);
        // From here the group splits.  Assigning rows to the CTA's own few tokens keeps a handful of
        // threads busy, and nothing expert-level depends on it: warps 1..4 (the row group) assign the
        // rows, release the movers and write the metadata of the own tokens, while the other warps
        // (the duty group) already derive the expert-level outputs from the staged table.  (One after
        // the other, the expert-level outputs ended after the last copy and set the kernel's duration.)
        constexpr int kRowWarps = 4, kRowThreads = kRowWarps * 32;
        if (gw < kRowWarps) {
            const int rn = kRowThreads;
            local_rows_dedup(p, t0, t1, ids_sm, rm, c, order_sm, pos_raw, key, row_sm, arr, gtid, rn);
            if (x.early0 && gw == 0) {
                // The copies of the CTA's first row leave from here: lane j has just worked out where slot j of
                // the first token goes (its own write to pos_raw), and the row was asked for before the routing
                // table was (and prefetched into L2 before that), so it sits in the ring's first stage or is
                // about to.  The mover warp, which needs another 0.5 us to notice the release and get going,
                // starts with the second row.  (Measured per layer, 512 tokens: 25.2 us against 25.6; neither
                // this nor the prefetch of the rows changes anything without the other.)
                const int where = lane < p.k ? pos_raw[lane] : -1;
                const bool got = mbar_wait(&full_bar[0], 0, abortp);
                if (got && where >= 0) bulk_store(p.recv_x + (size_t)where * p.rowB + out_off, smem, out_bytes);
                bulk_commit();
                if (!got && lane == 0) {
                    report(p.status, kErrTimeout);
                    *abortp = 1;
                }
            }
            group_sync(1, rn);
            if (gtid == 0) trace(p, c, kTrFinalized);
            if (p.ordered) {   // a destination table is set: the copies of a token in its order (else pos_raw is pos)
                order_destinations(p, pos_raw, key, pos, ntok * p.k, gtid, rn);
                group_sync(1, rn);
            }
            unsigned ticket = 0u, ep_mine = 0u;
            if (gtid == 0) {
                mbar_arrive(&ready_bar);
                trace(p, c, kTrReady);
                // The epoch: nothing needs it before the kernel's last lines.  A relaxed load (nothing
                // is ordered against it); its value is in hand before the ticket is taken -- the store
                // to shared memory needs it -- and the ticket's answer is looked at at the end.
                ep_mine = epoch_from_counter(ld_relaxed(p.epoch_ctr));
                *x.epoch_late = ep_mine;
                ticket = atomicAdd(p.done_ticket, 1u);
            }
            if (kFp8) {
                // FP8 rows: every copy waits for a quantised row, so this group goes straight on to quantise
                // (its first warp to issue the copies; the warps of the duty group take no part, a CTA of
                // this kernel has few rows).  The metadata of the own tokens is written by the loader warp,
                // which is idle once the CTA's few rows are asked for.
                if (gtid == 0) epoch_finish_check_in(p, ticket, ep_mine);
                return 1;
            }
            if (part == 0) {
                float* w_own = reinterpret_cast<float*>(key);   // the ordering keys are no longer needed
                for (int i = gtid; i < ntok * p.k; i += rn) w_own[i] = __ldg(p.topk_w + (size_t)t0 * p.k + i);
            }
            local_clean_own_duplicates(p, t0, t1, ids_sm, gtid, rn);   // (rank-level rows do not depend on them)
            group_sync(1, rn);
            if (p.trace && gtid == 0) p.trace[(size_t)c * kTraceSlots + 11] = trace_ns(p);
            if (part == 0) local_meta_dedup(p, t0, t1, ids_sm, pos_raw, row_sm, reinterpret_cast<float*>(key), gtid, rn);
            if (gtid == 0) {
                epoch_finish_check_in(p, ticket, ep_mine);
                if (p.trace) p.trace[(size_t)c * kTraceSlots + 12] = trace_ns(p);
            }
        } else if (kFp8 && warp - x.qwarp0 < x.nq) {
            return 1;   // FP8 rows: the first warps behind the row group quantise as well
        } else {
            // expert-level outputs of rank r: shared by Q CTAs so that no CTA trails the others
            const int dgw0 = kFp8 ? max(kRowWarps, x.qwarp0 + x.nq - 1) : kRowWarps;   // first warp of the duty group
            const int dn = gn - dgw0 * 32, dw = nw - dgw0;
            const int Q = p.grid / p.R > 1 ? p.grid / p.R : 1;
            // ... once the movers are released: started earlier, these warps take issue slots and
            // shared-memory bandwidth from the few threads every copy of this CTA is waiting for
            const bool go = mbar_wait_idle(&ready_bar, 0, abortp);
            for (int u = c; go && u < p.R * Q; u += p.grid)
                local_rank_duty(p, u / Q, u % Q, Q, ids_sm, rm, hist, gw - dgw0, dw, lane, gtid - dgw0 * 32, dn, 3);
            if (gtid == dgw0 * 32) trace(p, c, kTrScanned);   // deferred outputs written
            if (kFp8) return go ? 3 : 0;   // (these warps do not quantise: the row group's warps do)
        }
    } else if (kMode == kModeLocal) {
        // every CTA: bitmaps over the whole routing table -> totals, the rows before its
        // own tokens, and (CTAs with a source-rank duty) that rank's counts
        int* tot = hist;
        int* pre = hist + p.B;
        int* eo = hist + 2 * p.B;
        stage_ids(p, 0, p.T, ids_sm, gtid, gn);
        stage_small(gn);
        group_sync(1, gn);
        if (gtid == 0) {
            mbar_arrive(x.staged_bar);   // the mover may fetch rows now
            trace(p, c, kTrCounted);
        }
        local_counts_all_bins(p, ids_sm, bmaps, t0, tot, pre, eo, gtid, gn, gw, nw, lane, 1);
        if (gtid == 0) trace(p, c, kTrScanSeen);
        ids = ids_sm + (size_t)t0 * p.k;
        finalize_chunk(p, t0, t1, ids, w_sm,
                       [&](int e, int tl) { return eo[e] + pre[e] + bits_in_range(bmaps, e, t0, t0 + tl); },
                       [&](int r, int tl) { return pre[p.E + r] + bits_in_range(bmaps, p.E + r, t0, t0 + tl); },
                       part == 0, c, order_sm, pos_raw, key, arr, gtid, gn);
        group_sync(1, gn);
        if (gtid == 0) trace(p, c, kTrFinalized);
        if (p.ordered) {   // a destination table is set: the copies of a token in its order (else pos_raw is pos)
            order_destinations(p, pos_raw, key, pos, ntok * p.k, gtid, gn);
            group_sync(1, gn);
        }
        if (gtid == 0) {
            mbar_arrive(&ready_bar);
            trace(p, c, kTrReady);
            *x.epoch_late = read_epoch_and_check_in(p);   // nothing needs it before the kernel's last lines
        }
        // outputs nobody inside this kernel waits for
        if (c == 0) write_totals(p, tot, eo, gtid, gn);
        if (part == 0)
            for (int s = ch; s < p.S; s += p.nchunks) write_source_from_maps(p, s, bmaps, eo, gtid, gn);   // source ranks this CTA reports
    } else {
        // FP8 rows with a count group: TokenCnt itself -- staging the ids, the bitmaps, publishing the
        // chunk's counts -- is pure computation and is done by all 15 warps; then the warps behind the
        // count group leave to quantise, and the count group alone goes through the steps that mostly
        // wait for other CTAs (flag exchange, CalCumSum duty) and assigns the rows.
        const bool split = kFp8 && x.beside;
        const int an = split ? kThreads - 32 : gn, aw = split ? kWarps - 1 : nw;
        const int bid = split ? 4 : 1;   // barrier of the count group once the others have left
        stage_ids(p, t0, t1, ids_sm, gtid, an);
        stage_small(an);
        group_sync(1, an);
        if (kFp8 && gtid == 0) mbar_arrive(x.staged_bar);   // the loader may fetch rows now
        build_bin_maps(p, ids_sm, ntok, bmaps, gw, aw, lane);
        group_sync(1, an);
        if (kMode == kModeFused) publish_chunk_counts(p, ch, t0, t1, bmaps, gtid, an);
        if (split) {
            group_sync(1, an);          // the counts are stored (the flag is released further down)
            if (gw >= nw) return 2;     // off to quantise
        }
        int deferred = -1;
        // The mover warp fetched the epoch while the table was staged; one thread makes sure it has
        // arrived, the barrier that follows hands it to the others.
        unsigned ep = 0;
        auto learn_epoch = [&]() {
            if (gtid == 0) (void)mbar_wait(x.epoch_bar, 0, abortp);
            group_sync(bid, gn);
            ep = *reinterpret_cast<volatile unsigned*>(x.epoch_late);
        };
        if (kMode == kModeFused) {
            learn_epoch();
            if (gtid == 0) {
                if (ch != p.withhold) {
                    st_release(p.hist_flag + ch, ep);   // release: cumulative over what the barrier above ordered
                }
                trace(p, c, kTrCounted);
            }
            // CalCumSum duty: this CTA serves rank ch (and ch + nchunks, ...)
            bool lost = false;  // a wait of this thread ran out
            for (int r = ch; r < p.R; r += p.nchunks) {
                for (int cc = gtid; cc < p.nchunks; cc += gn)
                    if (!wait_flag(p.hist_flag + cc, ep, abortp)) lost = true;
                if (group_or(bid, gn, lost || *abortp)) { lost = true; break; }  // same answer for all
                if (gtid == 0) trace(p, c, kTrHistSeen);
                scan_rank_publish(p, r, hist, gw, nw, lane, bid);
                if (gtid == 0) {
                    st_release(p.scan_flag + r, ep);
                    trace(p, c, kTrScanned);
                }
                if (r + p.nchunks < p.R) {
                    scan_rank_sources(p, r, hist, gtid, gn);
                    group_sync(bid, gn);
                } else {
                    deferred = r;   // cnt / src_offset: after our own movers are released
                }
            }
            // every slot of this chunk may need any rank's bases
            if (!lost)
                for (int r = gtid; r < p.R; r += gn)
                    if (!wait_flag(p.scan_flag + r, ep, abortp)) lost = true;
            ok = !group_or(bid, gn, lost || *abortp);
            if (gtid == 0) trace(p, c, kTrScanSeen);
            if (!ok && gtid == 0) {
                report(p.status, kErrTimeout);
                abort_flag = 1;
            }
        }
        if (ok) {
            // rows before a token = rows of earlier chunks (+ the expert's offset in its
            // region), published by the prefix-sum step, + earlier tokens of this chunk.
            // The published part is fetched once per bin into shared memory (one round
            // trip to L2), the rest is bit counting.
            const int32_t* cb = p.chunk_base + ch;   // [bin][chunk]
            int* base_sm = hist + p.B;   // second half of the scratch (the first may hold scan totals)
            for (int b = gtid; b < p.B; b += gn)
                base_sm[b] = __ldcg(cb + (size_t)b * p.nchunks) + (b < p.E ? __ldcg(p.expert_offset + b) : 0);
            group_sync(bid, gn);
            finalize_chunk(p, t0, t1, ids, w_sm,
                           [&](int e, int tl) { return base_sm[e] + bits_in_range(bmaps, e, 0, tl); },
                           [&](int r, int tl) { return base_sm[p.E + r] + bits_in_range(bmaps, p.E + r, 0, tl); },
                           true, c, order_sm, pos_raw, key, kSteal ? nullptr : arr, gtid, gn);
            group_sync(bid, gn);
            if (gtid == 0) trace(p, c, kTrFinalized);
            if (p.ordered) {   // a destination table is set: the copies of a token in its order (else pos_raw is pos)
                order_destinations(p, pos_raw, key, pos, ntok * p.k, gtid, gn);
                group_sync(bid, gn);
            }
        }
        if (gtid == 0) {
            mbar_arrive(&ready_bar);
            trace(p, c, kTrReady);
        }
        if (ok && kSteal) {
            // this chunk's destinations, for CTAs that run out of work and take over some of its tokens
            for (int i = gtid; i < ntok * p.k; i += gn) p.copy_pos[(size_t)t0 * p.k + i] = pos[i];
            if (kMode == kModeFused) group_sync(bid, gn);
            else learn_epoch();   // (with kernel boundaries instead of flags nothing has asked for it yet)
            if (gtid == 0) {
                st_release(p.pos_flag + ch, ep);
            }
        }
        if (ok && deferred >= 0) scan_rank_sources(p, deferred, hist, gtid, gn);
    }
    return ok ? 1 : 0;
}

// ------------------------------------------------------------ FP8: quantise and store
// Two roles around a ring of quantised rows (payload + scales).  The quantising warps turn the
// rows the loader has fetched into FP8 and know nothing about destinations (own rows) -- so they
// can run beside the layout; the store issuer sends every quantised row to its destinations
// with bulk copies once the layout is done.
//
// Shared-memory bookkeeping behind the input ring's items: out_src[os] = where the row of
// output stage os comes from (chunk << 16 | index, -1 = nothing follows), out_pos[os] = the
// destinations of a row taken over from another chunk.
struct Fp8Ring {
    uint8_t* out_ring;
    const int* item_src;   // [kMaxStages]
    const int* item_pos;   // [kMaxStages, k]
    int* out_src;          // [kMaxOutStages]
    int* out_pos;          // [kMaxOutStages, k]
    int g0;                // first scale group of this CTA's piece
    unsigned scale_bytes;  // its scales travel with the payload
    bool scale_bulk;       // ... by a bulk copy when their size allows it
};
__device__ __forceinline__ Fp8Ring fp8_ring(const Cta& x) {
    const Params& p = x.p;
    int* item = reinterpret_cast<int*>(x.smem + x.pl.off_item);
    Fp8Ring q;
    q.out_ring = x.smem + x.pl.off_out;
    q.item_src = item;
    q.out_src = item + kMaxStages;
    q.item_pos = item + kMaxStages + kMaxOutStages;
    q.out_pos = item + kMaxStages + kMaxOutStages + kMaxStages * p.k;
    q.g0 = x.part * (p.G / p.parts);
    q.scale_bytes = (unsigned)(p.G / p.parts) * 4u;
    q.scale_bulk = (q.scale_bytes & 15u) == 0;
    return q;
}

// Quantising warp qw of nq.
template <bool kSteal>
__device__ __forceinline__ void fp8_quantiser(Cta& x, int qw) {
    UBEP_CTA_LOCALS(x, false);
    const Fp8Ring q = fp8_ring(x);
    const int nvec = (int)in_bytes / 16;          // 8-channel vectors in this CTA's piece
    unsigned long long w_in = 0, w_out = 0, t_cmp = 0, tq = 0;
    for (int n = 0; kSteal || n < ntok; ++n) {
        const int s = n % stages, os = n % out_stages;
        if (p.trace) tq = trace_ns(p);
        if (!mbar_wait_idle(&full_bar[s], (n / stages) & 1, abortp)) break;
        if (p.trace) { unsigned long long t2 = trace_ns(p); w_in += t2 - tq; tq = t2; }
        if (n >= out_stages && !mbar_wait_idle(&out_empty[os], ((n / out_stages) - 1) & 1, abortp)) break;
        if (p.trace) { unsigned long long t2 = trace_ns(p); w_out += t2 - tq; tq = t2; }
        const int from = kSteal ? q.item_src[s] : ((ch << 16) | n);
        if (from < 0) {
            // the loader's closing item: pass it on to the store issuer and leave
            if (qw == 0 && lane == 0) q.out_src[os] = -1;
            __syncwarp();
            if (lane == 0) mbar_arrive(&out_full[os]);
            break;
        }
        if (kSteal && qw == 0) {
            if ((from >> 16) != ch)   // a row of another chunk: its destinations travel with it
                for (int j = lane; j < p.k; j += 32) q.out_pos[os * p.k + j] = q.item_pos[s * p.k + j];
            if (lane == 0) q.out_src[os] = from;
        }
        const uint8_t* src = smem + (size_t)s * pl.stage_bytes;
        uint8_t* dst = q.out_ring + (size_t)os * pl.out_stage_bytes;
        float* dst_scale = reinterpret_cast<float*>(dst + out_bytes);
        // two vectors per thread and trip, independent of each other
        for (int vb = qw * 32; vb < nvec; vb += 2 * nq * 32) {
            const int v0 = vb + lane, v1 = v0 + nq * 32;
            const bool ok0 = v0 < nvec, ok1 = v1 < nvec;
            uint4 in0 = make_uint4(0, 0, 0, 0), in1 = make_uint4(0, 0, 0, 0);
            if (ok0) in0 = *reinterpret_cast<const uint4*>(src + (size_t)v0 * 16);
            if (ok1) in1 = *reinterpret_cast<const uint4*>(src + (size_t)v1 * 16);
            uint2 q0, q1;
            float sc0, sc1;
            quantize8(in0, ok0, q0, sc0);
            quantize8(in1, ok1, q1, sc1);
            if (ok0) *reinterpret_cast<uint2*>(dst + (size_t)v0 * 8) = q0;
            if (ok1) *reinterpret_cast<uint2*>(dst + (size_t)v1 * 8) = q1;
            if ((lane & 15) == 0) {
                if (ok0) dst_scale[v0 >> 4] = sc0;
                if (ok1) dst_scale[v1 >> 4] = sc1;
            }
        }
        fence_proxy_async_smem();   // the bulk stores read what we just wrote
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(&out_full[os]);
            mbar_arrive(&empty_bar[s]);
        }
        if (p.trace) t_cmp += trace_ns(p) - tq;
    }
    if (p.trace && qw == 0 && lane == 0) {
        p.trace[(size_t)c * kTraceSlots + 11] = w_in;
        p.trace[(size_t)c * kTraceSlots + 12] = w_out;
        p.trace[(size_t)c * kTraceSlots + 13] = t_cmp;
    }
}

// Store issuer (one warp, after the layout): lane j issues the copy of slot j.
template <bool kSteal>
__device__ __forceinline__ void fp8_store_issuer(Cta& x) {
    UBEP_CTA_LOCALS(x, false);
    const Fp8Ring q = fp8_ring(x);
    const int Gp = p.G / p.parts;   // scale groups of this CTA's piece
    bool sok = true;
    unsigned long long w_full = 0, w_read = 0, tq = 0;
    for (int n = 0; kSteal || n < ntok; ++n) {
        const int os = n % out_stages;
        if (p.trace) tq = trace_ns(p);
        sok = mbar_wait(&out_full[os], (n / out_stages) & 1, abortp);
        if (p.trace) w_full += trace_ns(p) - tq;
        sok = __all_sync(0xffffffffu, sok);
        const int from = kSteal ? q.out_src[os] : ((ch << 16) | n);
        if (!sok || from < 0) break;
        if (n == 0 && lane == 0) trace(p, c, kTrFirstRow);
        const int* wpos = (from >> 16) == ch ? pos + (from & 0xffff) * p.k : q.out_pos + os * p.k;
        const uint8_t* src = q.out_ring + (size_t)os * pl.out_stage_bytes;
        // lanes 0..k-1: payload of slot j; lanes k..2k-1: its scales (when bulk-storable)
        for (int j = lane; j < (q.scale_bulk ? 2 * p.k : p.k); j += 32) {
            const int jj = j < p.k ? j : j - p.k;
            const int where = wpos[jj];
            if (where < 0) continue;
            if (j < p.k) {
                bulk_store(p.recv_x + (size_t)where * p.rowB + out_off, src, out_bytes);
                if (kSteal) atomicAdd(&arr[where / p.cap], 1);
            } else {
                bulk_store(p.recv_scale + (size_t)where * p.G + q.g0, src + out_bytes, q.scale_bytes);
            }
        }
        if (!q.scale_bulk) {   // a piece of scales that no bulk copy can carry: plain stores
            const float* sc = reinterpret_cast<const float*>(src + out_bytes);
            for (int i = lane; i < p.k * Gp; i += 32) {
                const int jj = i / Gp, g = i - jj * Gp;
                const int where = wpos[jj];
                if (where >= 0) p.recv_scale[(size_t)where * p.G + q.g0 + g] = sc[g];
            }
        }
        bulk_commit();
        if (n + 1 >= kStorePending) {
            if (p.trace) tq = trace_ns(p);
            bulk_wait_read<kStorePending - 1>();   // every lane: the copies of the row kStorePending - 1 back have read it
            if (p.trace) w_read += trace_ns(p) - tq;
            __syncwarp();
            if (lane == 0) mbar_arrive(&out_empty[(n + 1 - kStorePending) % out_stages]);
        }
    }
    if (!sok && lane == 0) {
        report(p.status, kErrTimeout);
        abort_flag = 1;
    }
    bulk_wait_all<0>();
    if (p.trace && lane == 0) {
        p.trace[(size_t)c * kTraceSlots + 14] = w_full;
        p.trace[(size_t)c * kTraceSlots + 15] = w_read;
    }
}

// --------------------------------------------------------------------- dispatch kernel
// Warp roles: warp 0 = mover; warps 1..15 = layout group (count, prefix sums, row
// assignment).  FP8 rows: warp 0 only loads; either the layout group is warps 1 .. count_warps and
// the warps behind them quantise beside it (the kernels whose layout waits for other CTAs or was
// computed by earlier launches), or all 15 warps compute the layout and warps 2..15 quantise
// afterwards (the flag-free kernel, whose layout is pure computation); warp 1 issues the stores
// once the layout is done.
template <int kMode, bool kFp8, bool kSteal>
__global__ void __launch_bounds__(kThreads, 1) dispatch_kernel(const Params p, const SmemPlan pl) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];    // input row landed
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];   // FP8: input row consumed
    __shared__ __align__(8) uint64_t out_full[kMaxOutStages];    // FP8: quantised row written
    __shared__ __align__(8) uint64_t out_empty[kMaxOutStages];   // FP8: its stores have read it
    __shared__ __align__(8) uint64_t ready_bar;               // rows assigned, movers may go
    __shared__ __align__(8) uint64_t epoch_bar;               // epoch_sm holds this launch's epoch
    __shared__ __align__(8) uint64_t staged_bar;              // flag-free kernel: the routing table is in shared memory
    __shared__ int abort_flag;
    __shared__ unsigned epoch_sm;

    const int tid = threadIdx.x;
    const int c = blockIdx.x;
    const int part = c % p.parts, ch = c / p.parts;
    const int t0 = (int)chunk_begin(ch, p.T, p.nchunks), t1 = (int)chunk_begin(ch + 1, p.T, p.nchunks);
    const int stages = pl.stages;
    const bool beside = kFp8 && kMode != kModeLocal && p.count_warps > 0;
    const int nw = beside ? p.count_warps : kWarps - 1;      // layout group: warps 1 .. nw
    const int qwarp0 = beside ? nw + 1 : 2;                    // FP8: warps qwarp0 .. qwarp0 + nq - 1 quantise
    // (flag-free kernel with rank-level rows: a CTA has few rows, and the warps that do not quantise write
    // the expert-level outputs meanwhile)
    const int nq = kFp8 ? min(kMode == kModeLocal && p.local_fast ? min(p.quant_warps, kFastQuantWarps) : p.quant_warps, kWarps - qwarp0)
                        : kWarps - 2;
    int* arr = reinterpret_cast<int*>(smem + pl.off_arr);
    griddep_launch();   // the next kernel in the stream may be placed as soon as SMs have room

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], nq);
        }
        for (int s = 0; s < pl.out_stages; ++s) {
            mbar_init(&out_full[s], nq);
            mbar_init(&out_empty[s], 1);
        }
        mbar_init(&ready_bar, 1);
        mbar_init(&epoch_bar, 1);
        mbar_init(&staged_bar, 1);
        abort_flag = 0;
        epoch_sm = 0u;
        mbar_fence_init();
    }
    for (int r = tid; r < p.R; r += kThreads) arr[r] = 0;
    if (kMode == kModeLocal) {
        // The routing table is the first thing every CTA of the flag-free kernel needs, and it comes cold
        // from HBM.  A prefetch into L2 reads no value, so it may run ahead of the wait below: L2 is where
        // an earlier kernel's stores to the table land too, so the line cannot go stale.
        const char* tab = reinterpret_cast<const char*>(p.topk_idx);
        const size_t bytes = (size_t)p.T * p.k * 4;
        for (size_t off = ((size_t)c * kThreads + tid) * 128; off < bytes; off += (size_t)p.grid * kThreads * 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(tab + off));
        // The same for the CTA's own pieces of its rows: inside a layer they come from HBM while it is still
        // writing back what the kernels before left in L2, and the first of them is what the first copy waits for.
        const unsigned piece = (unsigned)(p.H * 2 / p.parts);
        const int lines = (int)((piece + 127u) / 128u);
        const char* xs = reinterpret_cast<const char*>(p.x) + (size_t)t0 * p.H * 2 + (size_t)part * piece;
        for (int i = tid; i < (t1 - t0) * lines; i += kThreads) {
            const int tl = i / lines, l = i - tl * lines;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(xs + (size_t)tl * p.H * 2 + (size_t)l * 128));
        }
    }
    griddep_wait();     // shared-memory set-up done; everything below reads what earlier kernels wrote
    // The epoch is not read here, in front of everything: the flag-free kernel needs it only for the
    // arrival counters at its very end and reads it once the movers are released; in the other
    // kernels the mover warp fetches it while the layout group stages the routing table.
    if (tid == 0) trace_begin(p, c);
    __syncthreads();
    const unsigned epoch = 0u;

    const unsigned in_bytes = (unsigned)(p.H * 2 / p.parts);   // this CTA's piece of a bf16 row
    const unsigned out_bytes = (unsigned)(p.rowB / p.parts);   // and of a payload row
    Cta x{p, pl, smem, full_bar, empty_bar, out_full, out_empty, &ready_bar, &epoch_bar, &staged_bar, &abort_flag,
          tid, tid & 31, tid >> 5, c, part, ch, t0, t1, t1 - t0, stages, nq,
          nw * 32, nw, pl.out_stages, qwarp0, beside,
          reinterpret_cast<int*>(smem + pl.off_ids),
          reinterpret_cast<int*>(smem + pl.off_ord),    // destinations in issue order
          reinterpret_cast<int*>(smem + (p.ordered ? pl.off_pos : pl.off_ord)),   // in slot order (the same array
                                                                                  // when no table reorders them)
          reinterpret_cast<int*>(smem + pl.off_key),
          reinterpret_cast<float*>(smem + pl.off_w),
          BinMaps{reinterpret_cast<unsigned*>(smem + pl.off_mask), reinterpret_cast<unsigned*>(smem + pl.off_bm),
                  pl.map_wb, pl.map_bp, pl.map_groups},
          reinterpret_cast<int*>(smem + pl.off_hist), arr, reinterpret_cast<int*>(smem + pl.off_order),
          epoch, in_bytes, out_bytes, &epoch_sm, (size_t)part * in_bytes, (size_t)part * out_bytes,
          kMode == kModeLocal && p.local_fast != 0,
          // (its stage is never loaded a second time, no order of destinations is asked for, a lane per copy)
          kMode == kModeLocal && p.local_fast != 0 && !kFp8 && !kSteal && !p.ordered && p.k <= 32 && t1 > t0 &&
              t1 - t0 <= stages,
          0};

    if (x.warp == 0) {
        mover_warp<kMode, kFp8, kSteal>(x);
    } else {
        const int lg = layout_group<kMode, kFp8, kSteal>(x);   // 0 = a wait ran out, 1 = done, 2 = left to quantise
        if (!kFp8 && x.early0 && x.warp == 1) bulk_wait_all<0>();   // the first row's copies (issued by this warp)
        if (kFp8 && lg == 2) {
            if (x.warp - qwarp0 < nq) fp8_quantiser<kSteal>(x, x.warp - qwarp0);   // beside the rest of the layout
        } else if (kFp8 && lg == 1) {
            if (x.warp == 1) fp8_store_issuer<kSteal>(x);
            else if (!beside && x.warp - 2 < nq) fp8_quantiser<kSteal>(x, x.warp - 2);
        }
    }
    __syncthreads();
    const unsigned half = epoch_sm & 1u;
    if (abort_flag) {
        // leaving early.  The arrival counters of the next call live in the other half; they are
        // cleared here too, otherwise the call after the next one would add to stale totals.
        // (epoch_sm == 0: the call gave up before it learnt its epoch and has used neither half.)
        if (c == 0 && epoch_sm != 0u) {
            for (int r = tid; r < p.R; r += kThreads) p.arrival[(half ^ 1u) * p.R + r] = 0;
            if (tid == 0) p.claimed[half ^ 1u] = 0;
        }
        // the newest load of every ring stage may still be landing
        if (tid == 0) {
            for (int n = max(0, x.issued - stages); n < x.issued; ++n)
                (void)mbar_wait(&full_bar[n % stages], (n / stages) & 1, nullptr);
        }
        return;
    }
    // pieces of this CTA's rows have landed: add them to the per-region arrival counters
    // (unit: eighths of a row, so that the total does not depend on the column split)
    fence_proxy_async();   // rows written through the async proxy, counters through the generic one
    for (int r = tid; r < p.R; r += kThreads)
        if (arr[r]) red_release_add(p.arrival + half * p.R + r, (unsigned)(arr[r] * (8 / p.parts)));
    // the arrival counters of the next call live in the other half; clear them now
    if (c == 0) {
        for (int r = tid; r < p.R; r += kThreads) p.arrival[(half ^ 1u) * p.R + r] = 0;
        if (tid == 0) p.claimed[half ^ 1u] = 0;   // same for the count of tokens handed out
    }
    if (tid == 0) trace(p, c, kTrEnd);
}

// ---------------------------------------------------------------------------- combine
// One thread per 16-byte vector of the output row: K independent 128-bit gathers, fp32
// fused multiply-adds in slot order, one round-to-nearest-even pack to bf16.
template <int K>
__global__ void __launch_bounds__(256) combine_kernel(const uint16_t* __restrict__ y,
                                                     const int32_t* __restrict__ slot_pos,
                                                     const float* __restrict__ topk_w, int T, int H, int k,
                                                     uint16_t* __restrict__ out) {
    const int nvec = H / 8;
    const int64_t total = (int64_t)T * nvec;
    const int kk = K > 0 ? K : k;
    griddep_launch();   // lets a dispatch that follows in the stream be placed while this kernel drains
    griddep_wait();     // (only matters when this kernel itself was launched ahead of its predecessor's end)
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total;
         u += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(u / nvec), v = (int)(u - (int64_t)t * nvec);
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
        if (K > 0) {
            constexpr int KK = K > 0 ? K : 1;
            uint4 q[KK];
            float w[KK];
            int wh[KK];
#pragma unroll
            for (int j = 0; j < KK; ++j) {
                wh[j] = __ldg(slot_pos + (size_t)t * KK + j);
                w[j] = __ldg(topk_w + (size_t)t * KK + j);
            }
#pragma unroll
            for (int j = 0; j < KK; ++j) {
                q[j] = make_uint4(0, 0, 0, 0);
                if (wh[j] >= 0) q[j] = __ldg(reinterpret_cast<const uint4*>(y + (size_t)wh[j] * H) + v);
            }
#pragma unroll
            for (int j = 0; j < KK; ++j) {
                if (wh[j] < 0) continue;  // an empty slot contributes nothing
                const uint32_t ww[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[2 * i] = __fmaf_rn(w[j], __uint_as_float(ww[i] << 16), acc[2 * i]);
                    acc[2 * i + 1] = __fmaf_rn(w[j], __uint_as_float(ww[i] & 0xffff0000u), acc[2 * i + 1]);
                }
            }
        } else {
            for (int j = 0; j < kk; ++j) {
                const int where = __ldg(slot_pos + (size_t)t * kk + j);
                if (where < 0) continue;
                const float w = __ldg(topk_w + (size_t)t * kk + j);
                const uint4 q = __ldg(reinterpret_cast<const uint4*>(y + (size_t)where * H) + v);
                const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[2 * i] = __fmaf_rn(w, __uint_as_float(ww[i] << 16), acc[2 * i]);
                    acc[2 * i + 1] = __fmaf_rn(w, __uint_as_float(ww[i] & 0xffff0000u), acc[2 * i + 1]);
                }
            }
        }
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
            o[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        reinterpret_cast<uint4*>(out + (size_t)t * H)[v] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// ---------------------------------------------------------------- counts-only layout
// ubep_get_dispatch_layout: every CTA histograms its token chunk in shared memory, writes
// the chunk histogram to scratch, and the last CTA to finish (ticket) sums the chunks.
__global__ void __launch_bounds__(256) layout_kernel(const Params p, int32_t* num_tokens_per_rank,
                                                    int32_t* num_tokens_per_expert,
                                                    uint8_t* is_token_in_rank, int32_t* scratch_hist,
                                                    unsigned* ticket) {
    extern __shared__ int sm_i[];
    __shared__ bool last;
    const int B = p.B, k = p.k, R = p.R, n = gridDim.x, c = blockIdx.x;
    const int t0 = (int)chunk_begin(c, p.T, n), t1 = (int)chunk_begin(c + 1, p.T, n);
    for (int b = threadIdx.x; b < B; b += blockDim.x) sm_i[b] = 0;
    if (is_token_in_rank) {
        uint8_t* z = is_token_in_rank + (size_t)t0 * R;
        for (size_t i = threadIdx.x; i < (size_t)(t1 - t0) * R; i += blockDim.x) z[i] = 0;
    }
    __syncthreads();
    for (int t = t0 + threadIdx.x; t < t1; t += blockDim.x) {
        int seen[kMaxTopk], seen_e[kMaxTopk];
        for (int j = 0; j < k; ++j) {
            int e = resolve_expert(p, t, __ldg(p.topk_idx + (size_t)t * k + j));
            for (int jj = 0; jj < j; ++jj)
                if (e >= 0 && seen_e[jj] == e) {   // an expert named twice: reported, the later slot counts as empty
                    report(p.status, kErrBadIndex);
                    e = -1;
                }
            seen_e[j] = e;
            int r = -1;
            if (e >= 0) {
                atomicAdd(&sm_i[e], 1);
                r = e / p.L;
                bool first = true;
                for (int jj = 0; jj < j; ++jj) first = first && seen[jj] != r;
                if (first) {
                    atomicAdd(&sm_i[p.E + r], 1);
                    if (is_token_in_rank) is_token_in_rank[(size_t)t * R + r] = 1;
                }
            }
            seen[j] = r;
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < B; b += blockDim.x) scratch_hist[(size_t)c * B + b] = sm_i[b];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(ticket, 1u) == (unsigned)(n - 1);
    __syncthreads();
    if (!last) return;
    __threadfence();
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        int sum = 0;
        for (int cc = 0; cc < n; ++cc) sum += __ldcg(scratch_hist + (size_t)cc * B + b);
        if (b < p.E) {
            if (num_tokens_per_expert) num_tokens_per_expert[b] = sum;
        } else if (num_tokens_per_rank) {
            num_tokens_per_rank[b - p.E] = sum;
        }
    }
    if (threadIdx.x == 0) *ticket = 0;  // ready for the next call
}

// ------------------------------------------------------------------------- launchers

static int round_up_i(int v, int m) { return (v + m - 1) / m * m; }

// Shared-memory plan of the dispatch kernel for one call; -1 if it cannot fit.
int plan_dispatch(const Params& p, int mode, int max_smem, SmemPlan* out) {
    SmemPlan pl{};
    const int chunk_tokens = (p.T + p.nchunks - 1) / p.nchunks;
    const int chunk_slots = chunk_tokens * p.k;
    const int map_tokens = mode == kModeLocal ? p.T : chunk_tokens;   // tokens the bitmaps cover
    const int64_t ids_ints = (int64_t)map_tokens * p.k;
    int hist_ints = mode == kModeLocal ? 2 * p.B + p.E : 2 * p.B;
    if (hist_ints < 64) hist_ints = 64;   // the per-rank duty of the flag-free kernel keeps 2 x 32 ints here
    pl.map_groups = (map_tokens + 31) / 32;
    pl.map_wb = (p.B + 31) / 32;
    pl.map_bp = pl.map_wb * 32;
    pl.stage_bytes = round_up_i(p.H * 2 / p.parts, 128);
    pl.out_stage_bytes = p.payload ? round_up_i(p.rowB / p.parts + (p.G / p.parts) * 4, 128) : 0;
    const int64_t mask_ints = (int64_t)pl.map_groups * 32;
    const int64_t bm_ints = (int64_t)pl.map_groups * pl.map_bp;
    const int item_ints = (kMaxStages + kMaxOutStages) * (p.k + 1);
    const int64_t ints = ids_ints + mask_ints + bm_ints + 4 * (int64_t)chunk_slots + hist_ints + 2 * p.R + item_ints;
    const int64_t fixed = ints * 4 + 128 + 1536;  // 1.5 KB: static shared memory
    // no more stages than rows this CTA will ever hold at once
    const int want = chunk_tokens + 3 < 4 ? 4 : chunk_tokens + 3;
    const bool beside = p.payload && mode != kModeLocal && p.count_warps > 0;
    if (!beside) {
        // the quantising warps (if any) start after the layout: a deep input ring that the loader fills
        // meanwhile, a short ring of quantised rows
        pl.out_stages = p.payload ? kOutStages : 0;
        const int64_t rest = max_smem - fixed - (int64_t)pl.out_stages * pl.out_stage_bytes;
        if (rest < 4 * (int64_t)pl.stage_bytes) return -1;
        pl.stages = (int)(rest / pl.stage_bytes);
        if (pl.stages > kMaxStages) pl.stages = kMaxStages;
        if (pl.stages > want) pl.stages = want;
    } else {
        // the quantising warps run beside the layout: a short input ring (enough loads in flight to keep
        // them busy) and as many quantised rows as fit, which wait for the layout
        const int64_t room = max_smem - fixed;
        if (room < 2 * (int64_t)pl.stage_bytes + 4 * (int64_t)pl.out_stage_bytes) return -1;
        pl.stages = 4;
        while (pl.stages > 2 && room < (int64_t)pl.stages * pl.stage_bytes + 4 * (int64_t)pl.out_stage_bytes) --pl.stages;
        pl.out_stages = (int)((room - (int64_t)pl.stages * pl.stage_bytes) / pl.out_stage_bytes);
        if (pl.out_stages > kMaxOutStages) pl.out_stages = kMaxOutStages;
        if (pl.out_stages > want) pl.out_stages = want < 4 ? 4 : want;
        // what is left over goes to the input ring
        const int more = (int)((room - (int64_t)pl.out_stages * pl.out_stage_bytes) / pl.stage_bytes);
        pl.stages = more > kMaxStages ? kMaxStages : more;
        if (pl.stages > want) pl.stages = want;
    }
    int at = pl.stages * pl.stage_bytes;
    pl.off_out = at; at += pl.out_stages * pl.out_stage_bytes;
    pl.off_ids = at; at += (int)ids_ints * 4;
    pl.off_mask = at; at += (int)mask_ints * 4;
    pl.off_bm = at; at += (int)bm_ints * 4;
    pl.off_pos = at; at += chunk_slots * 4;
    pl.off_key = at; at += chunk_slots * 4;
    pl.off_ord = at; at += chunk_slots * 4;
    pl.off_w = at; at += chunk_slots * 4;
    pl.off_hist = at; at += hist_ints * 4;
    pl.off_arr = at; at += p.R * 4;
    pl.off_order = at; at += p.R * 4;
    pl.off_item = at; at += item_ints * 4;
    pl.total = round_up_i(at, 128);
    *out = pl;
    return 0;
}

// Launch that lets the kernel be placed while its predecessor in the stream drains (the
// kernels above call griddep_wait() before they read anything).  `together`: a cooperative
// launch -- the kernel's CTAs wait for flags that other CTAs of the same grid publish, so they
// must all be resident at once; the runtime then refuses a grid that cannot be (a synchronous
// error instead of CTAs spinning until their bounded waits run out) and starts the grid only
// when every CTA has a place.  Such a kernel is not launched ahead of its predecessor's end.
template <typename... KArgs, typename... Args>
static cudaError_t launch_overlapped(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t st,
                                     bool together, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (together) {
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
    } else {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
    }
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

// The dynamic shared-memory limit of a kernel is a sticky attribute: per kernel instance and
// device only a larger request has to reach the runtime (the call costs host time that an
// enqueue-bound caller sees on every dispatch).  `granted` belongs to one kernel instance.
constexpr int kAttrDevices = 64;
static cudaError_t allow_dynamic_smem(const void* kern, int bytes, std::atomic<int>* granted) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool cached = dev >= 0 && dev < kAttrDevices;
    if (cached && granted[dev].load(std::memory_order_relaxed) >= bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && cached) granted[dev].store(bytes, std::memory_order_relaxed);
    return e;
}

template <int kMode, bool kFp8, bool kSteal>
static cudaError_t launch_dispatch_s(const Params& p, const SmemPlan& pl, cudaStream_t st) {
    auto kern = dispatch_kernel<kMode, kFp8, kSteal>;
    static std::atomic<int> granted[kAttrDevices];
    cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(kern), pl.total, granted);
    if (e != cudaSuccess) return e;
    return launch_overlapped(kern, p.grid, kThreads, (size_t)pl.total, st, kMode == kModeFused, p, pl);
}

template <int kMode, bool kFp8>
static cudaError_t launch_dispatch_t(const Params& p, const SmemPlan& pl, cudaStream_t st) {
    if (kMode != kModeLocal && p.steal) return launch_dispatch_s<kMode, kFp8, true>(p, pl, st);
    return launch_dispatch_s<kMode, kFp8, false>(p, pl, st);
}

// TokenCnt and CalCumSum as two launches over the whole routing table (chunk histograms, then per rank
// the prefix over chunks, expert offsets, totals and the per-source tables).
cudaError_t launch_count_scan(const Params& p, const SmemPlan& pl, cudaStream_t st) {
    cudaError_t e;
    const int count_smem = pl.off_pos - pl.off_ids;   // ids + both bitmap arrays
    static std::atomic<int> granted[kAttrDevices];
    if ((e = allow_dynamic_smem(reinterpret_cast<const void*>(count_kernel), count_smem, granted)) != cudaSuccess)
        return e;
    count_kernel<<<p.nchunks, 256, count_smem, st>>>(p, pl);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    scan_kernel<<<p.R, 256, sizeof(int) * (p.L + 1), st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_dispatch(const Params& p, int mode, const SmemPlan& pl, cudaStream_t st, int* launches) {
    cudaError_t e;
    *launches = 1;
    if (mode == kModePhased) {
        if ((e = launch_count_scan(p, pl, st)) != cudaSuccess) return e;
        *launches = 3;
        return p.payload ? launch_dispatch_t<kModePhased, true>(p, pl, st)
                         : launch_dispatch_t<kModePhased, false>(p, pl, st);
    }
    if (mode == kModeLocal)
        return p.payload ? launch_dispatch_t<kModeLocal, true>(p, pl, st)
                         : launch_dispatch_t<kModeLocal, false>(p, pl, st);
    return p.payload ? launch_dispatch_t<kModeFused, true>(p, pl, st)
                     : launch_dispatch_t<kModeFused, false>(p, pl, st);
}

template <int K>
static cudaError_t launch_combine_k(bool ahead, int g, cudaStream_t st, const uint16_t* y, const int32_t* slot_pos,
                                    const float* topk_w, int T, int H, int k, uint16_t* out) {
    if (ahead) return launch_overlapped(combine_kernel<K>, g, 256, 0, st, false, y, slot_pos, topk_w, T, H, k, out);
    combine_kernel<K><<<g, 256, 0, st>>>(y, slot_pos, topk_w, T, H, k, out);
    return cudaGetLastError();
}

// `ahead`: let the kernel be placed while its predecessor in the stream still runs (it waits for the
// predecessor's end before it reads anything).  Worth 0.4 us per layer beside the short decode-sized
// dispatch; beside a long dispatch the parked CTAs were measured to slow it down by far more than the
// launch latency they hide, so the caller asks for it only for small T.
cudaError_t launch_combine(const uint16_t* y, const int32_t* slot_pos, const float* topk_w, int T, int H, int k,
                           uint16_t* out, int num_sms, bool ahead, cudaStream_t st) {
    const int64_t total = (int64_t)T * (H / 8);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)num_sms * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const int g = (int)blocks;
    switch (k) {
        case 1: return launch_combine_k<1>(ahead, g, st, y, slot_pos, topk_w, T, H, k, out);
        case 2: return launch_combine_k<2>(ahead, g, st, y, slot_pos, topk_w, T, H, k, out);
        case 4: return launch_combine_k<4>(ahead, g, st, y, slot_pos, topk_w, T, H, k, out);
        case 8: return launch_combine_k<8>(ahead, g, st, y, slot_pos, topk_w, T, H, k, out);
        default: return launch_combine_k<0>(ahead, g, st, y, slot_pos, topk_w, T, H, k, out);
    }
}

// A kernel that does nothing, one CTA per SM: what a launch costs by itself.
__global__ void __launch_bounds__(32) empty_kernel(int) {
    griddep_launch();
    griddep_wait();
}

cudaError_t launch_empty(int num_sms, bool ahead, cudaStream_t st) {
    if (ahead) return launch_overlapped(empty_kernel, num_sms, 32, 0, st, false, 0);
    empty_kernel<<<num_sms, 32, 0, st>>>(0);
    return cudaGetLastError();
}

cudaError_t launch_layout(const Params& p, int32_t* num_tokens_per_rank, int32_t* num_tokens_per_expert,
                          uint8_t* is_token_in_rank, int32_t* scratch_hist, unsigned* ticket, cudaStream_t st) {
    layout_kernel<<<p.nchunks, 256, sizeof(int) * p.B, st>>>(p, num_tokens_per_rank, num_tokens_per_expert,
                                                             is_token_in_rank, scratch_hist, ticket);
    return cudaGetLastError();
}

}  // namespace ubep
