// Layout steps of dispatch as device functions: TokenCnt (stage_ids + count_slots),
// CalCumSum (scan_rank, or local_layout when every CTA derives it from the whole routing
// table) and slot -> row assignment (finalize_chunk).  They are shared by the three-launch
// pipeline, where kernel boundaries order them, and by the persistent kernel, where
// readiness flags do (Sec. 3.2 of the paper: kernel decomposition).
#pragma once

#include "ubep_common.cuh"

namespace ubep {

// Physical expert of slot (t, j): logical id -> phys[l][t mod ncopies[l]] when a replica
// table is set.  -1 for an empty slot; ids out of range are reported and treated as empty.
__device__ __forceinline__ int resolve_expert(const Params& p, int t, int raw) {
    if (raw == -1) return -1;
    int e = raw;
    if (p.phys != nullptr) {
        if (raw < 0 || raw >= p.E_log) { report(p.status, kErrBadIndex); return -1; }
        int nc = __ldg(p.ncopies + raw);
        if (nc < 1 || nc > p.C) { report(p.status, kErrBadIndex); return -1; }
        e = __ldg(p.phys + (size_t)raw * p.C + (t % nc));
    }
    if (e < 0 || e >= p.E) { report(p.status, kErrBadIndex); return -1; }
    return e;
}

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
    }
    return v;
}

// Resolved expert ids of tokens [t0, t1) into shared memory, one coalesced pass.
__device__ __forceinline__ void stage_ids(const Params& p, int t0, int t1, int* ids, int tid, int nthreads) {
    const int k = p.k, n = (t1 - t0) * k;
    const int32_t* src = p.topk_idx + (size_t)t0 * k;
    for (int i = tid; i < n; i += nthreads) ids[i] = resolve_expert(p, t0 + i / k, __ldg(src + i));
}

// ------------------------------------------------------------------- TokenCnt
// One warp walks the slots of tokens [t0, t1) in token order (ids staged in shared memory,
// index 0 = slot (t0, 0)).  For every slot it records how many earlier slots of the range
// chose the same expert (loc_e) and, for the first slot a token has on a rank, how many
// earlier tokens of the range visit that rank (loc_r; later slots of the token on that rank
// copy it).  hist[B] receives the range's histogram.  When `partial` is given, the running
// histogram is also written out at every source-rank boundary inside the range.  Equal ids
// inside a batch of 32 slots are ranked with match_any / popc.
__device__ void count_slots(const Params& p, int t0, int t1, const int* ids, int* hist, int* loc_e, int* loc_r,
                            int32_t* partial, int lane) {
    const int T = p.T, k = p.k, B = p.B, S = p.S;
    for (int b = lane; b < B; b += 32) hist[b] = 0;
    __syncwarp();
    const int tpb = 32 / k;  // whole tokens per batch
    int s_next = partial ? (int)(((int64_t)t0 * S + T - 1) / T) : S;  // smallest s with src_begin(s) >= t0
    const unsigned lt = (1u << lane) - 1u;
    const int tok = lane / k, j = lane - tok * k;
    const int base_lane = lane - j;
    int t = t0;
    while (true) {
        while (t < t1 && s_next < S && src_begin(s_next, T, S) == t) {
            for (int b = lane; b < B; b += 32) partial[(size_t)s_next * B + b] = hist[b];
            ++s_next;
        }
        if (t >= t1) break;
        int lim = t1;
        if (s_next < S) lim = min(lim, src_begin(s_next, T, S));
        const int nb = min(tpb, lim - t);
        const bool active = lane < nb * k;
        const int li = (t - t0 + tok) * k + j;
        const int e = active ? ids[li] : -1;
        const int r = e >= 0 ? e / p.L : -1;
        // is this the first slot of its token on rank r?
        bool first = e >= 0;
        int jf = j;
        for (int jj = 0; jj < k; ++jj) {
            int rr = __shfl_sync(0xffffffffu, r, min(base_lane + jj, 31));
            if (jj < j && first && rr == r) { first = false; jf = jj; }
        }
        // expert bins
        unsigned m = __match_any_sync(0xffffffffu, e >= 0 ? (unsigned)e : (0x40000000u | lane));
        int le = -1;
        if (e >= 0) le = hist[e] + __popc(m & lt);
        __syncwarp();
        if (e >= 0 && (m & lt) == 0) hist[e] += __popc(m);
        // rank bins, first slots only
        unsigned m2 = __match_any_sync(0xffffffffu, first ? (unsigned)r : (0x40000000u | lane));
        int lr = -1;
        if (first) lr = hist[p.E + r] + __popc(m2 & lt);
        __syncwarp();
        if (first && (m2 & lt) == 0) hist[p.E + r] += __popc(m2);
        __syncwarp();
        int lr_first = __shfl_sync(0xffffffffu, lr, min(base_lane + jf, 31));
        if (e >= 0 && !first) lr = lr_first;
        if (active) {
            loc_e[li] = le;
            loc_r[li] = first ? lr : (e >= 0 ? -2 - lr : -1);  // later slots on a rank: -2 - row
        }
        t += nb;
    }
    __syncwarp();
}

// loc_r encoding: >= 0 first slot of its token on that rank (value = local row count);
// <= -2 a later slot sharing the row -2 - value; -1 empty slot.
__device__ __forceinline__ bool locr_first(int v) { return v >= 0; }
__device__ __forceinline__ int locr_value(int v) { return v >= 0 ? v : -2 - v; }

// ------------------------------------------------------------------ CalCumSum
// Prefix sums for the bins of rank r (its L experts and its rank bin), run by a group of
// nw warps that share barrier `bar_id`.  One pass over the chunk histograms gives, per bin,
// the exclusive prefix over chunks (chunk_base) and the total; the expert offsets inside
// the region follow from the totals.  `sm` holds L + 1 ints.  Inputs written by other CTAs
// are read past L1 (__ldcg).  scan_rank_publish must complete before the rank's readiness
// flag is released; scan_rank_sources only fills cnt / src_offset, which no mover needs.
__device__ void scan_rank_publish(const Params& p, int r, int* sm, int gw, int nw, int lane, int bar_id) {
    const int n = p.nchunks, L = p.L, B = p.B, E = p.E;
    const int nb = L + 1;
    for (int bi = gw; bi < nb; bi += nw) {
        const int bin = bi < L ? r * L + bi : E + r;
        int carry = 0;
        for (int c0 = 0; c0 < n; c0 += 32) {
            const int c = c0 + lane;
            const int v = c < n ? __ldcg(p.chunk_hist + (size_t)c * B + bin) : 0;
            const int incl = warp_incl_scan(v, lane);
            if (c < n) p.chunk_base[(size_t)c * B + bin] = carry + incl - v;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) sm[bi] = carry;
    }
    group_sync(bar_id, nw * 32);
    if (gw == 0) {
        // exclusive scan of the L expert totals (L may exceed 32)
        int run = 0;
        for (int i0 = 0; i0 < L; i0 += 32) {
            const int i = i0 + lane;
            const int v = i < L ? sm[i] : 0;
            const int incl = warp_incl_scan(v, lane);
            if (i < L) {
                p.expert_offset[r * L + i] = run + incl - v;
                p.num_tokens_per_expert[r * L + i] = v;
            }
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            p.num_tokens_per_rank[r] = sm[L];
            p.num_rows_per_rank[r] = p.dedup ? sm[L] : run;
        }
    }
    group_sync(bar_id, nw * 32);
}

__device__ void scan_rank_sources(const Params& p, int r, const int* sm, int gtid, int gn) {
    // tokens before each source boundary = chunk prefix + running histogram at the boundary
    const int n = p.nchunks, L = p.L, B = p.B, T = p.T, S = p.S, E = p.E;
    for (int i = gtid; i < S * L; i += gn) {
        const int s = i / L, bi = i - s * L, bin = r * L + bi;
        const int eo = __ldcg(p.expert_offset + bin);
        const int b0 = src_begin(s, T, S);
        const int pre0 = __ldcg(p.chunk_base + (size_t)chunk_of(b0, T, n) * B + bin) +
                         __ldcg(p.partial + (size_t)s * B + bin);
        int pre1 = sm[bi];
        if (s + 1 < S) {
            const int b1 = src_begin(s + 1, T, S);
            pre1 = __ldcg(p.chunk_base + (size_t)chunk_of(b1, T, n) * B + bin) +
                   __ldcg(p.partial + (size_t)(s + 1) * B + bin);
        }
        p.src_offset[(size_t)s * E + bin] = eo + pre0;
        p.cnt[(size_t)s * E + bin] = pre1 - pre0;
    }
}

// ------------------------------------------------ CalCumSum without communication
// Every CTA histograms the whole routing table (ids of all T tokens staged in shared
// memory): tot[B] over all tokens, pre[B] over tokens before t0.  CTA `duty_s` (< S) also
// gets the per-source numbers of source rank duty_s: spre (tokens before its first token)
// and scnt (its own tokens), expert bins only.  Run by gn threads between barriers.
__device__ void local_histograms(const Params& p, const int* ids, int t0, int duty_s, int* tot, int* pre, int* spre,
                                 int* scnt, int gtid, int gn) {
    const int k = p.k, L = p.L, E = p.E, T = p.T;
    const int b0 = duty_s >= 0 ? src_begin(duty_s, T, p.S) : 0;
    const int b1 = duty_s >= 0 ? src_begin(duty_s + 1, T, p.S) : 0;
    for (int t = gtid; t < T; t += gn) {
        const int* row = ids + (size_t)t * k;
        const bool before = t < t0;
        for (int j = 0; j < k; ++j) {
            const int e = row[j];
            if (e < 0) continue;
            const int r = e / L;
            bool first = true;
            for (int jj = 0; jj < j; ++jj) {
                const int e2 = row[jj];
                if (e2 >= 0 && e2 / L == r) { first = false; break; }
            }
            atomicAdd(&tot[e], 1);
            if (before) atomicAdd(&pre[e], 1);
            if (first) {
                atomicAdd(&tot[E + r], 1);
                if (before) atomicAdd(&pre[E + r], 1);
            }
            if (duty_s >= 0) {
                if (t < b0) atomicAdd(&spre[e], 1);
                else if (t < b1) atomicAdd(&scnt[e], 1);
            }
        }
    }
}

// -------------------------------------------------------- slot -> row assignment
// Turns the range-local counts of this CTA's tokens [t0, t1) into final rows.  base_e(e) /
// base_r(r) give the rows taken by earlier tokens (plus the expert's offset in its region).
// Writes slot_row / slot_pos, the per-row metadata (only when `write_meta`; with column
// parts one CTA of the group does it) and leaves in pos[] the global row to copy to
// (rank * cap + row), or -1.  arr[r] counts the rows this CTA sends to rank r.
template <typename BaseE, typename BaseR>
__device__ void finalize_chunk(const Params& p, int t0, int t1, const int* ids, const int* loc_e, const int* loc_r,
                               BaseE base_e, BaseR base_r, bool write_meta, int* pos, int* arr, int gtid, int gn) {
    const int k = p.k, L = p.L;
    const int nslots = (t1 - t0) * k;
    for (int li = gtid; li < nslots; li += gn) {
        const int t = t0 + li / k;
        const size_t i = (size_t)t0 * k + li;
        const int e = ids[li];
        int where = -1, row = -1, gpos = -1;
        if (e >= 0) {
            const int r = e / L;
            const bool first = !p.dedup || locr_first(loc_r[li]);
            if (!p.dedup) {
                row = base_e(e) + loc_e[li];
            } else {
                row = base_r(r) + locr_value(loc_r[li]);
                if (write_meta) {
                    const int at = base_e(e) + loc_e[li];
                    if (at < p.er_cap) p.expert_rows[(size_t)r * p.er_cap + at] = row;
                    else report(p.status, kErrCapacity);
                }
            }
            if (row >= p.cap) {
                report(p.status, kErrCapacity);
            } else {
                gpos = r * p.cap + row;
                if (first) {
                    where = gpos;
                    atomicAdd(&arr[r], 1);
                    if (write_meta) {
                        p.recv_src_idx[where] = t;
                        if (!p.dedup) {
                            p.recv_weight[where] = __ldg(p.topk_w + i);
                        } else {
                            const int* row_ids = ids + (li / k) * k;
                            for (int jj = 0; jj < k; ++jj) {
                                const int e2 = row_ids[jj];
                                const bool here = e2 >= 0 && e2 / L == r;
                                p.recv_topk_idx[(size_t)where * k + jj] = here ? e2 % L : -1;
                                p.recv_topk_w[(size_t)where * k + jj] =
                                    here ? __ldg(p.topk_w + (size_t)t * k + jj) : 0.0f;
                            }
                        }
                    }
                }
            }
        }
        if (write_meta) {
            p.slot_row[i] = row;
            p.slot_pos[i] = gpos;
        }
        pos[li] = where;
    }
}

// Per token, put the destinations into the order of the destination-ordering table rotated
// by the worker id (Sec. 3.3: each worker visits a re-mapped destination sequence).  Only
// the issue order of the copies changes.  order_sm[R] is the table in shared memory.  One
// thread per token, insertion sort on <= 32 keys.
__device__ void order_destinations(const Params& p, int worker, const int* order_sm, int* pos, int ntok, int gtid,
                                   int gn) {
    const int k = p.k, R = p.R;
    const int rot = worker % R;
    for (int n = gtid; n < ntok; n += gn) {
        int* q = pos + n * k;
        int m = 0;
        for (int j = 0; j < k; ++j)
            if (q[j] >= 0) q[m++] = q[j];
        for (int j = m; j < k; ++j) q[j] = -1;
        for (int a = 1; a < m; ++a) {
            const int v = q[a];
            int kv = order_sm[v / p.cap] - rot;
            kv += kv < 0 ? R : 0;
            int b = a - 1;
            while (b >= 0) {
                int kb = order_sm[q[b] / p.cap] - rot;
                kb += kb < 0 ? R : 0;
                if (kb <= kv) break;
                q[b + 1] = q[b];
                --b;
            }
            q[b + 1] = v;
        }
    }
}

}  // namespace ubep
