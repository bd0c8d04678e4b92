// Layout steps of dispatch as device functions: TokenCnt (count_chunk), CalCumSum
// (scan_rank) and slot -> row assignment (finalize_chunk).  They are shared by the
// three-launch pipeline, where kernel boundaries order them, and by the persistent
// kernel, where readiness flags do (Sec. 3.2 of the paper: kernel decomposition).
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

// ------------------------------------------------------------------- TokenCnt
// One warp walks the slots of chunk c in token order.  For every slot it records how many
// earlier slots of the chunk chose the same expert (and, for the first slot a token has on
// a rank, how many earlier tokens of the chunk visit that rank); the chunk histogram goes
// to chunk_hist[c], and its running value at every source-rank boundary inside the chunk
// to partial[s].  Equal ids inside a batch of 32 slots are ranked with match_any / popc.
__device__ void count_chunk(const Params& p, int c, int* hist, int lane) {
    const int T = p.T, k = p.k, B = p.B, S = p.S;
    const int t0 = (int)chunk_begin(c, T, p.nchunks), t1 = (int)chunk_begin(c + 1, T, p.nchunks);
    for (int b = lane; b < B; b += 32) hist[b] = 0;
    __syncwarp();
    const int tpb = 32 / k;                       // whole tokens per batch
    int s_next = (int)(((int64_t)t0 * S + T - 1) / T);  // smallest s with src_begin(s) >= t0
    const unsigned lt = (1u << lane) - 1u;
    int t = t0;
    while (true) {
        while (t < t1 && s_next < S && src_begin(s_next, T, S) == t) {
            for (int b = lane; b < B; b += 32) p.partial[(size_t)s_next * B + b] = hist[b];
            ++s_next;
        }
        if (t >= t1) break;
        int lim = t1;
        if (s_next < S) lim = min(lim, src_begin(s_next, T, S));
        const int nb = min(tpb, lim - t);
        const int tok = lane / k, j = lane - tok * k;
        const bool active = lane < nb * k;
        const int tt = t + tok;
        int e = -1;
        if (active) e = resolve_expert(p, tt, __ldg(p.topk_idx + (size_t)tt * k + j));
        const int r = e >= 0 ? e / p.L : -1;
        // is this the first slot of its token on rank r?
        bool first = e >= 0;
        int jf = j;
        const int base_lane = lane - j;
        for (int jj = 0; jj < k; ++jj) {
            int rr = __shfl_sync(0xffffffffu, r, min(base_lane + jj, 31));
            if (jj < j && first && rr == r) { first = false; jf = jj; }
        }
        // expert bins
        unsigned m = __match_any_sync(0xffffffffu, e >= 0 ? (unsigned)e : (0x40000000u | lane));
        int loc_e = -1;
        if (e >= 0) loc_e = hist[e] + __popc(m & lt);
        __syncwarp();
        if (e >= 0 && (m & lt) == 0) hist[e] += __popc(m);
        // rank bins, first slots only
        unsigned m2 = __match_any_sync(0xffffffffu, first ? (unsigned)r : (0x40000000u | lane));
        int loc_r = -1;
        if (first) loc_r = hist[p.E + r] + __popc(m2 & lt);
        __syncwarp();
        if (first && (m2 & lt) == 0) hist[p.E + r] += __popc(m2);
        __syncwarp();
        int lr_first = __shfl_sync(0xffffffffu, loc_r, min(base_lane + jf, 31));
        if (e >= 0 && !first) loc_r = lr_first;
        if (active) {
            size_t i = (size_t)tt * k + j;
            if (!p.dedup) {
                p.slot_row[i] = loc_e;
            } else {
                p.slot_row[i] = loc_r;
                p.slot_aux[i] = loc_e;
            }
        }
        t += nb;
    }
    __syncwarp();
    for (int b = lane; b < B; b += 32) p.chunk_hist[(size_t)c * B + b] = hist[b];
}

// ------------------------------------------------------------------ CalCumSum
// Prefix sums for the bins of rank r (its L experts and its rank bin), run by a group of
// nw warps that share barrier `bar_id`: totals, expert offsets inside the region, the base
// of every bin for every chunk, and the per-source counts and offsets.  `sm` holds L + 1
// ints.  Inputs written by other CTAs are read past L1 (__ldcg).
__device__ void scan_rank(const Params& p, int r, int* sm, int gw, int nw, int lane, int bar_id) {
    const int n = p.nchunks, L = p.L, B = p.B, T = p.T, S = p.S, E = p.E;
    const int nb = L + 1;
    for (int bi = gw; bi < nb; bi += nw) {
        const int bin = bi < L ? r * L + bi : E + r;
        int sum = 0;
        for (int c = lane; c < n; c += 32) sum += __ldcg(p.chunk_hist + (size_t)c * B + bin);
        sum = warp_sum(sum);
        if (lane == 0) sm[bi] = sum;
    }
    group_sync(bar_id, nw * 32);
    if (gw == 0) {
        int rows = 0;
        if (p.dedup) {
            rows = sm[L];
        } else {
            for (int i = lane; i < L; i += 32) rows += sm[i];
            rows = warp_sum(rows);
        }
        if (lane == 0) p.num_rows_per_rank[r] = rows;
    }
    for (int bi = gw; bi < nb; bi += nw) {
        const int bin = bi < L ? r * L + bi : E + r;
        int eo = 0;
        if (bi < L) {
            for (int i = lane; i < bi; i += 32) eo += sm[i];
            eo = warp_sum(eo);
        }
        const int tot = sm[bi];
        int carry = 0;
        for (int c0 = 0; c0 < n; c0 += 32) {
            const int c = c0 + lane;
            const int v = c < n ? __ldcg(p.chunk_hist + (size_t)c * B + bin) : 0;
            const int incl = warp_incl_scan(v, lane);
            if (c < n) p.chunk_base[(size_t)c * B + bin] = eo + carry + incl - v;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            if (bi < L) {
                p.expert_offset[bin] = eo;
                p.num_tokens_per_expert[bin] = tot;
            } else {
                p.num_tokens_per_rank[r] = tot;
            }
        }
        __syncwarp();
        if (bi < L) {
            // count of tokens before each source boundary = chunk prefix + running histogram
            for (int s = lane; s < S; s += 32) {
                const int b0 = src_begin(s, T, S);
                const int pre0 = __ldcg(p.chunk_base + (size_t)chunk_of(b0, T, n) * B + bin) - eo +
                                 __ldcg(p.partial + (size_t)s * B + bin);
                int pre1 = tot;
                if (s + 1 < S) {
                    const int b1 = src_begin(s + 1, T, S);
                    pre1 = __ldcg(p.chunk_base + (size_t)chunk_of(b1, T, n) * B + bin) - eo +
                           __ldcg(p.partial + (size_t)(s + 1) * B + bin);
                }
                p.src_offset[(size_t)s * E + bin] = eo + pre0;
                p.cnt[(size_t)s * E + bin] = pre1 - pre0;
            }
        }
    }
}

// -------------------------------------------------------- slot -> row assignment
// Turns the chunk-local counts of chunk c into final rows, writes the per-row metadata and
// leaves, for every slot of the chunk, the global row (rank * cap + row) to copy to in
// pos[] (-1: nothing to copy).  arr[r] counts the rows this chunk sends to rank r.
// Run by `gn` threads (gtid = 0..gn-1) after chunk_base is known.
__device__ void finalize_chunk(const Params& p, int c, int* pos, int* arr, int gtid, int gn) {
    const int k = p.k, B = p.B, L = p.L;
    const int t0 = (int)chunk_begin(c, p.T, p.nchunks), t1 = (int)chunk_begin(c + 1, p.T, p.nchunks);
    const int nslots = (t1 - t0) * k;
    const int32_t* base = p.chunk_base + (size_t)c * B;
    for (int li = gtid; li < nslots; li += gn) {
        const int t = t0 + li / k, j = li % k;
        const size_t i = (size_t)t0 * k + li;
        const int e = resolve_expert(p, t, __ldg(p.topk_idx + i));
        int where = -1;
        if (e < 0) {
            p.slot_row[i] = -1;
            p.slot_pos[i] = -1;
        } else {
            const int r = e / L;
            bool first = true;
            if (p.dedup)
                for (int jj = 0; jj < j; ++jj) {
                    int e2 = resolve_expert(p, t, __ldg(p.topk_idx + (size_t)t * k + jj));
                    if (e2 >= 0 && e2 / L == r) { first = false; break; }
                }
            int row;
            if (!p.dedup) {
                row = __ldcg(base + e) + p.slot_row[i];
            } else {
                row = __ldcg(base + p.E + r) + p.slot_row[i];
                const int at = __ldcg(base + e) + p.slot_aux[i];
                if (at < p.er_cap) p.expert_rows[(size_t)r * p.er_cap + at] = row;
                else report(p.status, kErrCapacity);
            }
            p.slot_row[i] = row;
            p.slot_pos[i] = row < p.cap ? r * p.cap + row : -1;
            if (row >= p.cap) {
                report(p.status, kErrCapacity);
            } else if (first) {
                where = r * p.cap + row;
                p.recv_src_idx[where] = t;
                if (!p.dedup) {
                    p.recv_weight[where] = __ldg(p.topk_w + i);
                } else {
                    for (int jj = 0; jj < k; ++jj) {
                        int e2 = resolve_expert(p, t, __ldg(p.topk_idx + (size_t)t * k + jj));
                        bool here = e2 >= 0 && e2 / L == r;
                        p.recv_topk_idx[(size_t)where * k + jj] = here ? e2 % L : -1;
                        p.recv_topk_w[(size_t)where * k + jj] = here ? __ldg(p.topk_w + (size_t)t * k + jj) : 0.0f;
                    }
                }
                atomicAdd(&arr[r], 1);
            }
        }
        pos[li] = where;
    }
}

// Per token, put the destinations into the order of the destination-ordering table rotated
// by the worker id (Sec. 3.3: each worker visits a re-mapped destination sequence).  Only
// the issue order of the copies changes.  One thread per token, insertion sort on <= 32 keys.
__device__ void order_destinations(const Params& p, int c, int* pos, int ntok, int gtid, int gn) {
    const int k = p.k, R = p.R;
    const int rot = c % R;
    for (int n = gtid; n < ntok; n += gn) {
        int* q = pos + n * k;
        int m = 0;
        for (int j = 0; j < k; ++j)
            if (q[j] >= 0) q[m++] = q[j];
        for (int j = m; j < k; ++j) q[j] = -1;
        for (int a = 1; a < m; ++a) {
            const int v = q[a];
            const int kv = (__ldg(p.order_pos + v / p.cap) - rot + R) % R;
            int b = a - 1;
            while (b >= 0 && (__ldg(p.order_pos + q[b] / p.cap) - rot + R) % R > kv) {
                q[b + 1] = q[b];
                --b;
            }
            q[b + 1] = v;
        }
    }
}

}  // namespace ubep
