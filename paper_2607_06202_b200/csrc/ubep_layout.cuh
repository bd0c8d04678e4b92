// Layout steps of dispatch as device functions: TokenCnt (stage_ids + build_bin_maps),
// CalCumSum (scan_rank_*, or bit counts over the whole routing table when every CTA derives
// it alone) and slot -> row assignment (finalize_chunk).  They are shared by the three-launch
// pipeline, where kernel boundaries order them, and by the persistent kernel, where
// readiness flags do (Sec. 3.2 of the paper: kernel decomposition).
#pragma once

#include "ubep_common.cuh"

namespace ubep {

// (The functions that are not forced inline have internal linkage: more than one source
// file includes this header.)

// Physical expert of slot (t, j): logical id -> phys[l][t mod ncopies[l]] when a replica
// table is set.  -1 for an empty slot; ids out of range are reported and treated as empty.
// v / L for 0 <= v < 65536, with magic = ceil(2^32 / L)
__device__ __forceinline__ int fast_div(int v, unsigned magic) { return (int)__umulhi((unsigned)v, magic); }

// `bad` is set instead of reporting on the spot: a call to the out-of-line report() inside an unrolled loop,
// taken or not, was measured to cost about 125 cycles per slot (the staging of a 512-token table: 1865
// cycles per warp with the calls, 840 without).  The caller reports once, after its loop.
__device__ __forceinline__ int resolve_expert(const Params& p, int t, int raw, bool& bad) {
    if (raw == -1) return -1;
    int e = raw;
    if (p.phys != nullptr) {
        if (raw < 0 || raw >= p.E_log) { bad = true; return -1; }
        int nc = __ldg(p.ncopies + raw);
        if (nc < 1 || nc > p.C) { bad = true; return -1; }
        e = __ldg(p.phys + (size_t)raw * p.C + (t % nc));
    }
    if (e < 0 || e >= p.E) { bad = true; return -1; }
    return e;
}
__device__ __forceinline__ int resolve_expert(const Params& p, int t, int raw) {
    bool bad = false;
    const int e = resolve_expert(p, t, raw, bad);
    if (bad) report(p.status, kErrBadIndex);
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

// Staged slot: physical expert id in the low 16 bits, its rank above; -1 = empty slot.
__device__ __forceinline__ int slot_expert(int v) { return v & 0xffff; }
__device__ __forceinline__ int slot_rank(int v) { return v >> 16; }

// Place of a rank in the destination-ordering table rotated by the worker id.
__device__ __forceinline__ int rotated_key(const int* order_sm, int r, int worker, int R) {
    int kv = order_sm[r] - worker % R;
    return kv < 0 ? kv + R : kv;
}

// One slot of the routing table, resolved and packed (expert | rank << 16), -1 for an empty slot or a bad
// id (`bad` is set then).  `slot` is its index in the whole table; the token it belongs to is worked out
// only where a replica has to be picked, and nothing branches per slot without a replica table: a lone
// warp staging four slots per thread spent 1300 cycles on the divisions and branches of the earlier form.
__device__ __forceinline__ int pack_slot(const Params& p, size_t slot, int raw, bool& bad) {
    int e = raw;
    if (p.phys != nullptr) {
        const bool in = (unsigned)e < (unsigned)p.E_log;
        bad |= !in && e != -1;
        const int nc = in ? __ldg(p.ncopies + e) : 1;
        const bool okc = in && nc >= 1 && nc <= p.C;
        bad |= in && !okc;
        const int t = (int)((unsigned)slot / (unsigned)p.k);   // (the table has fewer than 2^31 slots)
        e = okc ? __ldg(p.phys + (size_t)e * p.C + (t % nc)) : -1;
        bad |= okc && e < 0;
    }
    const bool valid = (unsigned)e < (unsigned)p.E;
    bad |= !valid && e != -1;
    const int r = p.L == 1 ? e : fast_div(e, p.L_magic);
    return valid ? (e | (r << 16)) : -1;
}

// Resolved expert ids (with their ranks) of tokens [t0, t1) into shared memory.  The raw ids
// are gathered several at a time before any of them is resolved, so that the loads overlap.
__device__ __forceinline__ void stage_ids(const Params& p, int t0, int t1, int* ids, int tid, int nthreads) {
    const int k = p.k, n = (t1 - t0) * k;
    const size_t slot0 = (size_t)t0 * k;
    const int32_t* src = p.topk_idx + slot0;
    bool bad = false;
    if ((slot0 & 3) == 0 && (n & 3) == 0) {
        // 16-byte loads and stores, four of them in flight per thread
        const int4* src4 = reinterpret_cast<const int4*>(src);
        const int n4 = n >> 2;
        for (int i0 = tid; i0 < n4; i0 += 4 * nthreads) {
            int4 raw[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * nthreads;
                raw[u] = i < n4 ? __ldg(src4 + i) : make_int4(-1, -1, -1, -1);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * nthreads;
                if (i < n4) {
                    const size_t s4 = slot0 + 4 * (size_t)i;
                    *reinterpret_cast<int4*>(ids + 4 * i) =
                        make_int4(pack_slot(p, s4, raw[u].x, bad), pack_slot(p, s4 + 1, raw[u].y, bad),
                                  pack_slot(p, s4 + 2, raw[u].z, bad), pack_slot(p, s4 + 3, raw[u].w, bad));
                }
            }
        }
    } else {
        for (int i0 = tid; i0 < n; i0 += 8 * nthreads) {
            int raw[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * nthreads;
                raw[u] = i < n ? __ldg(src + i) : -1;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * nthreads;
                if (i < n) ids[i] = pack_slot(p, slot0 + i, raw[u], bad);
            }
        }
    }
    if (bad) report(p.status, kErrBadIndex);
}

// ------------------------------------------------------------------- TokenCnt
// Counting without ordered atomics: for a range of tokens, every bin (E expert bins then R
// rank bins) gets a bitmap with one bit per token of the range.  A token selects an expert
// at most once, so "how many earlier tokens of the range chose this bin" -- the stable rank
// the row placement needs -- is a population count of the bits below the token, and the
// range's histogram is the population count of all bits.
//
// Built per group of 32 tokens and word of 32 bins: each lane ORs the bins of its own token
// into a register, then the warp transposes the 32x32 bit tile (lane = token, bit = bin ->
// lane = bin, bit = token) with five shuffle steps and stores it bin-major (bm).
struct BinMaps {
    unsigned* mask_t;  // [groups * 32] scratch words (duty bitmaps of the flag-free kernel)
    unsigned* bm;      // [groups, bp] bit (token & 31) of word [token >> 5][bin]
    int wb;            // words per token row that carry bins: ceil(B / 32)
    int bp;            // bins padded to a multiple of 32
    int groups;        // 32-token groups of the range
};

__device__ __forceinline__ unsigned transpose32(unsigned x, int lane) {
    unsigned m = 0x0000ffffu;
#pragma unroll
    for (int j = 16; j != 0; j >>= 1) {
        const unsigned y = __shfl_xor_sync(0xffffffffu, x, j);
        if ((lane & j) == 0) x ^= ((((x >> j) ^ y) & m) << j);
        else x ^= (((y >> j) ^ x) & m);
        m ^= m << (j >> 1);
    }
    return x;  // bit b of lane i before == bit i of lane b after
}

// ids: staged slots of the range (index 0 = first token's slot 0); run by nw warps.  One unit
// of work = one 32-token group x one 32-bin word: the lane (= token) collects the bins of
// that word its token selected, the warp transposes the tile and stores it bin-major.
// With many units per warp (a whole routing table) a unit covers four words instead: the token's
// slots are read once and sorted into four registers, which costs a third of the instructions.
//
// A token may name an expert once.  A second slot with the same expert finds the expert's bit
// already set: it is reported (kErrBadIndex) and its staged id is overwritten with -1, so that
// every later step treats it as an empty slot.  (Warps working on other words of the same tokens
// may still read the old value meanwhile; they only take the rank bit from it, which the first
// occurrence sets as well.)
static __device__ void build_bin_maps(const Params& p, int* ids, int ntok, const BinMaps& bmaps, int gw, int nw,
                               int lane) {
    const int k = p.k;
    const int units = bmaps.groups * bmaps.wb;
    if (units > 2 * nw) {
        const int blocks = (bmaps.wb + 3) / 4;
        for (int u = gw; u < bmaps.groups * blocks; u += nw) {
            const int g = u / blocks, w0 = (u - g * blocks) * 4;
            const int tl = g * 32 + lane;
            unsigned m[4] = {0u, 0u, 0u, 0u};
            if (tl < ntok) {
                for (int j = 0; j < k; ++j) {
                    const int v = ids[tl * k + j];
                    if (v < 0) continue;
                    const int e = slot_expert(v), rb = p.E + slot_rank(v);
                    const int we = (e >> 5) - w0, wr = (rb >> 5) - w0;
                    const unsigned be = 1u << (e & 31), br = 1u << (rb & 31);
                    bool dup = false;
#pragma unroll
                    for (int q = 0; q < 4; ++q) dup = dup || (we == q && (m[q] & be) != 0u);
                    if (dup) {
                        report(p.status, kErrBadIndex);
                        ids[tl * k + j] = -1;
                        continue;
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) m[q] |= (we == q ? be : 0u) | (wr == q ? br : 0u);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (w0 + q < bmaps.wb) bmaps.bm[(size_t)g * bmaps.bp + (w0 + q) * 32 + lane] = transpose32(m[q], lane);
        }
        return;
    }
    for (int u = gw; u < units; u += nw) {
        const int g = u / bmaps.wb, w = u - g * bmaps.wb;
        const int tl = g * 32 + lane;
        unsigned m = 0u;
        if (tl < ntok) {
            for (int j = 0; j < k; ++j) {
                const int v = ids[tl * k + j];
                if (v < 0) continue;
                const int e = slot_expert(v), rb = p.E + slot_rank(v);
                const unsigned be = (e >> 5) == w ? 1u << (e & 31) : 0u;
                if (m & be) {
                    report(p.status, kErrBadIndex);
                    ids[tl * k + j] = -1;
                    continue;
                }
                m |= be | ((rb >> 5) == w ? 1u << (rb & 31) : 0u);
            }
        }
        bmaps.bm[(size_t)g * bmaps.bp + w * 32 + lane] = transpose32(m, lane);
    }
}

// Tokens with local index in [lo, hi) that selected `bin`.
__device__ __forceinline__ int bits_in_range(const BinMaps& bmaps, int bin, int lo, int hi) {
    if (hi <= lo) return 0;
    const int g0 = lo >> 5, g1 = (hi - 1) >> 5;
    int c = 0;
    for (int g = g0; g <= g1; ++g) {
        unsigned w = bmaps.bm[(size_t)g * bmaps.bp + bin];
        if (g == g0) w &= 0xffffffffu << (lo & 31);
        if (g == g1 && (hi & 31) != 0) w &= (1u << (hi & 31)) - 1u;
        c += __popc(w);
    }
    return c;
}

// Chunk histogram and its running value at the source-rank boundaries inside the chunk
// (tokens [t0, t1), bitmaps over the chunk), written to chunk_hist[ch] and partial[s].
static __device__ void publish_chunk_counts(const Params& p, int ch, int t0, int t1, const BinMaps& bmaps, int gtid,
                                     int gn) {
    const int T = p.T, S = p.S, B = p.B;
    const int s_lo = (int)(((int64_t)t0 * S + T - 1) / T);  // smallest s with src_begin(s) >= t0
    int nbnd = 0, bnd[4];                                    // boundaries inside the chunk (first four cached)
    for (int s = s_lo; s < S; ++s) {
        const int bs = src_begin(s, T, S);
        if (bs >= t1) break;
        if (nbnd < 4) bnd[nbnd] = bs;
        ++nbnd;
    }
    for (int b = gtid; b < B; b += gn) {
        p.chunk_hist[(size_t)b * p.nchunks + ch] = bits_in_range(bmaps, b, 0, t1 - t0);   // [bin][chunk]
        for (int q = 0; q < nbnd; ++q) {
            const int bs = q < 4 ? bnd[q] : src_begin(s_lo + q, T, S);
            p.partial[(size_t)(s_lo + q) * B + b] = bits_in_range(bmaps, b, 0, bs - t0);
        }
    }
}

// ------------------------------------------------------------------ CalCumSum
// Prefix sums for the bins of rank r (its L experts and its rank bin), run by a group of
// nw warps that share barrier `bar_id`.  One pass over the chunk histograms gives, per bin,
// the exclusive prefix over chunks (chunk_base) and the total; the expert offsets inside
// the region follow from the totals.  chunk_hist and chunk_base are stored [bin][chunk], so the
// chunks of a bin -- what this step reads and writes, with all CTAs waiting for it -- lie side
// by side.  `sm` holds L + 1 ints.  Inputs written by other CTAs
// are read past L1 (__ldcg).  scan_rank_publish must complete before the rank's readiness
// flag is released; scan_rank_sources only fills cnt / src_offset, which no mover needs.
static __device__ void scan_rank_publish(const Params& p, int r, int* sm, int gw, int nw, int lane, int bar_id) {
    const int n = p.nchunks, L = p.L, E = p.E;
    const int nb = L + 1;
    for (int bi = gw; bi < nb; bi += nw) {
        const int bin = bi < L ? r * L + bi : E + r;
        // lane l owns the `per` consecutive chunks starting at l * per: all loads first (one
        // round trip to L2), a serial sum per lane, one warp scan, a serial prefix per lane
        const int per = (n + 31) / 32;
        int v[kMaxChunks / 32];
        int mine = 0;
#pragma unroll
        for (int i = 0; i < kMaxChunks / 32; ++i) {
            const int c = lane * per + i;
            v[i] = (i < per && c < n) ? __ldcg(p.chunk_hist + (size_t)bin * n + c) : 0;
        }
#pragma unroll
        for (int i = 0; i < kMaxChunks / 32; ++i) mine += v[i];
        const int incl = warp_incl_scan(mine, lane);
        int run = incl - mine;
#pragma unroll
        for (int i = 0; i < kMaxChunks / 32; ++i) {
            const int c = lane * per + i;
            if (i < per && c < n) p.chunk_base[(size_t)bin * n + c] = run;
            run += v[i];
        }
        const int carry = __shfl_sync(0xffffffffu, incl, 31);
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

static __device__ void scan_rank_sources(const Params& p, int r, const int* sm, int gtid, int gn) {
    // tokens before each source boundary = chunk prefix + running histogram at the boundary
    const int n = p.nchunks, L = p.L, B = p.B, T = p.T, S = p.S, E = p.E;
    for (int i = gtid; i < S * L; i += gn) {
        const int s = i / L, bi = i - s * L, bin = r * L + bi;
        const int eo = __ldcg(p.expert_offset + bin);
        const int b0 = src_begin(s, T, S);
        const int pre0 = __ldcg(p.chunk_base + (size_t)bin * n + chunk_of(b0, T, n)) +
                         __ldcg(p.partial + (size_t)s * B + bin);
        int pre1 = sm[bi];
        if (s + 1 < S) {
            const int b1 = src_begin(s + 1, T, S);
            pre1 = __ldcg(p.chunk_base + (size_t)bin * n + chunk_of(b1, T, n)) +
                   __ldcg(p.partial + (size_t)(s + 1) * B + bin);
        }
        p.src_offset[(size_t)s * E + bin] = eo + pre0;
        p.cnt[(size_t)s * E + bin] = pre1 - pre0;
    }
}

// -------------------------------------------------------- slot -> row assignment
// Final rows of this CTA's tokens [t0, t1).  rows_e(e, tl) / rows_r(r, tl) return how many
// rows precede local token tl in expert e's segment (offset of the segment included) / in
// rank r's region.  Writes slot_row / slot_pos and the per-row metadata (only when
// `write_meta`; with column parts one CTA of the group does it) and leaves in pos[] the
// global row to copy to (rank * cap + row), or -1, and in dst_key[] the place of that row's
// rank in the destination-ordering table rotated by the worker id (R for "no copy").
// w_sm: the tokens' gate weights, staged.  (Rows per rank are counted by whoever copies them.)
// kPeers (ranks on different GPUs, arenas of identical layout): what belongs to the receiver
// of a row -- its metadata and its expert row list -- is written into the arena of that rank,
// peer_delta[r] bytes away from this GPU's own.
template <bool kPeers, typename T>
__device__ __forceinline__ T* toward_peer(T* ptr, long long delta) {
    return kPeers ? reinterpret_cast<T*>(reinterpret_cast<char*>(ptr) + delta) : ptr;
}
template <bool kPeers = false, typename RowsE, typename RowsR>
__device__ void finalize_chunk(const Params& p, int t0, int t1, const int* ids, const float* w_sm, RowsE rows_e,
                               RowsR rows_r, bool write_meta, int worker, const int* order_sm, int* pos,
                               int* dst_key, int* arr, int gtid, int gn, const long long* peer_delta = nullptr) {
    const int k = p.k, L = p.L, R = p.R;
    const int rot = worker % R;
    const int nslots = (t1 - t0) * k;
    for (int li = gtid; li < nslots; li += gn) {
        const int tl = li / k, j = li - tl * k;
        const int t = t0 + tl;
        const size_t i = (size_t)t0 * k + li;
        const int packed = ids[li];
        int where = -1, row = -1, gpos = -1, r = 0;
        if (packed >= 0) {
            const int e = slot_expert(packed);
            r = slot_rank(packed);
            const long long pd = kPeers ? peer_delta[r] : 0;
            bool first = true;
            if (!p.dedup) {
                row = rows_e(e, tl);
            } else {
                for (int jj = 0; jj < j; ++jj) {
                    const int v2 = ids[li - j + jj];
                    if (v2 >= 0 && slot_rank(v2) == r) { first = false; break; }
                }
                row = rows_r(r, tl);
                if (write_meta) {
                    const int at = rows_e(e, tl);
                    if (at < p.er_cap) toward_peer<kPeers>(p.expert_rows, pd)[(size_t)r * p.er_cap + at] = row;
                    else report(p.status, kErrCapacity);
                }
            }
            if (row >= p.cap) {
                report(p.status, kErrCapacity);
            } else {
                gpos = r * p.cap + row;
                if (first) {
                    where = gpos;
                    if (arr) atomicAdd(&arr[r], 1);   // rows this CTA will copy to rank r (null: counted at copy time)
                    if (write_meta) {
                        toward_peer<kPeers>(p.recv_src_idx, pd)[where] = t;
                        if (!p.dedup) {
                            toward_peer<kPeers>(p.recv_weight, pd)[where] = w_sm[li];
                        } else {
                            const int* row_ids = ids + tl * k;
                            for (int jj = 0; jj < k; ++jj) {
                                const int v2 = row_ids[jj];
                                const bool here = v2 >= 0 && slot_rank(v2) == r;
                                toward_peer<kPeers>(p.recv_topk_idx, pd)[(size_t)where * k + jj] =
                                    here ? slot_expert(v2) - r * L : -1;
                                toward_peer<kPeers>(p.recv_topk_w, pd)[(size_t)where * k + jj] =
                                    here ? w_sm[tl * k + jj] : 0.0f;
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
        int kv = R;            // empty slots are issued last
        if (where >= 0) {
            kv = order_sm[r] - rot;
            kv += kv < 0 ? R : 0;
        }
        dst_key[li] = kv;
    }
}

// ------------------------------------------------- flag-free layout, every bin
// From the staged table of all T tokens (ids: T * k slots): the bitmaps of every bin, then per bin
// the total (tot), the count among the tokens before t0 (pre) and per expert the offset inside its
// rank's region (eo).  Run by the gn threads (nw warps) that share barrier `bar`; ends with that
// barrier.  Used by every kernel in which a CTA derives the layout alone.
static __device__ void local_counts_all_bins(const Params& p, int* ids, const BinMaps& bmaps, int t0, int* tot,
                                             int* pre, int* eo, int gtid, int gn, int gw, int nw, int lane, int bar) {
    build_bin_maps(p, ids, p.T, bmaps, gw, nw, lane);
    group_sync(bar, gn);
    for (int b = gtid; b < p.B; b += gn) {
        const int before = bits_in_range(bmaps, b, 0, t0);
        pre[b] = before;
        tot[b] = before + bits_in_range(bmaps, b, t0, p.T);
    }
    group_sync(bar, gn);
    for (int e = gtid; e < p.E; e += gn) {
        int o = 0;
        for (int q = (e / p.L) * p.L; q < e; ++q) o += tot[q];
        eo[e] = o;
    }
    group_sync(bar, gn);
}

// Rows region r receives, from the totals.
__device__ __forceinline__ int rows_of_rank(const Params& p, const int* tot, int r) {
    if (p.dedup) return tot[p.E + r];
    int rows = 0;
    for (int q = r * p.L; q < (r + 1) * p.L; ++q) rows += tot[q];
    return rows;
}

// The counts and offsets that are the same for everybody, written by one CTA.
static __device__ void write_totals(const Params& p, const int* tot, const int* eo, int gtid, int gn) {
    for (int e = gtid; e < p.E; e += gn) {
        p.expert_offset[e] = eo[e];
        p.num_tokens_per_expert[e] = tot[e];
    }
    for (int r = gtid; r < p.R; r += gn) {
        p.num_tokens_per_rank[r] = tot[p.E + r];
        p.num_rows_per_rank[r] = rows_of_rank(p, tot, r);
    }
}

// What source rank s reports (cnt, src_offset), from bitmaps over the whole table.
static __device__ void write_source_from_maps(const Params& p, int s, const BinMaps& bmaps, const int* eo, int gtid,
                                              int gn) {
    const int b0 = src_begin(s, p.T, p.S), b1 = src_begin(s + 1, p.T, p.S);
    for (int e = gtid; e < p.E; e += gn) {
        p.cnt[(size_t)s * p.E + e] = bits_in_range(bmaps, e, b0, b1);
        p.src_offset[(size_t)s * p.E + e] = eo[e] + bits_in_range(bmaps, e, 0, b0);
    }
}

// --------------------------------------------- flag-free layout, dedup fast path
// With one row per (token, rank) the movers only need rank-level rows: row of token t in
// region r = number of earlier tokens that visit r.  One 32-bit word per token and 32 ranks
// says which ranks it visits; transposed per group of 32 tokens it becomes, per rank, a
// bitmap over tokens, and the row is a population count.  Everything expert-level (offsets,
// counts per source, the per-expert row lists) is produced after the movers are released,
// each rank's share by one CTA.
struct RankMaps {
    unsigned* rbm;  // [groups, rp] rank bitmaps over all T tokens
    unsigned* dbm;  // [groups, 32] duty bitmaps: bit l < L = local expert l, bit L = the rank itself
    int wr;         // words of ranks per token: ceil(R / 32), at most kRankWords
    int rp;         // wr * 32
    int groups;     // ceil(T / 32)
};
constexpr int kRankWords = 4;


// Stage the slots (packed id | rank << 16) of the token groups [0, g_end) and build their rank bitmaps;
// lane = token, one group of 32 tokens per warp and trip.  Every CTA of the flag-free kernel runs this
// redundantly before its first copy and the step is bound by instruction issue (16 warps on four
// schedulers), so the common case -- no replica table, at most 32 ranks, eight slots per token -- is a
// variant of its own without per-slot branches: measured per warp and group, warm, 2380 cycles for the
// general form with a branch and a possible call per slot, about 1100 for this one.
// (An expert named twice by a token does not change any rank-level row, so this step, which every
// copy waits for, does not look for it; that happens once the movers are released.
// Looking for it here was measured to cost 2.5 us per dispatch of 512 tokens.)
template <bool kPlain, int kK>   // kPlain: no replica table, one word of ranks; kK: slots per token if fixed
__device__ __forceinline__ void stage_and_rank_maps_pass(const Params& p, int* ids, const RankMaps& rm, int g_end,
                                                         int gw, int nw, int lane) {
    const int k = kK ? kK : p.k, T = p.T;
    const bool vec = (k & 3) == 0;   // a token's ids are whole 16-byte words (topk_idx is 16-byte aligned)
    constexpr int kW = kPlain ? 1 : kRankWords;
    bool bad = false;
    for (int g = gw; g < g_end; g += nw) {
        const int t = g * 32 + lane;
        unsigned m[kW];
#pragma unroll
        for (int w = 0; w < kW; ++w) m[w] = 0u;
        if (t < T) {
            const int32_t* src = p.topk_idx + (size_t)t * k;
            for (int j0 = 0; j0 < k; j0 += 8) {       // up to eight ids in flight
                int raw[8];
                if (vec) {
                    const int4 a = __ldg(reinterpret_cast<const int4*>(src + j0));
                    const int4 b = j0 + 4 < k ? __ldg(reinterpret_cast<const int4*>(src + j0 + 4)) : make_int4(-1, -1, -1, -1);
                    raw[0] = a.x; raw[1] = a.y; raw[2] = a.z; raw[3] = a.w;
                    raw[4] = b.x; raw[5] = b.y; raw[6] = b.z; raw[7] = b.w;
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u) raw[u] = j0 + u < k ? __ldg(src + j0 + u) : -1;
                }
                int pk[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    int e = raw[u];   // (slots past the k-th hold -1)
                    if (!kPlain && p.phys != nullptr) {
                        const bool in = (unsigned)e < (unsigned)p.E_log;
                        bad |= !in && e != -1;
                        const int nc = in ? __ldg(p.ncopies + e) : 1;
                        const bool okc = in && nc >= 1 && nc <= p.C;
                        bad |= in && !okc;
                        e = okc ? __ldg(p.phys + (size_t)e * p.C + (t % nc)) : -1;
                        bad |= okc && e < 0;
                    }
                    const bool valid = (unsigned)e < (unsigned)p.E;
                    bad |= !valid && e != -1;
                    const int r = fast_div(e, p.L_magic);
                    pk[u] = valid ? (e | (r << 16)) : -1;
                    if (kPlain) {
                        m[0] |= valid ? 1u << r : 0u;
                    } else {
#pragma unroll
                        for (int w = 0; w < kW; ++w) m[w] |= (valid && w == (r >> 5)) ? 1u << (r & 31) : 0u;
                    }
                }
                // (one 16-byte store per four slots: scalar stores of a lane's slots, 32 bytes apart from
                // the next lane's, would meet in four banks)
                if (vec) {
                    *reinterpret_cast<int4*>(ids + (size_t)t * k + j0) = make_int4(pk[0], pk[1], pk[2], pk[3]);
                    if (j0 + 4 < k) *reinterpret_cast<int4*>(ids + (size_t)t * k + j0 + 4) = make_int4(pk[4], pk[5], pk[6], pk[7]);
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (j0 + u < k) ids[t * k + j0 + u] = pk[u];
                }
            }
        }
#pragma unroll
        for (int w = 0; w < kW; ++w)
            if (w < rm.wr) rm.rbm[(size_t)g * rm.rp + w * 32 + lane] = transpose32(m[w], lane);
    }
    if (bad) report(p.status, kErrBadIndex);
}
static __device__ void local_stage_and_rank_maps(const Params& p, int* ids, const RankMaps& rm, int g_end, int gw, int nw,
                                          int lane) {
    if (p.phys == nullptr && rm.wr == 1) {
        if (p.k == 8) stage_and_rank_maps_pass<true, 8>(p, ids, rm, g_end, gw, nw, lane);
        else stage_and_rank_maps_pass<true, 0>(p, ids, rm, g_end, gw, nw, lane);
    } else {
        stage_and_rank_maps_pass<false, 0>(p, ids, rm, g_end, gw, nw, lane);
    }
}

// Tokens below t that visit rank r.
__device__ __forceinline__ int rank_rows_before(const RankMaps& rm, int r, int t) {
    int c = 0;
    const int g1 = t >> 5;
    for (int g = 0; g < g1; ++g) c += __popc(rm.rbm[(size_t)g * rm.rp + r]);
    if (t & 31) c += __popc(rm.rbm[(size_t)g1 * rm.rp + r] & ((1u << (t & 31)) - 1u));
    return c;
}

// Destinations of this CTA's tokens [t0, t1): pos_raw (slot order), dst_key (only with a destination
// table), row_sm, arr.  Every copy of the CTA waits for this step and a handful of threads run it, so it
// is written for latency: no branch per slot, the token's other slots compared in registers, the bit
// counts of the groups below the token unrolled (independent loads), one report after the loop.
// (Ordering the destinations with warp shuffles right here instead of in a separate pass
// was measured slower on the decode shape and is not done.)
template <int kK>   // slots per token if fixed
__device__ __forceinline__ void rows_dedup_pass(const Params& p, int t0, int t1, const int* ids_all, const RankMaps& rm,
                                                int worker, const int* order_sm, int* pos_raw, int* dst_key, int* row_sm,
                                                int* arr, int gtid, int gn) {
    const int k = kK ? kK : p.k;
    const int nslots = (t1 - t0) * k;
    const int rot = worker % p.R;
    bool full = false;
    for (int li = gtid; li < nslots; li += gn) {
        const int tl = li / k, j = li - tl * k, t = t0 + tl;
        const int* tok = ids_all + (size_t)t * k;
        const int packed = tok[j];
        const bool have = packed >= 0;
        const int r = have ? slot_rank(packed) : 0;
        bool first = have;   // no earlier slot of the token names the same rank (-1 >> 16 is no rank)
        if (kK == 8) {
            const int4 a = *reinterpret_cast<const int4*>(tok), b = *reinterpret_cast<const int4*>(tok + 4);
            const int v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
            for (int jj = 0; jj < 7; ++jj) first = first && !(jj < j && slot_rank(v[jj]) == r);
        } else {
            for (int jj = 0; jj < j; ++jj) first = first && slot_rank(tok[jj]) != r;
        }
        // tokens below t that visit rank r
        const int g1 = t >> 5;
        const unsigned* col = rm.rbm + r;
        int row = __popc(col[(size_t)g1 * rm.rp] & ((1u << (t & 31)) - 1u));
#pragma unroll 8
        for (int g = 0; g < g1; ++g) row += __popc(col[(size_t)g * rm.rp]);
        const bool fits = row < p.cap;
        full = full || (have && !fits);
        const bool send = first && fits;
        if (send) atomicAdd(&arr[r], 1);
        pos_raw[li] = send ? r * p.cap + row : -1;
        if (p.ordered) {
            int kv = order_sm[r] - rot;
            kv = kv < 0 ? kv + p.R : kv;
            dst_key[li] = send ? kv : p.R;
        }
        row_sm[li] = have ? row : -1;
    }
    if (full) report(p.status, kErrCapacity);
}
static __device__ void local_rows_dedup(const Params& p, int t0, int t1, const int* ids_all, const RankMaps& rm,
                                 int worker, const int* order_sm, int* pos_raw, int* dst_key, int* row_sm, int* arr,
                                 int gtid, int gn) {
    if (p.k == 8) rows_dedup_pass<8>(p, t0, t1, ids_all, rm, worker, order_sm, pos_raw, dst_key, row_sm, arr, gtid, gn);
    else rows_dedup_pass<0>(p, t0, t1, ids_all, rm, worker, order_sm, pos_raw, dst_key, row_sm, arr, gtid, gn);
}

// The ids of a token must be distinct: the later of two slots naming one expert is reported
// (kErrBadIndex) and emptied.  In the flag-free kernel every CTA holds the whole table, but only two
// things read expert ids from it: the metadata of the CTA's own tokens, for which this empties the
// repeated slots of tokens [t0, t1) in the CTA's copy, and the per-rank duty, whose bitmaps take a
// repeated expert once by construction (it reports it) and whose row lists write the same entry twice.
static __device__ void local_clean_own_duplicates(const Params& p, int t0, int t1, int* ids_all, int gtid, int gn) {
    const int k = p.k;
#pragma unroll 1
    for (int t = t0 + gtid; t < t1; t += gn) {
        int* row = ids_all + (size_t)t * k;
#pragma unroll 1
        for (int j = 1; j < k; ++j) {
            const int v = row[j];
            if (v < 0) continue;
            bool dup = false;
#pragma unroll 1
            for (int jj = 0; jj < j; ++jj) dup = dup || row[jj] == v;   // same expert => same packed word
            if (dup) {
                report(p.status, kErrBadIndex);
                row[j] = -1;
            }
        }
    }
}

// Metadata of this CTA's own tokens (after the movers were released).
static __device__ void local_meta_dedup(const Params& p, int t0, int t1, const int* ids_all, const int* pos_raw,
                                 const int* row_sm, const float* w_own, int gtid, int gn) {
    const int k = p.k, L = p.L;
    const int nslots = (t1 - t0) * k;
#pragma unroll 1
    for (int li = gtid; li < nslots; li += gn) {
        const int tl = li / k, t = t0 + tl;
        const size_t i = (size_t)t0 * k + li;
        const int packed = ids_all[i];
        const int row = packed >= 0 ? row_sm[li] : -1;   // (a slot emptied as a duplicate has no row)
        p.slot_row[i] = row;
        p.slot_pos[i] = (packed >= 0 && row >= 0 && row < p.cap) ? slot_rank(packed) * p.cap + row : -1;
        const int where = pos_raw[li];
        if (where >= 0) {
            const int r = slot_rank(packed);
            p.recv_src_idx[where] = t;
            if ((k & 3) == 0) {   // rows of the two arrays start on 16-byte boundaries: four slots per store
#pragma unroll 1
                for (int j4 = 0; j4 < k; j4 += 4) {
                    int e4[4];
                    float w4[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int v2 = ids_all[(size_t)t * k + j4 + u];
                        const bool here = v2 >= 0 && slot_rank(v2) == r;
                        e4[u] = here ? slot_expert(v2) - r * L : -1;
                        w4[u] = here ? w_own[tl * k + j4 + u] : 0.0f;
                    }
                    *reinterpret_cast<int4*>(p.recv_topk_idx + (size_t)where * k + j4) = make_int4(e4[0], e4[1], e4[2], e4[3]);
                    *reinterpret_cast<float4*>(p.recv_topk_w + (size_t)where * k + j4) = make_float4(w4[0], w4[1], w4[2], w4[3]);
                }
            } else {
#pragma unroll 1
                for (int jj = 0; jj < k; ++jj) {
                    const int v2 = ids_all[(size_t)t * k + jj];
                    const bool here = v2 >= 0 && slot_rank(v2) == r;
                    p.recv_topk_idx[(size_t)where * k + jj] = here ? slot_expert(v2) - r * L : -1;
                    p.recv_topk_w[(size_t)where * k + jj] = here ? w_own[tl * k + jj] : 0.0f;
                }
            }
        }
    }
}

// Everything about rank r that nobody inside the kernel waits for: expert totals and
// offsets, tokens per rank, counts and offsets per source rank, the per-expert row lists.
// Needs L < 32.  `sm` holds 2 * 32 ints.  Run by the whole layout group (barrier bar_id).
// The rank's share is cut into Q parts handled by Q different CTAs: part q writes every
// Q-th entry of the per-source tables and of the row lists; part 0 also writes the totals.
static __device__ void local_rank_duty(const Params& p, int r, int q, int Q, const int* ids_all, const RankMaps& rm,
                                int* sm, int gw, int nw, int lane, int gtid, int gn, int bar_id) {
    const int k = p.k, L = p.L, T = p.T, S = p.S, E = p.E;
#pragma unroll 1
    for (int g = gw; g < rm.groups; g += nw) {
        const int t = g * 32 + lane;
        unsigned m = 0u;
        if (t < T)
#pragma unroll 1
            for (int j = 0; j < k; ++j) {
                const int v = ids_all[(size_t)t * k + j];
                if (v >= 0 && slot_rank(v) == r) {
                    const unsigned bit = 1u << (slot_expert(v) - r * L);
                    if (m & bit) report(p.status, kErrBadIndex);   // an expert named twice by this token
                    m |= bit | (1u << L);
                }
            }
        rm.dbm[(size_t)g * 32 + lane] = transpose32(m, lane);
    }
    group_sync(bar_id, gn);
    if (p.trace && gtid == 0) p.trace[(size_t)blockIdx.x * kTraceSlots + 13] = trace_ns(p);
    auto bits = [&](int l, int lo, int hi) {   // tokens in [lo, hi) with bit l
        if (hi <= lo) return 0;
        const int g0 = lo >> 5, g1 = (hi - 1) >> 5;
        int c = 0;
#pragma unroll 1
        for (int g = g0; g <= g1; ++g) {
            unsigned w = rm.dbm[(size_t)g * 32 + l];
            if (g == g0) w &= 0xffffffffu << (lo & 31);
            if (g == g1 && (hi & 31) != 0) w &= (1u << (hi & 31)) - 1u;
            c += __popc(w);
        }
        return c;
    };
    int* tot = sm;
    int* eo = sm + 32;
    if (gtid <= L) tot[gtid] = bits(gtid, 0, T);
    group_sync(bar_id, gn);
    if (gtid <= L) {
        int o = 0;
#pragma unroll 1
        for (int i = 0; i < gtid; ++i) o += tot[i];
        eo[gtid] = o;
        if (q == 0) {
            if (gtid < L) {
                p.expert_offset[r * L + gtid] = o;
                p.num_tokens_per_expert[r * L + gtid] = tot[gtid];
            } else {
                p.num_tokens_per_rank[r] = tot[L];
                p.num_rows_per_rank[r] = tot[L];
            }
        }
    }
    group_sync(bar_id, gn);
#pragma unroll 1
    for (int i = q + Q * gtid; i < S * L; i += Q * gn) {
        const int s = i / L, l = i - s * L;
        const int b0 = src_begin(s, T, S), b1 = src_begin(s + 1, T, S);
        p.cnt[(size_t)s * E + r * L + l] = bits(l, b0, b1);
        p.src_offset[(size_t)s * E + r * L + l] = eo[l] + bits(l, 0, b0);
    }
    if (p.trace && gtid == 0) p.trace[(size_t)blockIdx.x * kTraceSlots + 14] = trace_ns(p);
#pragma unroll 1
    for (int i = q + Q * gtid; i < T * k; i += Q * gn) {
        const int v = ids_all[i];
        if (v < 0 || slot_rank(v) != r) continue;
        const int t = i / k, l = slot_expert(v) - r * L;
        const int at = eo[l] + bits(l, 0, t);
        if (at < p.er_cap) p.expert_rows[(size_t)r * p.er_cap + at] = bits(L, 0, t);
        else report(p.status, kErrCapacity);
    }
    group_sync(bar_id, gn);   // sm and dbm are reused by the next rank
}

// Per token, put the destinations into the order of the destination-ordering table rotated
// by the worker id (Sec. 3.3: each worker visits a re-mapped destination sequence).  Only
// the issue order of the copies changes.  One thread per slot: its place is the number of
// the token's slots with a smaller key (ties keep slot order).  Reads pos / key, writes pos_out.
static __device__ void order_destinations(const Params& p, const int* pos, const int* key, int* pos_out, int nslots,
                                   int gtid, int gn) {
    const int k = p.k;
    for (int li = gtid; li < nslots; li += gn) {
        const int tl = li / k, j = li - tl * k;
        const int* kk = key + tl * k;
        const int kv = kk[j];
        int place = 0;
        for (int jj = 0; jj < k; ++jj) {
            const int ko = kk[jj];
            place += (ko < kv || (ko == kv && jj < j)) ? 1 : 0;
        }
        pos_out[tl * k + place] = pos[li];
    }
}

}  // namespace ubep
