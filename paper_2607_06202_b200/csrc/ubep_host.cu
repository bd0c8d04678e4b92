// C ABI of the library (declared in include/ubep.h): argument checks, arena layout and
// kernel launches.  No device memory is allocated here and no stream is created.
#include <atomic>
#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/ubep.h"
#include "ubep_kernels.h"
#include "ubep_sync.h"
#include "ubep_sharded.h"

using ubep::Params;

namespace {

std::atomic<uint64_t> g_launches{0};

constexpr size_t kAlign = 256;
constexpr int kStealMinTokensPerChunk = 40;  // shorter slices: the hand-out costs more than the tail it removes (measured)
constexpr int kDefaultCountWarps = 8;            // FP8: warps of the count group while the others quantise (measured sweep;
                                                 // -1 in the buffer = this default, and none with token stealing)
constexpr int64_t kLocalMaxSlots = 8192;        // small-T limit of the combine launch mode and of the protocol / sharded paths
// AUTO's crossovers between the flag-free and the flag-exchanging schedule, in routing-table slots (T * k);
// measured over three shape families (H / E / R = 7168 / 256 / 32, 4096 / 128 / 16, 7168 / 288 / 72), top-8,
// 64 .. 2048 tokens: the crossover follows the slots, not the number of bins.
constexpr int64_t kLocalFastMaxSlots = 16384;     // one row per (token, rank), bf16 rows: the rank-level fast path
                                                  // (2048 tokens: 50.4 against 58.4 us; larger tables do not fit in shared memory)
constexpr int64_t kLocalFastFp8MaxSlots = 8192;   // the same with FP8 rows (1024 tokens: 25.3 against 31.5 us, 1536: 39.4 against 38.4)
constexpr int64_t kLocalAllBinsMaxSlots = 3072;   // every bin's bitmaps have to be built, bf16 rows
constexpr int64_t kLocalAllBinsFp8MaxSlots = 1536;   // ... FP8 rows
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct ArenaLayout {
    size_t off[UBEP_VIEW_COUNT_];
    size_t slot_pos, copy_pos, chunk_hist, partial, chunk_base, trace;
    size_t flags_begin, hist_flag, scan_flag, status, ticket, epoch_ctr, done_ticket, cursor, pos_flag, claimed,
        order_pos, flags_end, peer_delta;
    size_t total;
    int er_cap, nchunks, S, rowB, G, B;
};

bool valid_config(const ubep_config_t& c) {
    if (c.num_ranks < 1 || c.num_experts < 1 || c.num_experts % c.num_ranks != 0) return false;
    if (c.num_experts > 65535) return false;  // staged slots pack the expert id into 16 bits
    if (c.topk < 1 || c.topk > ubep::kMaxTopk) return false;
    if (c.hidden < 8 || c.hidden % 8 != 0) return false;
    if (c.payload != UBEP_PAYLOAD_BF16 && c.payload != UBEP_PAYLOAD_FP8_E4M3) return false;
    if (c.payload == UBEP_PAYLOAD_FP8_E4M3 && c.hidden % 128 != 0) return false;
    if (c.max_tokens < 1 || c.rows_per_rank_cap < 1 || c.num_src_ranks < 0) return false;
    if (c.dedup != 0 && c.dedup != 1) return false;
    if (c.pipeline < UBEP_PIPELINE_AUTO || c.pipeline > UBEP_PIPELINE_LOCAL) return false;
    if (c.num_ctas < 0 || c.num_ctas > ubep::kMaxChunks) return false;
    if ((int64_t)c.num_ranks * c.rows_per_rank_cap > INT32_MAX) return false;
    if ((int64_t)c.max_tokens * c.topk > INT32_MAX) return false;
    return true;
}

// nchunks == 0 means "not known yet": size for the largest value allowed.
ArenaLayout make_layout(const ubep_config_t& c, int nchunks) {
    ArenaLayout a{};
    const size_t R = c.num_ranks, E = c.num_experts, H = c.hidden, k = c.topk, cap = c.rows_per_rank_cap;
    const size_t L = E / R;
    a.S = c.num_src_ranks > 0 ? c.num_src_ranks : c.num_ranks;
    a.rowB = c.payload ? (int)H : (int)(2 * H);
    a.G = (int)(H / 128);
    a.B = (int)(E + R);
    a.nchunks = nchunks > 0 ? nchunks : ubep::kMaxChunks;
    a.er_cap = c.dedup ? (int)(cap * (k < L ? k : L)) : 0;
    const size_t S = a.S, n = a.nchunks, B = a.B, Tk = (size_t)c.max_tokens * k;
    size_t at = 0;
    auto take = [&](size_t bytes) { size_t o = at; at = align_up(at + bytes); return o; };
    a.off[UBEP_VIEW_RECV_X] = take(R * cap * a.rowB);
    a.off[UBEP_VIEW_RECV_SCALE] = take(c.payload ? R * cap * a.G * 4 : 0);
    a.off[UBEP_VIEW_RECV_SRC_IDX] = take(R * cap * 4);
    a.off[UBEP_VIEW_RECV_WEIGHT] = take(c.dedup ? 0 : R * cap * 4);
    a.off[UBEP_VIEW_RECV_TOPK_IDX] = take(c.dedup ? R * cap * k * 4 : 0);
    a.off[UBEP_VIEW_RECV_TOPK_W] = take(c.dedup ? R * cap * k * 4 : 0);
    a.off[UBEP_VIEW_EXPERT_ROWS] = take(R * (size_t)a.er_cap * 4);
    a.off[UBEP_VIEW_CNT] = take(S * E * 4);
    a.off[UBEP_VIEW_SRC_OFFSET] = take(S * E * 4);
    a.off[UBEP_VIEW_EXPERT_OFFSET] = take(E * 4);
    a.off[UBEP_VIEW_NUM_TOKENS_PER_EXPERT] = take(E * 4);
    a.off[UBEP_VIEW_NUM_ROWS_PER_RANK] = take(R * 4);
    a.off[UBEP_VIEW_NUM_TOKENS_PER_RANK] = take(R * 4);
    a.off[UBEP_VIEW_SLOT_ROW] = take(Tk * 4);
    a.slot_pos = take(Tk * 4);
    a.copy_pos = take(Tk * 4);
    a.chunk_hist = take(n * B * 4);
    a.partial = take(S * B * 4);
    a.chunk_base = take(n * B * 4);
    a.off[UBEP_VIEW_TRACE] = a.trace = take(n * ubep::kTraceSlots * 8);
    a.flags_begin = at;
    a.hist_flag = take(n * 4);
    a.scan_flag = take(R * 4);
    a.off[UBEP_VIEW_ARRIVAL] = take(2 * R * 4);
    a.status = take(4);
    a.ticket = take(4);
    a.off[UBEP_VIEW_EPOCH] = a.epoch_ctr = take(4);
    a.done_ticket = take(4);
    a.cursor = take(n * 4);
    a.pos_flag = take(n * 4);
    a.claimed = take(8);
    a.off[UBEP_VIEW_SHARD_ARRIVAL] = take(8);
    a.flags_end = at;
    a.order_pos = take(R * 4);
    a.peer_delta = take(R * 8);
    a.total = at;
    return a;
}

// Wire buffer of the readiness-protocol dispatch (byte offsets).
struct WireLayout {
    size_t off[UBEP_SYNC_VIEW_COUNT_];
    size_t flags_begin, sp_dirty, seq_ticket, scan_count, flags_end, total;
    int tff_blocks, sp_row;
};

WireLayout make_wire_layout(const ubep_config_t& c, int nchunks) {
    WireLayout w{};
    // bytes of one row on the wire: the bf16 row, or the e4m3 payload followed by its fp32 scales
    const size_t R = c.num_ranks, cap = c.rows_per_rank_cap;
    const size_t rowB = c.payload ? (size_t)c.hidden + 4 * (size_t)(c.hidden / 128) : 2 * (size_t)c.hidden;
    const int payload = UBEP_SYNC_BLOCK_BYTES - UBEP_SYNC_FLAG_BYTES;
    w.tff_blocks = (int)((rowB + payload - 1) / payload);
    w.sp_row = (int)((rowB + UBEP_SYNC_BLOCK_BYTES - 1) / UBEP_SYNC_BLOCK_BYTES * UBEP_SYNC_BLOCK_BYTES);
    size_t at = 0;
    auto take = [&](size_t bytes) { size_t o = at; at = align_up(at + bytes); return o; };
    w.off[UBEP_SYNC_VIEW_TFF_WIRE] = take(R * cap * (size_t)w.tff_blocks * UBEP_SYNC_BLOCK_BYTES);
    w.off[UBEP_SYNC_VIEW_SP_WIRE] = take(R * cap * (size_t)w.sp_row);
    w.flags_begin = at;
    w.off[UBEP_SYNC_VIEW_CHECKSUM] = take(2 * R * 8);
    w.off[UBEP_SYNC_VIEW_COUNTERS] = take(4 * R * 4);
    w.sp_dirty = take(4);   // (inside the range that is cleared when the wire is re-filled)
    w.off[UBEP_SYNC_VIEW_SEQ] = take(4);
    w.seq_ticket = take(4);
    w.scan_count = take(8);
    w.off[UBEP_SYNC_VIEW_TIMES] = take((size_t)(nchunks > 0 ? nchunks : ubep::kMaxChunks) * ubep::kSyncTimeSlots * 8);
    w.flags_end = at;
    w.total = at;
    return w;
}

}  // namespace

struct ubep_buffer {
    ubep_config_t cfg;
    ArenaLayout lay;
    uint8_t* arena;
    int num_sms;
    int max_smem;
    int sm_khz;
    uint32_t epoch;
    int32_t withhold;
    int32_t tracing;
    int32_t quant_warps;
    int32_t count_warps;     // FP8 with flags / kernel boundaries: warps that compute the layout (0 = all, quantise afterwards)
    int32_t prefetch_rows;   // FP8: rows fetched before the layout is done, at most
    cudaStream_t last_stream;
    const int32_t* phys;
    const int32_t* ncopies;
    int32_t E_log, C;
    int32_t ordered;    // a destination-ordering table has been set
    int32_t my_rank;    // sharded use (ubep_set_peers): this GPU's rank, -1 otherwise
    uint8_t* wire;      // readiness-protocol wire buffer (caller-owned) or null
    WireLayout wlay;
    bool sp_dirty;      // an earlier call may have left non-sentinel blocks in the SP wire
    std::string cuda_error;
};

namespace {

int cuda_fail(ubep_buffer* b, cudaError_t e) {
    if (b) b->cuda_error = cudaGetErrorString(e);
    return UBEP_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
T* at(ubep_buffer* b, size_t off) { return reinterpret_cast<T*>(b->arena + off); }

Params make_params(ubep_buffer* b, int T) {
    const ubep_config_t& c = b->cfg;
    const ArenaLayout& a = b->lay;
    Params p{};
    p.T = T; p.H = c.hidden; p.E = c.num_experts; p.R = c.num_ranks; p.L = p.E / p.R; p.k = c.topk;
    p.S = a.S; p.cap = c.rows_per_rank_cap; p.payload = c.payload; p.dedup = c.dedup;
    p.rowB = a.rowB; p.G = a.G; p.B = a.B; p.nchunks = a.nchunks; p.er_cap = a.er_cap;
    p.parts = 1; p.grid = a.nchunks;
    p.L_magic = p.L == 1 ? 0xffffffffu : (unsigned)((0x100000000ull + (uint64_t)p.L - 1) / (uint64_t)p.L);
    p.local_fast = (c.dedup && p.L < 32 && p.L > 1 && p.R <= 32 * ubep::kRankWordsHost) ? 1 : 0;
    p.epoch_ctr = at<unsigned>(b, a.epoch_ctr);
    p.done_ticket = at<unsigned>(b, a.done_ticket);
    p.withhold = -1;
    p.phys = b->phys; p.ncopies = b->ncopies; p.E_log = b->E_log; p.C = b->C;
    p.order_pos = at<int32_t>(b, a.order_pos);
    p.ordered = b->ordered;
    p.recv_x = at<uint8_t>(b, a.off[UBEP_VIEW_RECV_X]);
    p.recv_scale = at<float>(b, a.off[UBEP_VIEW_RECV_SCALE]);
    p.recv_src_idx = at<int32_t>(b, a.off[UBEP_VIEW_RECV_SRC_IDX]);
    p.recv_weight = at<float>(b, a.off[UBEP_VIEW_RECV_WEIGHT]);
    p.recv_topk_idx = at<int32_t>(b, a.off[UBEP_VIEW_RECV_TOPK_IDX]);
    p.recv_topk_w = at<float>(b, a.off[UBEP_VIEW_RECV_TOPK_W]);
    p.expert_rows = at<int32_t>(b, a.off[UBEP_VIEW_EXPERT_ROWS]);
    p.cnt = at<int32_t>(b, a.off[UBEP_VIEW_CNT]);
    p.src_offset = at<int32_t>(b, a.off[UBEP_VIEW_SRC_OFFSET]);
    p.expert_offset = at<int32_t>(b, a.off[UBEP_VIEW_EXPERT_OFFSET]);
    p.num_tokens_per_expert = at<int32_t>(b, a.off[UBEP_VIEW_NUM_TOKENS_PER_EXPERT]);
    p.num_rows_per_rank = at<int32_t>(b, a.off[UBEP_VIEW_NUM_ROWS_PER_RANK]);
    p.num_tokens_per_rank = at<int32_t>(b, a.off[UBEP_VIEW_NUM_TOKENS_PER_RANK]);
    p.slot_row = at<int32_t>(b, a.off[UBEP_VIEW_SLOT_ROW]);
    p.slot_pos = at<int32_t>(b, a.slot_pos);
    p.copy_pos = at<int32_t>(b, a.copy_pos);
    p.cursor = at<unsigned>(b, a.cursor);
    p.pos_flag = at<unsigned>(b, a.pos_flag);
    p.claimed = at<unsigned>(b, a.claimed);
    p.steal = 0;
    p.quant_warps = b->quant_warps;
    p.count_warps = b->count_warps < 0 ? kDefaultCountWarps : b->count_warps;
    p.prefetch_rows = b->prefetch_rows;
    p.chunk_hist = at<int32_t>(b, a.chunk_hist);
    p.partial = at<int32_t>(b, a.partial);
    p.chunk_base = at<int32_t>(b, a.chunk_base);
    p.hist_flag = at<unsigned>(b, a.hist_flag);
    p.scan_flag = at<unsigned>(b, a.scan_flag);
    p.arrival = at<unsigned>(b, a.off[UBEP_VIEW_ARRIVAL]);
    p.status = at<int32_t>(b, a.status);
    p.trace = b->tracing ? at<unsigned long long>(b, a.trace) : nullptr;
    p.ns_per_cycle_q20 = (unsigned)((1000000.0 / (double)b->sm_khz) * 1048576.0 + 0.5);
    p.my_rank = b->my_rank;
    p.tok0 = 0;
    p.tok1 = T;
    p.peer_delta = at<long long>(b, a.peer_delta);
    p.shard_arrival = at<unsigned>(b, a.off[UBEP_VIEW_SHARD_ARRIVAL]);
    return p;
}

// Makes the buffer's device current for the scope of one call.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev) {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) {
            err = cudaSetDevice(dev);
            switched = err == cudaSuccess;
        }
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" {

size_t ubep_buffer_bytes(const ubep_config_t* cfg) {
    if (!cfg || !valid_config(*cfg)) return 0;
    return make_layout(*cfg, cfg->num_ctas).total;
}

int ubep_buffer_create(const ubep_config_t* cfg, void* dev_arena, size_t bytes, ubep_buffer_t** out) {
    if (!cfg || !out || !dev_arena || !valid_config(*cfg)) return UBEP_ERR_ARG;
    *out = nullptr;
    if ((reinterpret_cast<uintptr_t>(dev_arena) & (kAlign - 1)) != 0) return UBEP_ERR_ARENA;
    if (bytes < make_layout(*cfg, cfg->num_ctas).total) return UBEP_ERR_ARENA;
    DeviceGuard guard(cfg->device);
    if (guard.err != cudaSuccess) return UBEP_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return UBEP_ERR_CUDA;
    ubep_buffer* b = new (std::nothrow) ubep_buffer();
    if (!b) return UBEP_ERR_ARG;
    b->cfg = *cfg;
    b->num_sms = prop.multiProcessorCount;
    b->max_smem = (int)prop.sharedMemPerBlockOptin;
    b->sm_khz = prop.clockRate > 0 ? prop.clockRate : 1965000;
    int n = cfg->num_ctas > 0 ? cfg->num_ctas : b->num_sms;
    if (n > b->num_sms) n = b->num_sms;  // all CTAs of the persistent kernel must be resident
    if (n > ubep::kMaxChunks) n = ubep::kMaxChunks;
    b->lay = make_layout(*cfg, n);
    b->arena = static_cast<uint8_t*>(dev_arena);
    b->epoch = 0;
    b->withhold = -1;
    b->tracing = 0;
    b->quant_warps = ubep::kWarps - 2;
    b->count_warps = -1;
    b->prefetch_rows = INT32_MAX;
    b->last_stream = nullptr;
    b->phys = nullptr;
    b->ncopies = nullptr;
    b->E_log = 0;
    b->C = 0;
    b->ordered = 0;
    b->my_rank = -1;
    b->wire = nullptr;
    b->wlay = WireLayout{};
    b->sp_dirty = false;
    cudaError_t e = cudaMemset(b->arena + b->lay.flags_begin, 0, b->lay.flags_end - b->lay.flags_begin);
    if (e == cudaSuccess) {
        std::vector<int32_t> ident(cfg->num_ranks);
        for (int r = 0; r < cfg->num_ranks; ++r) ident[r] = r;
        e = cudaMemcpy(b->arena + b->lay.order_pos, ident.data(), sizeof(int32_t) * ident.size(),
                       cudaMemcpyHostToDevice);
    }
    if (e != cudaSuccess) {
        delete b;
        return UBEP_ERR_CUDA;
    }
    *out = b;
    return UBEP_OK;
}

int ubep_buffer_destroy(ubep_buffer_t* buf) {
    if (!buf) return UBEP_ERR_ARG;
    delete buf;
    return UBEP_OK;
}

int ubep_set_replicas(ubep_buffer_t* buf, const int32_t* phys, const int32_t* ncopies, int32_t E_log, int32_t C) {
    if (!buf) return UBEP_ERR_ARG;
    if (!phys && !ncopies) {
        buf->phys = nullptr; buf->ncopies = nullptr; buf->E_log = 0; buf->C = 0;
        return UBEP_OK;
    }
    if (!phys || !ncopies || E_log < 1 || C < 1) return UBEP_ERR_ARG;
    buf->phys = phys; buf->ncopies = ncopies; buf->E_log = E_log; buf->C = C;
    return UBEP_OK;
}

int ubep_set_dest_order(ubep_buffer_t* buf, const int32_t* order) {
    if (!buf) return UBEP_ERR_ARG;
    const int R = buf->cfg.num_ranks;
    std::vector<int32_t> posv(R, -1);
    for (int i = 0; i < R; ++i) {
        const int r = order ? order[i] : i;
        if (r < 0 || r >= R || posv[r] != -1) return UBEP_ERR_ARG;  // not a permutation
        posv[r] = i;
    }
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    // ordered after earlier work on the stream of the last call, then waited for
    cudaError_t e = cudaMemcpyAsync(buf->arena + buf->lay.order_pos, posv.data(), sizeof(int32_t) * R,
                                    cudaMemcpyHostToDevice, buf->last_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(buf->last_stream);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    buf->ordered = order != nullptr;
    return UBEP_OK;
}

int ubep_get_dispatch_layout(ubep_buffer_t* buf, const int32_t* topk_idx, int32_t T, int32_t* num_tokens_per_rank,
                             int32_t* num_tokens_per_expert, uint8_t* is_token_in_rank, void* cuda_stream) {
    if (!buf || T < 0 || T > buf->cfg.max_tokens || (T > 0 && !topk_idx) || !aligned16(topk_idx)) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    buf->last_stream = st;
    Params p = make_params(buf, T);
    p.topk_idx = topk_idx;
    cudaError_t e = ubep::launch_layout(p, num_tokens_per_rank, num_tokens_per_expert, is_token_in_rank,
                                        p.chunk_hist, at<unsigned>(buf, buf->lay.ticket), st);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    g_launches += 1;
    return UBEP_OK;
}

int ubep_dispatch(ubep_buffer_t* buf, const void* x, const int32_t* topk_idx, const float* topk_w, int32_t T,
                  void* cuda_stream) {
    if (!buf || T < 0 || T > buf->cfg.max_tokens) return UBEP_ERR_ARG;
    if (T > 0 && (!x || !topk_idx || !topk_w)) return UBEP_ERR_ARG;
    if (!aligned16(x) || !aligned16(topk_idx) || !aligned16(topk_w)) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    buf->last_stream = st;
    if (T == 0) {
        // nothing to route: every count and offset is zero (one contiguous block of the arena)
        const size_t lo = buf->lay.off[UBEP_VIEW_CNT], hi = buf->lay.off[UBEP_VIEW_SLOT_ROW];
        cudaError_t e0 = cudaMemsetAsync(buf->arena + lo, 0, hi - lo, st);
        return e0 == cudaSuccess ? UBEP_OK : cuda_fail(buf, e0);
    }
    buf->epoch += 1;
    Params p = make_params(buf, T);
    p.x = static_cast<const uint16_t*>(x);
    p.topk_idx = topk_idx;
    p.topk_w = topk_w;
    p.withhold = buf->withhold;
    buf->withhold = -1;
    // AUTO: a routing table that fits in shared memory is cheaper to recount in every CTA
    // than to exchange through flags; larger ones use the decomposed kernel.
    int mode = buf->cfg.pipeline;
    if (mode == UBEP_PIPELINE_AUTO) {
        // With the rank-level fast path the flag-free kernel wins up to about 1800 tokens of top-8 (bf16 rows);
        // when every CTA has to build the bitmaps of every bin it wins only for a few hundred tokens, and
        // with FP8 rows (whose quantising warps are the layout warps there, so nothing moves before the
        // layout and its outputs are done) for fewer still.
        const int64_t slots = (int64_t)T * p.k;
        const int64_t limit = p.local_fast ? (p.payload ? kLocalFastFp8MaxSlots : kLocalFastMaxSlots)
                                           : (p.payload ? kLocalAllBinsFp8MaxSlots : kLocalAllBinsMaxSlots);
        const bool local = slots <= limit;
        mode = local ? UBEP_PIPELINE_LOCAL : UBEP_PIPELINE_FUSED;
    }
    ubep::SmemPlan pl{};
    int launches = 0;
    p.parts = 1;
    p.grid = p.nchunks;
    if (mode == UBEP_PIPELINE_LOCAL) {
        // split rows into column parts until the slices of work are balanced to ~5 %
        const int n = buf->lay.nchunks;
        // The CTA with the most work sets the pace: ceil(T / chunks) tokens of 1 / parts of a row each.
        // Smaller pieces cost more per byte (measured on the decode shape: 4 parts + 8 %, 8 parts + 60 %).
        int best = 1;
        double best_cost = 0.0;
        static const double kPiecePenalty[4] = {1.0, 1.0, 1.08, 1.6};
        for (int parts = 1, i = 0; parts <= 8; parts *= 2, ++i) {
            const int chunks = n / parts;
            if (chunks < 1 || (p.H * 2 / parts) % 16 != 0 || (p.H * 2) % parts != 0) break;
            if (p.payload && ((p.H / parts) % 128 != 0 || p.H % parts != 0)) break;
            // FP8 rows: a piece's scales must still be a bulk copy (a multiple of 16 bytes); with plain stores for
            // the scales and payload pieces under 2 KB a dispatch of 384 tokens took 33 us against 21 us for 512
            if (p.payload && parts > 1 && ((p.G / parts) * 4) % 16 != 0) break;
            const double cost = (double)((T + chunks - 1) / chunks) / parts * kPiecePenalty[i];
            if (parts == 1 || cost < best_cost * 0.999) {
                best = parts;
                best_cost = cost;
            }
        }
        p.parts = best;
        p.nchunks = n / best;
        p.grid = p.nchunks * best;
        if (ubep::plan_dispatch(p, mode, buf->max_smem, &pl) != 0) {
            if (buf->cfg.pipeline == UBEP_PIPELINE_LOCAL) return UBEP_ERR_ARG;
            mode = UBEP_PIPELINE_FUSED;   // table too large for shared memory
            p.parts = 1;
            p.nchunks = n;
            p.grid = n;
        }
    }
    // slices that are long enough are handed out in blocks so that faster SMs can take over the tail of slower ones
    if (mode != UBEP_PIPELINE_LOCAL) p.steal = T >= kStealMinTokensPerChunk * p.nchunks ? 1 : 0;
    // With token stealing the count group is not used unless asked for: measured equal at top-8 and slower at
    // top-4 (16384 tokens: 161 against 174 us) -- every hand-out is a round trip that idle quantising warps do not hide.
    if (p.steal && buf->count_warps < 0) p.count_warps = 0;
    if (mode != UBEP_PIPELINE_LOCAL && ubep::plan_dispatch(p, mode, buf->max_smem, &pl) != 0) return UBEP_ERR_ARG;
    cudaError_t e = ubep::launch_dispatch(p, mode, pl, st, &launches);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    g_launches += launches;
    return UBEP_OK;
}

int ubep_combine(ubep_buffer_t* buf, const void* y, const float* topk_w, int32_t T, void* out, void* cuda_stream) {
    if (!buf || T < 0 || T > buf->cfg.max_tokens) return UBEP_ERR_ARG;
    if (T > 0 && (!y || !topk_w || !out)) return UBEP_ERR_ARG;
    if (!aligned16(y) || !aligned16(topk_w) || !aligned16(out)) return UBEP_ERR_ARG;
    if (T == 0) return UBEP_OK;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    buf->last_stream = st;
    cudaError_t e = ubep::launch_combine(static_cast<const uint16_t*>(y), at<int32_t>(buf, buf->lay.slot_pos), topk_w,
                                         T, buf->cfg.hidden, buf->cfg.topk, static_cast<uint16_t*>(out),
                                         buf->num_sms, (int64_t)T * buf->cfg.topk <= kLocalMaxSlots, st);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    g_launches += 1;
    return UBEP_OK;
}

size_t ubep_sync_wire_bytes(const ubep_config_t* cfg) {
    if (!cfg || !valid_config(*cfg)) return 0;
    return make_wire_layout(*cfg, cfg->num_ctas).total;
}

int ubep_sync_attach(ubep_buffer_t* buf, void* dev_wire, size_t bytes, void* cuda_stream) {
    if (!buf || !dev_wire) return UBEP_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(dev_wire) & (kAlign - 1)) != 0) return UBEP_ERR_ARENA;
    if (bytes < make_wire_layout(buf->cfg, buf->cfg.num_ctas).total) return UBEP_ERR_ARENA;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const WireLayout w = make_wire_layout(buf->cfg, buf->lay.nchunks);
    uint8_t* base = static_cast<uint8_t*>(dev_wire);
    // flags of no call (0), sentinel everywhere (0xFF bytes = bf16 code 0xFFFF), counters zero
    cudaError_t e = cudaMemsetAsync(base + w.off[UBEP_SYNC_VIEW_TFF_WIRE], 0,
                                    w.off[UBEP_SYNC_VIEW_SP_WIRE] - w.off[UBEP_SYNC_VIEW_TFF_WIRE], st);
    if (e == cudaSuccess)
        e = cudaMemsetAsync(base + w.off[UBEP_SYNC_VIEW_SP_WIRE], 0xFF, w.flags_begin - w.off[UBEP_SYNC_VIEW_SP_WIRE], st);
    if (e == cudaSuccess) e = cudaMemsetAsync(base + w.flags_begin, 0, w.flags_end - w.flags_begin, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    buf->wire = base;
    buf->wlay = w;
    buf->sp_dirty = false;
    return UBEP_OK;
}

int ubep_dispatch_sync(ubep_buffer_t* buf, int protocol, const void* x, const int32_t* topk_idx, const float* topk_w,
                       int32_t T, void* cuda_stream) {
    if (!buf || !buf->wire || protocol < UBEP_SYNC_SW || protocol > UBEP_SYNC_SP) return UBEP_ERR_ARG;
    if (T < 0 || T > buf->cfg.max_tokens) return UBEP_ERR_ARG;
    if (T > 0 && (!x || !topk_idx || !topk_w)) return UBEP_ERR_ARG;
    if (!aligned16(x) || !aligned16(topk_idx) || !aligned16(topk_w)) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    buf->last_stream = st;
    if (T == 0) {
        const size_t lo = buf->lay.off[UBEP_VIEW_CNT], hi = buf->lay.off[UBEP_VIEW_SLOT_ROW];
        cudaError_t e0 = cudaMemsetAsync(buf->arena + lo, 0, hi - lo, st);
        return e0 == cudaSuccess ? UBEP_OK : cuda_fail(buf, e0);
    }
    Params p = make_params(buf, T);
    p.x = static_cast<const uint16_t*>(x);
    p.topk_idx = topk_idx;
    p.topk_w = topk_w;
    p.trace = nullptr;
    p.parts = 1;
    p.grid = p.nchunks;
    ubep::SmemPlan pl{};
    const int extra = ubep::sync_extra_smem(p);
    // Small tables are recounted by every CTA; for larger ones TokenCnt and CalCumSum run as launches of their
    // own in front of the kernel, over the same chunks (as the phased schedule of ubep_dispatch does).
    const bool whole_table = (int64_t)T * buf->cfg.topk <= kLocalMaxSlots &&
                             ubep::plan_dispatch(p, UBEP_PIPELINE_LOCAL, buf->max_smem - extra, &pl) == 0;
    if (!whole_table && ubep::plan_dispatch(p, UBEP_PIPELINE_PHASED, buf->max_smem - extra, &pl) != 0)
        return UBEP_ERR_ARG;
    const WireLayout& w = buf->wlay;
    ubep::SyncParams sp{};
    sp.protocol = protocol;
    sp.tff_blocks = w.tff_blocks;
    sp.tff_wire = buf->wire + w.off[UBEP_SYNC_VIEW_TFF_WIRE];
    sp.sp_wire = buf->wire + w.off[UBEP_SYNC_VIEW_SP_WIRE];
    sp.checksum = reinterpret_cast<unsigned long long*>(buf->wire + w.off[UBEP_SYNC_VIEW_CHECKSUM]);
    sp.announced = reinterpret_cast<unsigned*>(buf->wire + w.off[UBEP_SYNC_VIEW_COUNTERS]);
    sp.sw_rows = sp.announced + 2 * (size_t)p.R;
    sp.seq_ctr = reinterpret_cast<unsigned*>(buf->wire + w.off[UBEP_SYNC_VIEW_SEQ]);
    sp.seq_ticket = reinterpret_cast<unsigned*>(buf->wire + w.seq_ticket);
    sp.sp_dirty = reinterpret_cast<unsigned*>(buf->wire + w.sp_dirty);
    sp.times = reinterpret_cast<unsigned long long*>(buf->wire + w.off[UBEP_SYNC_VIEW_TIMES]);
    cudaError_t e = cudaSuccess;
    if (buf->sp_dirty) {
        // a call that gave up may have left arrived blocks behind: every block back to the
        // sentinel, and the counters and the check-in ticket of that call back to zero
        e = cudaMemsetAsync(sp.sp_wire, 0xFF, w.flags_begin - w.off[UBEP_SYNC_VIEW_SP_WIRE], st);
        if (e == cudaSuccess)
            e = cudaMemsetAsync(buf->wire + w.off[UBEP_SYNC_VIEW_CHECKSUM], 0,
                                w.off[UBEP_SYNC_VIEW_SEQ] - w.off[UBEP_SYNC_VIEW_CHECKSUM], st);
        if (e != cudaSuccess) return cuda_fail(buf, e);
        buf->sp_dirty = false;
    }
    if (!whole_table) {
        e = ubep::launch_count_scan(p, pl, st);
        if (e != cudaSuccess) return cuda_fail(buf, e);
        g_launches += 2;
    }
    e = ubep::launch_sync_dispatch(p, pl, sp, whole_table, st);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    g_launches += 1;
    return UBEP_OK;
}

int ubep_sync_view(ubep_buffer_t* buf, int which, void** dev_ptr, int64_t shape[4]) {
    if (!buf || !buf->wire || !dev_ptr || !shape || which < 0 || which >= UBEP_SYNC_VIEW_COUNT_) return UBEP_ERR_ARG;
    const ubep_config_t& c = buf->cfg;
    int64_t s[4] = {1, 1, 1, 1};
    switch (which) {
        case UBEP_SYNC_VIEW_TFF_WIRE:
            s[0] = c.num_ranks; s[1] = c.rows_per_rank_cap; s[2] = (int64_t)buf->wlay.tff_blocks * UBEP_SYNC_BLOCK_BYTES;
            break;
        case UBEP_SYNC_VIEW_SP_WIRE: s[0] = c.num_ranks; s[1] = c.rows_per_rank_cap; s[2] = buf->wlay.sp_row; break;
        case UBEP_SYNC_VIEW_CHECKSUM: s[0] = 2; s[1] = c.num_ranks; break;
        case UBEP_SYNC_VIEW_COUNTERS: s[0] = 4; s[1] = c.num_ranks; break;
        case UBEP_SYNC_VIEW_TIMES: s[0] = buf->lay.nchunks; s[1] = ubep::kSyncTimeSlots; break;
        case UBEP_SYNC_VIEW_SEQ: s[0] = 1; break;
        default: return UBEP_ERR_ARG;
    }
    *dev_ptr = buf->wire + buf->wlay.off[which];
    for (int i = 0; i < 4; ++i) shape[i] = s[i];
    return UBEP_OK;
}

int ubep_sync_scan_sentinel(ubep_buffer_t* buf, const void* x, int32_t T, int64_t* count, void* cuda_stream) {
    if (!buf || !buf->wire || !count || T < 0 || (T > 0 && !x) || !aligned16(x)) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned long long* dev_count = reinterpret_cast<unsigned long long*>(buf->wire + buf->wlay.scan_count);
    unsigned long long host_count = 0;
    cudaError_t e = cudaMemsetAsync(dev_count, 0, sizeof(unsigned long long), st);
    if (e == cudaSuccess && T > 0) {
        e = ubep::launch_sentinel_scan(x, (long long)T * (buf->cfg.hidden / 8), dev_count, buf->num_sms, st);
        g_launches += 1;
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(&host_count, dev_count, sizeof(host_count), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    *count = (int64_t)host_count;
    return UBEP_OK;
}

int ubep_set_peers(ubep_buffer_t* buf, int32_t my_rank, void* const* peer_arenas) {
    if (!buf || !peer_arenas || my_rank < 0 || my_rank >= buf->cfg.num_ranks) return UBEP_ERR_ARG;
    const int R = buf->cfg.num_ranks;
    if (buf->lay.S != R) return UBEP_ERR_ARG;   // one source rank per GPU
    if (peer_arenas[my_rank] != buf->arena) return UBEP_ERR_ARG;
    std::vector<long long> delta(R);
    for (int r = 0; r < R; ++r) {
        if (!peer_arenas[r] || (reinterpret_cast<uintptr_t>(peer_arenas[r]) & (kAlign - 1)) != 0) return UBEP_ERR_ARENA;
        delta[r] = (long long)(reinterpret_cast<intptr_t>(peer_arenas[r]) - reinterpret_cast<intptr_t>(buf->arena));
    }
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaError_t e = cudaMemcpyAsync(buf->arena + buf->lay.peer_delta, delta.data(), sizeof(long long) * R,
                                    cudaMemcpyHostToDevice, buf->last_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(buf->last_stream);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    buf->my_rank = my_rank;
    return UBEP_OK;
}

int ubep_dispatch_sharded(ubep_buffer_t* buf, const void* x_local, const int32_t* topk_idx, const float* topk_w,
                          int32_t T, void* cuda_stream) {
    if (!buf || buf->my_rank < 0) return UBEP_ERR_ARG;
    if (T < 0 || T > buf->cfg.max_tokens) return UBEP_ERR_ARG;
    if (T > 0 && (!topk_idx || !topk_w)) return UBEP_ERR_ARG;
    if (!aligned16(x_local) || !aligned16(topk_idx) || !aligned16(topk_w)) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    buf->last_stream = st;
    if (T == 0) {
        const size_t lo = buf->lay.off[UBEP_VIEW_CNT], hi = buf->lay.off[UBEP_VIEW_SLOT_ROW];
        cudaError_t e0 = cudaMemsetAsync(buf->arena + lo, 0, hi - lo, st);
        return e0 == cudaSuccess ? UBEP_OK : cuda_fail(buf, e0);
    }
    Params p = make_params(buf, T);
    const int R = buf->cfg.num_ranks;
    p.tok0 = (int)((int64_t)buf->my_rank * T / R);
    p.tok1 = (int)((int64_t)(buf->my_rank + 1) * T / R);
    if (p.tok1 > p.tok0 && !x_local) return UBEP_ERR_ARG;
    p.x = static_cast<const uint16_t*>(x_local);
    p.topk_idx = topk_idx;
    p.topk_w = topk_w;
    p.trace = nullptr;
    p.parts = 1;
    p.grid = p.nchunks;
    ubep::SmemPlan pl{};
    const bool whole_table = (int64_t)T * buf->cfg.topk <= kLocalMaxSlots &&
                             ubep::plan_dispatch(p, UBEP_PIPELINE_LOCAL, buf->max_smem - ubep::sharded_extra_smem(p), &pl) == 0;
    cudaError_t e;
    if (whole_table) {
        e = ubep::launch_sharded_dispatch(p, pl, true, st);
        g_launches += 1;
    } else {
        // A table too large to recount in every CTA: TokenCnt and CalCumSum as launches of their own over the
        // whole (all-gathered) table -- every rank still derives every count alone, nothing is exchanged --
        // cut into R * m chunks so that no chunk straddles two ranks; m CTAs then move this rank's rows.
        const int m = buf->lay.nchunks / R;
        if (m < 1) return UBEP_ERR_ARG;   // more ranks than persistent CTAs
        p.nchunks = R * m;
        p.grid = m;
        p.trace = nullptr;
        if (ubep::plan_dispatch(p, UBEP_PIPELINE_PHASED, buf->max_smem - ubep::sharded_extra_smem(p), &pl) != 0)
            return UBEP_ERR_ARG;
        e = ubep::launch_count_scan(p, pl, st);
        if (e == cudaSuccess) e = ubep::launch_sharded_dispatch(p, pl, false, st);
        g_launches += 3;
    }
    if (e != cudaSuccess) return cuda_fail(buf, e);
    return UBEP_OK;
}

int ubep_wait_arrivals(ubep_buffer_t* buf, void* cuda_stream) {
    if (!buf || buf->my_rank < 0) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    buf->last_stream = st;
    cudaError_t e = ubep::launch_wait_arrivals(at<unsigned>(buf, buf->lay.off[UBEP_VIEW_SHARD_ARRIVAL]),
                                               at<int32_t>(buf, buf->lay.status), st);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    g_launches += 1;
    return UBEP_OK;
}

int ubep_combine_sharded(ubep_buffer_t* buf, const void* const* y_peers, const float* topk_w, int32_t T,
                         void* out_local, void* cuda_stream) {
    if (!buf || buf->my_rank < 0 || T < 0 || T > buf->cfg.max_tokens) return UBEP_ERR_ARG;
    if (T == 0) return UBEP_OK;
    const int R = buf->cfg.num_ranks;
    const int tok0 = (int)((int64_t)buf->my_rank * T / R), tok1 = (int)((int64_t)(buf->my_rank + 1) * T / R);
    if (!y_peers || !topk_w || (tok1 > tok0 && !out_local)) return UBEP_ERR_ARG;
    if (!aligned16(topk_w) || !aligned16(out_local) || (reinterpret_cast<uintptr_t>(y_peers) & 7u) != 0) return UBEP_ERR_ARG;
    if (tok1 == tok0) return UBEP_OK;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    buf->last_stream = st;
    cudaError_t e = ubep::launch_sharded_combine(reinterpret_cast<const uint16_t* const*>(y_peers),
                                                 at<int32_t>(buf, buf->lay.slot_pos), topk_w, tok0, tok1,
                                                 buf->cfg.hidden, buf->cfg.topk, buf->cfg.rows_per_rank_cap,
                                                 static_cast<uint16_t*>(out_local), buf->num_sms, st);
    if (e != cudaSuccess) return cuda_fail(buf, e);
    g_launches += 1;
    return UBEP_OK;
}

int ubep_view(ubep_buffer_t* buf, int which, void** dev_ptr, int64_t shape[4]) {
    if (!buf || !dev_ptr || !shape || which < 0 || which >= UBEP_VIEW_COUNT_) return UBEP_ERR_ARG;
    const ubep_config_t& c = buf->cfg;
    const ArenaLayout& a = buf->lay;
    const int64_t R = c.num_ranks, E = c.num_experts, cap = c.rows_per_rank_cap, k = c.topk, S = a.S;
    int64_t s[4] = {1, 1, 1, 1};
    bool present = true;
    switch (which) {
        case UBEP_VIEW_RECV_X: s[0] = R; s[1] = cap; s[2] = a.rowB; break;
        case UBEP_VIEW_RECV_SCALE: s[0] = R; s[1] = cap; s[2] = a.G; present = c.payload != 0; break;
        case UBEP_VIEW_RECV_SRC_IDX: s[0] = R; s[1] = cap; break;
        case UBEP_VIEW_RECV_WEIGHT: s[0] = R; s[1] = cap; present = !c.dedup; break;
        case UBEP_VIEW_RECV_TOPK_IDX:
        case UBEP_VIEW_RECV_TOPK_W: s[0] = R; s[1] = cap; s[2] = k; present = c.dedup != 0; break;
        case UBEP_VIEW_EXPERT_ROWS: s[0] = R; s[1] = a.er_cap; present = c.dedup != 0; break;
        case UBEP_VIEW_CNT:
        case UBEP_VIEW_SRC_OFFSET: s[0] = S; s[1] = E; break;
        case UBEP_VIEW_EXPERT_OFFSET:
        case UBEP_VIEW_NUM_TOKENS_PER_EXPERT: s[0] = E; break;
        case UBEP_VIEW_NUM_ROWS_PER_RANK:
        case UBEP_VIEW_NUM_TOKENS_PER_RANK: s[0] = R; break;
        case UBEP_VIEW_SLOT_ROW: s[0] = c.max_tokens; s[1] = k; break;
        case UBEP_VIEW_ARRIVAL: s[0] = 2; s[1] = R; break;
        case UBEP_VIEW_EPOCH: s[0] = 1; break;
        case UBEP_VIEW_TRACE: s[0] = a.nchunks; s[1] = ubep::kTraceSlots; break;
        case UBEP_VIEW_SHARD_ARRIVAL: s[0] = 2; break;
        default: return UBEP_ERR_ARG;
    }
    if (!present) {
        *dev_ptr = nullptr;
        for (int i = 0; i < 4; ++i) shape[i] = 0;
        return UBEP_OK;
    }
    *dev_ptr = buf->arena + a.off[which];
    for (int i = 0; i < 4; ++i) shape[i] = s[i];
    return UBEP_OK;
}

int ubep_status(ubep_buffer_t* buf, int32_t* last_async_status) {
    if (!buf || !last_async_status) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    int32_t v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, buf->arena + buf->lay.status, sizeof(v), cudaMemcpyDeviceToHost,
                                    buf->last_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(buf->last_stream);
    if (e == cudaSuccess && v != 0) {
        e = cudaMemsetAsync(buf->arena + buf->lay.status, 0, sizeof(v), buf->last_stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(buf->last_stream);
    }
    if (e != cudaSuccess) return cuda_fail(buf, e);
    if (v != 0) buf->sp_dirty = true;   // a call that gave up may not have put every sentinel back
    *last_async_status = v;
    return UBEP_OK;
}

uint32_t ubep_epoch(const ubep_buffer_t* buf) { return buf ? buf->epoch : 0; }

uint64_t ubep_launch_count(void) { return g_launches.load(); }

int ubep_debug_withhold_flag(ubep_buffer_t* buf, int32_t chunk) {
    if (!buf || chunk < -1 || chunk >= buf->lay.nchunks) return UBEP_ERR_ARG;
    buf->withhold = chunk;
    return UBEP_OK;
}

int ubep_debug_trace(ubep_buffer_t* buf, int32_t enable) {
    if (!buf) return UBEP_ERR_ARG;
    buf->tracing = enable != 0;
    return UBEP_OK;
}

int ubep_debug_set_quant_warps(ubep_buffer_t* buf, int32_t n) {
    if (!buf || n < 1 || n > ubep::kWarps - 2) return UBEP_ERR_ARG;
    buf->quant_warps = n;
    return UBEP_OK;
}

int ubep_debug_set_count_warps(ubep_buffer_t* buf, int32_t n) {
    if (!buf || n < -1 || n > ubep::kWarps - 3) return UBEP_ERR_ARG;
    buf->count_warps = n;
    return UBEP_OK;
}

int ubep_debug_set_prefetch_rows(ubep_buffer_t* buf, int32_t n) {
    if (!buf || n < 1) return UBEP_ERR_ARG;
    buf->prefetch_rows = n;
    return UBEP_OK;
}

int ubep_debug_empty_launch(ubep_buffer_t* buf, int32_t ahead, void* cuda_stream) {
    if (!buf) return UBEP_ERR_ARG;
    DeviceGuard guard(buf->cfg.device);
    if (guard.err != cudaSuccess) return cuda_fail(buf, guard.err);
    cudaError_t e = ubep::launch_empty(buf->num_sms, ahead != 0, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(buf, e);
    g_launches += 1;
    return UBEP_OK;
}

const char* ubep_last_cuda_error(const ubep_buffer_t* buf) { return buf ? buf->cuda_error.c_str() : ""; }

const char* ubep_strerror(int code) {
    switch (code) {
        case UBEP_OK: return "ok";
        case UBEP_ERR_ARG: return "invalid argument";
        case UBEP_ERR_CUDA: return "CUDA runtime error";
        case UBEP_ERR_CAPACITY: return "a receive region needs more rows than rows_per_rank_cap";
        case UBEP_ERR_TIMEOUT: return "a bounded wait on a readiness flag ran out";
        case UBEP_ERR_BAD_INDEX: return "expert id out of range, or an expert named twice by one token";
        case UBEP_ERR_ARENA: return "arena too small or misaligned";
        case UBEP_ERR_CHECKSUM: return "marker sum of a receive region differs from the announced checksum";
        default: return "unknown error";
    }
}

}  // extern "C"
