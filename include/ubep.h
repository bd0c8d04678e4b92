/*
 * ubep.h -- C ABI of the B200 (sm_100a) MoE token dispatch / combine library.
 *
 * The expert-parallel ranks are virtual: R disjoint receive regions inside one device
 * arena that the caller allocates.  The library allocates no device memory, creates no
 * stream and synchronises the host only where a call says so (ubep_status, and the set-up
 * calls ubep_set_dest_order, ubep_set_peers, ubep_sync_attach, ubep_sync_scan_sentinel).
 * Every pointer below is marked [host] or [dev]; all device pointers must be 16-byte aligned;
 * `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *
 * Notation: T tokens, H hidden size, E physical experts, R ranks, L = E / R experts per
 * rank (expert p lives on rank p / L), k = top-k, S source ranks (token t belongs to the
 * source rank s with floor(s*T/S) <= t < floor((s+1)*T/S)), cap = rows_per_rank_cap.
 *
 * All functions return UBEP_OK (0) or a negative error code.  Argument errors are
 * reported synchronously and nothing is launched.  Conditions found on the device
 * (a region overflowing its capacity, a bounded flag wait running out, an expert id out
 * of range or repeated within a token) never trap: the kernel records the first such code in a device status word,
 * skips the offending access and returns; ubep_status() reads and clears that word.
 */
#ifndef UBEP_H
#define UBEP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ubep_buffer ubep_buffer_t; /* opaque host-side bookkeeping, library-owned */

enum {
    UBEP_OK = 0,
    UBEP_ERR_ARG = -1,       /* null / misaligned pointer, size out of range, bad config      */
    UBEP_ERR_CUDA = -2,      /* a CUDA runtime call failed (see ubep_last_cuda_error)         */
    UBEP_ERR_CAPACITY = -3,  /* device: a region needs more than cap rows; extra rows dropped */
    UBEP_ERR_TIMEOUT = -4,   /* device: a bounded wait on a readiness flag ran out            */
    UBEP_ERR_BAD_INDEX = -5, /* device: an expert id outside [-1, E), or an expert named a    */
                             /* second time by one token, was treated as an empty slot        */
    UBEP_ERR_ARENA = -6,     /* arena too small or not 256-byte aligned                       */
    UBEP_ERR_CHECKSUM = -7   /* device: the marker sum a receiver computed differs from the   */
                             /* checksum its senders announced (ubep_dispatch_sync, DC)       */
};

enum { UBEP_PAYLOAD_BF16 = 0, UBEP_PAYLOAD_FP8_E4M3 = 1 };

/* How ubep_dispatch schedules its steps. */
enum {
    UBEP_PIPELINE_AUTO = 0,   /* LOCAL for small routing tables (how small depends on whether */
                              /* the one-row-per-rank fast path applies), else FUSED          */
    UBEP_PIPELINE_PHASED = 1, /* count -> prefix sums -> scatter as three launches; the        */
                              /* kernel boundaries play the role of the global barriers of    */
                              /* the bulk-synchronous dispatch (Sec. 2.3, phases 2-5)         */
    UBEP_PIPELINE_FUSED = 2,  /* one persistent kernel: count / prefix-sum warps publish      */
                              /* offsets through release/acquire flags while mover warps      */
                              /* already stream rows (kernel decomposition, Sec. 3.2).  Its   */
                              /* CTAs wait for one another, so all num_ctas of them must be   */
                              /* resident at once: the kernel is launched cooperatively, the  */
                              /* launch fails (UBEP_ERR_CUDA) if the grid cannot fit on the   */
                              /* device, and it starts only when every CTA has an SM -- a     */
                              /* caller that keeps SMs busy on other streams should create    */
                              /* the buffer with a smaller num_ctas                           */
    UBEP_PIPELINE_LOCAL = 3   /* one persistent kernel in which every CTA derives its offsets */
                              /* from the whole routing table itself (no flags; small T*k:    */
                              /* asked for explicitly with a table that does not fit in       */
                              /* shared memory, ubep_dispatch returns UBEP_ERR_ARG)           */
};

typedef struct {
    int32_t num_ranks;         /* R >= 1                                                       */
    int32_t num_experts;       /* E physical experts, E % R == 0                               */
    int32_t hidden;            /* H, multiple of 8 (bf16 payload) or of 128 (FP8 payload)      */
    int32_t topk;              /* k in [1, 32]                                                 */
    int32_t max_tokens;        /* largest T any call will pass                                 */
    int32_t rows_per_rank_cap; /* cap: rows each receive region can hold                       */
    int32_t num_src_ranks;     /* S >= 1 (0 = R)                                               */
    int32_t payload;           /* UBEP_PAYLOAD_*                                               */
    int32_t dedup;             /* 0: one row per (token, slot), expert-major;                  */
                               /* 1: one row per (token, rank), ascending token                */
    int32_t device;            /* CUDA device ordinal                                          */
    int32_t pipeline;          /* UBEP_PIPELINE_*                                              */
    int32_t num_ctas;          /* persistent CTAs / token chunks; 0 = number of SMs (never     */
                               /* more: one CTA per SM, all resident at once).  The            */
                               /* bookkeeping of one chunk lives in shared memory: a dispatch  */
                               /* whose T / num_ctas tokens do not fit there (a few thousand   */
                               /* slots per CTA) returns UBEP_ERR_ARG and launches nothing     */
} ubep_config_t;

/* Arrays that live in the arena; ubep_view() returns their device address and shape. */
enum {
    UBEP_VIEW_RECV_X = 0,        /* u8  [R, cap, rowB]  rowB = 2H (bf16) or H (FP8)            */
    UBEP_VIEW_RECV_SCALE = 1,    /* f32 [R, cap, H/128] FP8 payload only                       */
    UBEP_VIEW_RECV_SRC_IDX = 2,  /* i32 [R, cap]        token id of each row                   */
    UBEP_VIEW_RECV_WEIGHT = 3,   /* f32 [R, cap]        gate weight of the row (dedup = 0)     */
    UBEP_VIEW_RECV_TOPK_IDX = 4, /* i32 [R, cap, k]     local expert id or -1  (dedup = 1)     */
    UBEP_VIEW_RECV_TOPK_W = 5,   /* f32 [R, cap, k]     weight or 0            (dedup = 1)     */
    UBEP_VIEW_EXPERT_ROWS = 6,   /* i32 [R, er_cap]     per local expert, at expert_offset,    */
                                 /*                     ascending rows selecting it (dedup = 1)*/
    UBEP_VIEW_CNT = 7,           /* i32 [S, E]          tokens of source s choosing expert p   */
    UBEP_VIEW_SRC_OFFSET = 8,    /* i32 [S, E]          expert_offset + sum_{s'<s} cnt         */
    UBEP_VIEW_EXPERT_OFFSET = 9, /* i32 [E]             exclusive sum of counts inside a rank  */
    UBEP_VIEW_NUM_TOKENS_PER_EXPERT = 10, /* i32 [E]                                           */
    UBEP_VIEW_NUM_ROWS_PER_RANK = 11,     /* i32 [R]    rows written to each region            */
    UBEP_VIEW_NUM_TOKENS_PER_RANK = 12,   /* i32 [R]    distinct tokens routed to each rank    */
    UBEP_VIEW_SLOT_ROW = 13,     /* i32 [max_tokens, k] region-local row of each slot, or -1;  */
                                 /*                     the handle ubep_combine uses           */
    UBEP_VIEW_ARRIVAL = 14,      /* u32 [2, R]          eighths of rows landed per region (a   */
                                 /*                     region is complete at 8 * its row      */
                                 /*                     count); the n-th dispatch uses half    */
                                 /*                     (n & 1)                                */
    UBEP_VIEW_EPOCH = 15,        /* u32 [1]             dispatches completed on this buffer;   */
                                 /*                     readiness flags hold this count + 1    */
                                 /*                     while a dispatch runs, so replaying a  */
                                 /*                     captured CUDA graph needs no reset     */
    UBEP_VIEW_TRACE = 16,        /* u64 [chunks, 16]    per-CTA phase time stamps in ns of the */
                                 /*                     last traced dispatch (ubep_debug_trace)*/
    UBEP_VIEW_SHARD_ARRIVAL = 17,/* u32 [2]             sharded use: rows announced to this    */
                                 /*                     rank's region so far, rows expected so */
                                 /*                     far (both modulo 2^32, never reset)    */
    UBEP_VIEW_COUNT_ = 18
};

/*
 * Bytes of device memory the arena needs for this configuration (0 if the configuration
 * is invalid).  Operation: the receive address space is partitioned once, at
 * initialisation, so that senders can store rows straight into the destination's memory
 * (Sec. 4, "Global Load/Store for Point-to-Point Synchronization"; Sec. 2.3).
 */
size_t ubep_buffer_bytes(const ubep_config_t *cfg /*[host]*/);

/*
 * Lay the arrays out inside `dev_arena` ([dev], 256-byte aligned, >= ubep_buffer_bytes)
 * and zero the flag words (one synchronous memset).  The caller keeps ownership of the
 * arena and must keep it alive until ubep_buffer_destroy.  *out receives the handle.
 */
int ubep_buffer_create(const ubep_config_t *cfg /*[host]*/, void *dev_arena /*[dev]*/,
                       size_t bytes, ubep_buffer_t **out /*[host]*/);

/* Free the host bookkeeping.  The arena is the caller's and is not touched. */
int ubep_buffer_destroy(ubep_buffer_t *buf);

/*
 * Logical -> physical expert table for replicated experts (the paper only names expert
 * replication as an upper-layer strategy the library accepts, Sec. 6).  Slot (t, j) with
 * logical id l goes to phys[l][t mod ncopies[l]].  phys [dev] is [E_log, C] int32,
 * ncopies [dev] is [E_log] int32; both stay owned by the caller and must outlive the calls
 * that use them.  Passing NULLs removes the table.
 */
int ubep_set_replicas(ubep_buffer_t *buf, const int32_t *phys /*[dev]*/,
                      const int32_t *ncopies /*[dev]*/, int32_t E_log, int32_t C);

/*
 * Destination-ordering table (Sec. 3.3: the re-mapped expert sequence each worker sends
 * in).  `order` [host] is a permutation of 0..R-1; worker w issues the copies of one row
 * in the table's order rotated by w.  Results never depend on it.  NULL = no table: the
 * copies of a row are issued in slot order, which saves the ordering step of every dispatch
 * (on one GPU all destinations are the same memory, so the order changes nothing measurable).
 */
int ubep_set_dest_order(ubep_buffer_t *buf, const int32_t *order /*[host] [R]*/);

/*
 * TokenCnt only (Sec. 3.2; Sec. 2.3: ranges follow from per-expert counts): counts how
 * many distinct tokens go to each rank and how many tokens select each expert, and marks
 * which ranks each token visits.  topk_idx [dev] int32 [T, k] (expert id, or -1 = empty
 * slot; the ids of one token are distinct -- a repeated id is reported as UBEP_ERR_BAD_INDEX
 * and the later slot counts as empty).  Outputs [dev], caller-owned:
 * num_tokens_per_rank [R], num_tokens_per_expert [E], is_token_in_rank u8 [T, R]
 * (any of them may be NULL).  One launch on `cuda_stream`.
 */
int ubep_get_dispatch_layout(ubep_buffer_t *buf, const int32_t *topk_idx /*[dev]*/, int32_t T,
                             int32_t *num_tokens_per_rank /*[dev]*/,
                             int32_t *num_tokens_per_expert /*[dev]*/,
                             uint8_t *is_token_in_rank /*[dev]*/, void *cuda_stream);

/*
 * Counts without any caller-provided scratch (the paper has no counterpart; this entry
 * point exists for callers that may not allocate).  Same results as
 * ubep_get_dispatch_layout, but it needs no buffer handle and no arena: a caller that
 * runs inside somebody else's memory plan -- a plugin handed fixed input and output
 * tensors, code running while allocation is forbidden -- cannot reserve an arena, so the
 * chunk histograms live in a fixed array of UBEP_STATIC_MAX_BINS x 64 32-bit words
 * (about 257 KB) inside the library's device image.  Every GPU that loads the library holds
 * that array until the process exits.
 *
 * Limits: num_experts + num_ranks <= UBEP_STATIC_MAX_BINS, topk <= 32, num_experts %
 * num_ranks == 0; anything larger returns UBEP_ERR_ARG and launches nothing.  No replica
 * table; expert ids outside [-1, num_experts) are skipped.  topk_idx [dev] int32 [T, topk],
 * 16-byte aligned; outputs [dev] as for ubep_get_dispatch_layout (any may be NULL).
 *
 * The first call on each device looks up the array's device address (with that device
 * current) and keeps it; make that first call before any stream capture begins.  The call
 * itself calls no cudaMalloc, cudaFree or other allocating routine.  All calls on a device
 * share the one array: calls whose kernels may overlap on the GPU (different streams) race
 * on it -- keep them on one stream or otherwise ordered.  The array keeps the previous
 * call's contents; the kernel overwrites what it reads and re-arms its own counter.
 */
#define UBEP_STATIC_MAX_BINS 1024
int ubep_get_dispatch_layout_static(const int32_t *topk_idx /*[dev]*/, int32_t T, int32_t topk,
                                    int32_t num_experts, int32_t num_ranks,
                                    int32_t *num_tokens_per_rank /*[dev]*/,
                                    int32_t *num_tokens_per_expert /*[dev]*/,
                                    uint8_t *is_token_in_rank /*[dev]*/, void *cuda_stream);

/*
 * Dispatch (Sec. 2.3 phases 1-5 fused as in Sec. 3.2): counts, prefix-sum offsets, row
 * assignment, optional FP8 quantisation, and the copy of every token row into the receive
 * regions of the ranks that host its experts.  x [dev] bf16 [T, H]; topk_idx [dev] int32
 * [T, k]; topk_w [dev] fp32 [T, k].  Results land in the arena (ubep_view).  Rows at or
 * beyond a region's row count are not written.  An id outside [-1, E) and the second
 * occurrence of an expert within one token are reported (UBEP_ERR_BAD_INDEX) and handled as
 * if the slot held -1: every output equals that of the corrected table.  Asynchronous on `cuda_stream`; calls on
 * one buffer must be stream-ordered.
 */
int ubep_dispatch(ubep_buffer_t *buf, const void *x /*[dev]*/, const int32_t *topk_idx /*[dev]*/,
                  const float *topk_w /*[dev]*/, int32_t T, void *cuda_stream);

/*
 * Combine (Sec. 2.3: gathers expert outputs and restores the original token order):
 * out[t] = bf16( sum_j topk_w[t][j] * y[rank of slot j][slot_row[t][j]] ), fp32
 * accumulation in slot order with one fused multiply-add per slot.  y [dev] bf16
 * [R, cap, H] is caller-owned and indexed like the receive regions; out [dev] bf16
 * [T, H].  Uses the slot_row handle left by the last ubep_dispatch on this buffer.
 */
int ubep_combine(ubep_buffer_t *buf, const void *y /*[dev]*/, const float *topk_w /*[dev]*/,
                 int32_t T, void *out /*[dev]*/, void *cuda_stream);

/*
 * Token-level load partition with the prefix-sum search of Algorithm 1 (Sec. 3.3): the send
 * sequence is the experts in the order `order` ([dev] int32 [n], ids in [0, num_experts)),
 * expert e contributing counts[e] tokens ([dev] int32 [num_experts]).  It is cut into
 * n_workers contiguous slices whose sizes differ by at most one token; worker w starts at
 * global token floor(w * total / n_workers).  Outputs ([dev], caller-owned, n_workers + 1
 * entries each; entry n_workers closes the last slice): start_pos[w] = position in `order`
 * of the expert whose cumulative range covers that token (n if the worker has no work),
 * start_off[w] = offset inside that expert (int64), iters[w] = search iterations (may be
 * NULL).  One launch of one CTA on `cuda_stream`; ids of `order` out of range count as empty.
 */
int ubep_map_workers(const int32_t *order /*[dev]*/, const int32_t *counts /*[dev]*/, int32_t n,
                     int32_t num_experts, int32_t n_workers, int32_t *start_pos /*[dev]*/,
                     int64_t *start_off /*[dev]*/, int32_t *iters /*[dev]*/, void *cuda_stream);

/* ----------------------------------------------------------------------------------------
 * Readiness protocols (Sec. 3.4, "Data-as-Flag Synchronization").
 *
 * ubep_dispatch_sync is a second dispatch path in which the way a receiver learns that its
 * rows have landed is the protocol under study.  Every CTA of one persistent kernel first
 * sends the rows of its tokens (sender role) and then, for the receive region it is given,
 * waits until the protocol says that all expected rows are there (receiver role).  The four
 * protocols differ only in what the sender adds to the data and in what the receiver looks at:
 *
 *   SW   stop-and-wait, the scheme Data-as-Flag replaces: rows are stored into the region,
 *        then a fence, then one release-add per row on a counter of the region; the receiver
 *        waits for the counter to reach the region's row count.
 *   TFF  Token-Flag Fusion: every DataBlock carries a leading flag.  A B200 thread can store
 *        16 bytes as one access, not 512, so a DataBlock is UBEP_SYNC_BLOCK_BYTES = 16 bytes:
 *        a 4-byte flag (the sequence number of the call) and 12 bytes of payload, written with
 *        one 128-bit store into a wire buffer (payload efficiency 12/16 against the paper's
 *        480/512).  The receiver polls each block's flag, and moves the payload of arrived
 *        blocks into the region.  No fence and no counter on the sender side.
 *   DC   Data-for-Checksum: rows are stored into the region unchanged; the leading
 *        UBEP_SYNC_DC_MARKER_BYTES = 32 bytes of every UBEP_SYNC_DC_BLOCK_BYTES = 512 bytes
 *        of a row are its markers.  After its last row every sender adds, per region, the sum
 *        of the markers it sent (little-endian 64-bit words, modulo 2^64 -- the paper does not
 *        name the sum) to the region's checksum word and announces itself (one fence per
 *        sender and batch).  The receiver waits for all announcements, sums the markers it
 *        finds in its region and compares; a difference is reported as UBEP_ERR_CHECKSUM.
 *   SP   Sentinel Polling: the wire buffer of every region is pre-filled with the sentinel
 *        (bf16 code 0xFFFF, a NaN pattern no rounding of a number yields, in every element);
 *        rows are stored into it unchanged with 128-bit stores.  The receiver polls every
 *        16-byte block until it differs from the sentinel, moves it into the region and puts
 *        the sentinel back.  A 16-byte block of the input that equals the sentinel is never
 *        seen to arrive: the wait runs out and UBEP_ERR_TIMEOUT is reported
 *        (ubep_sync_scan_sentinel counts such blocks beforehand).
 *
 * The protocols assume that a naturally aligned 16-byte store of one thread becomes visible
 * as a whole, which holds on this hardware but is stronger than what the PTX memory model
 * promises for vector accesses.  All waits are bounded (about 1.5 s); a wait that runs out
 * records UBEP_ERR_TIMEOUT and the kernel returns.
 *
 * FP8 rows (UBEP_PAYLOAD_FP8_E4M3) travel quantised: the sender quantises a row once, and a wire row is
 * the H payload bytes followed by the 4 * H / 128 bytes of its scales (the W8A8 rows of the paper's
 * Table 3); Token-Flag blocks and Sentinel blocks are cut from that, the checksum markers from the
 * payload.  What arrives goes to the region's payload and scale arrays.
 *
 * Routing tables of any size: up to 8192 slots (T * k), and while the table with the bitmaps of all its
 * bins (T x (E + R) bits) fits in a CTA's shared memory, every CTA derives the layout from the whole
 * table, as UBEP_PIPELINE_LOCAL does (one launch); for a larger table the counting and prefix-sum
 * kernels of UBEP_PIPELINE_PHASED run in front of the protocol kernel (three launches).  One CTA per SM at most, launched
 * cooperatively (receivers wait for senders of the same grid, so the grid must be resident at once:
 * a grid that cannot be is refused with UBEP_ERR_CUDA instead of running into its timeouts).  Everything
 * ubep_dispatch leaves in the arena is left here too, with identical contents; ubep_combine
 * may follow.  The arrival counters of ubep_dispatch (UBEP_VIEW_ARRIVAL) are not touched.
 */
enum { UBEP_SYNC_SW = 0, UBEP_SYNC_TFF = 1, UBEP_SYNC_DC = 2, UBEP_SYNC_SP = 3 };
#define UBEP_SYNC_BLOCK_BYTES 16
#define UBEP_SYNC_FLAG_BYTES 4
#define UBEP_SYNC_DC_BLOCK_BYTES 512
#define UBEP_SYNC_DC_MARKER_BYTES 32
#define UBEP_SYNC_SENTINEL 0xFFFFu

/* Arrays of the wire buffer (ubep_sync_view). */
enum {
    UBEP_SYNC_VIEW_TFF_WIRE = 0, /* u8  [R, cap, 16 * ceil(W / 12)]  DataBlocks of every row; W = 2H, */
                                 /*     or H + 4 * H / 128 for FP8 rows                           */
    UBEP_SYNC_VIEW_SP_WIRE = 1,  /* u8  [R, cap, W rounded up to 16]  all sentinel between calls  */
    UBEP_SYNC_VIEW_CHECKSUM = 2, /* u64 [2, R]  DC: marker sums announced (half = call number & 1)*/
    UBEP_SYNC_VIEW_COUNTERS = 3, /* u32 [4, R]  DC announcements [2, R], then SW row counts [2, R]*/
    UBEP_SYNC_VIEW_TIMES = 4,    /* u64 [CTAs, 8]  device nanosecond timer of the last call, per CTA:
                                    0 kernel entry, 1 layout done, 2 last row sent, 3 receiver duty
                                    confirmed (= 2 for a CTA without one), 4 exit; 5-7 unused      */
    UBEP_SYNC_VIEW_SEQ = 5,      /* u32 [1]  number of ubep_dispatch_sync kernels that have run   */
    UBEP_SYNC_VIEW_COUNT_
};

/* Bytes of the wire buffer for this configuration (0 if it is invalid). */
size_t ubep_sync_wire_bytes(const ubep_config_t *cfg /*[host]*/);

/*
 * Gives the buffer a wire buffer ([dev], 256-byte aligned, at least ubep_sync_wire_bytes,
 * caller-owned, must outlive the buffer's last ubep_dispatch_sync) and initialises it on
 * `cuda_stream`: flags and counters zero, SP wire all sentinel.  Waits for the stream.
 */
int ubep_sync_attach(ubep_buffer_t *buf, void *dev_wire /*[dev]*/, size_t bytes, void *cuda_stream);

/*
 * Dispatch with readiness protocol `protocol` (UBEP_SYNC_*); arguments as ubep_dispatch.
 * One kernel launch, three for large routing tables (a memset before it when an earlier call left the SP wire dirty, which
 * the library learns when ubep_status reports that call's error; until then a word on the
 * device makes every Sentinel Polling call on that wire report UBEP_ERR_TIMEOUT and move nothing).  UBEP_ERR_ARG if no wire
 * buffer is attached or T exceeds the buffer's max_tokens.
 */
int ubep_dispatch_sync(ubep_buffer_t *buf, int protocol, const void *x /*[dev]*/,
                       const int32_t *topk_idx /*[dev]*/, const float *topk_w /*[dev]*/, int32_t T,
                       void *cuda_stream);

/* Device address and shape of one wire-buffer array; valid while the wire buffer is. */
int ubep_sync_view(ubep_buffer_t *buf, int which, void **dev_ptr /*[host]*/, int64_t shape[4] /*[host]*/);

/*
 * The check Sec. 3.4 asks for before Sentinel Polling is trusted: counts the 16-byte blocks
 * of x ([dev] bf16 [T, H]) that equal the sentinel into *count ([host]).  Runs on
 * `cuda_stream` and waits for it.  Needs an attached wire buffer (its counter word).
 */
int ubep_sync_scan_sentinel(ubep_buffer_t *buf, const void *x /*[dev]*/, int32_t T, int64_t *count /*[host]*/,
                            void *cuda_stream);

/* ----------------------------------------------------------------------------------------
 * Ranks on different GPUs (Sec. 2.3 and Sec. 4, "Global Load/Store for Point-to-Point
 * Synchronization"): rank r is GPU r, S = R, every GPU holds an arena of the same
 * configuration (hence the same layout) in memory its peers can address -- peer-to-peer
 * mappings over NVLink, which the caller sets up and passes in as plain device pointers.
 * Receive region r is used in arena r only.  One buffer handle per GPU and process.
 *
 * A dispatch of the global batch of T tokens then is, on every rank s:
 *   1. (caller) all-gather of the routing table, so that every rank holds topk_idx and
 *      topk_w of all T tokens -- 8 bytes per slot against 2H bytes per row;
 *   2. ubep_dispatch_sharded: the rank derives the whole layout from the table (every rank
 *      gets the same counts and offsets, each into its own arena), and stores the rows of its
 *      own tokens, floor(s*T/R) <= t < floor((s+1)*T/R), and their metadata straight into the
 *      regions of the ranks that host their experts (plain 128-bit stores to peer memory; no
 *      multicast, no collective).  Then one system-scope fence and one release-add per
 *      destination rank on that rank's arrival word;
 *   3. ubep_wait_arrivals: a one-CTA kernel that waits (bounded, about 1.5 s, then
 *      UBEP_ERR_TIMEOUT) until the local arrival word has reached the number of rows this
 *      rank's region receives.  The arrival words only grow (modulo 2^32); nothing is reset
 *      between calls, so a fast peer can never have its announcement wiped out.
 * ubep_combine_sharded gathers, for the rank's own tokens, expert-output rows from the ranks
 * that produced them with plain loads from peer memory.
 *
 * The caller orders the steps across ranks where data is reused: no rank may start dispatch
 * n + 1 before every rank has finished reading what dispatch n delivered, and no rank may
 * start combine before the y of every peer is complete (a barrier on the streams, e.g. an
 * NCCL one).  A table of up to 8192 slots is recounted by every CTA (one launch); a larger one --
 * or one whose bitmaps do not fit in a CTA's shared memory -- goes through two launches that count and
 * prefix-sum the whole table, in chunks that do not straddle ranks, and a third that moves the
 * rank's rows with (persistent CTAs / R) CTAs; R may not exceed the number of persistent CTAs then
 * (else UBEP_ERR_ARG).  No count is exchanged either way.  Both payloads (FP8 rows are
 * quantised by the sender; scales land in the receiver's scale array).  Kernels of different
 * ranks never wait for one another except in ubep_wait_arrivals, which therefore must not be
 * emulated by launches queued on one GPU ahead of the senders it waits for.
 */

/*
 * Puts the buffer in sharded use.  peer_arenas [host]: R device pointers, entry r = the
 * arena of rank r as this GPU addresses it (entry my_rank = the buffer's own arena).
 * Copies R offsets to the device on the stream of the last call and waits for it.
 */
int ubep_set_peers(ubep_buffer_t *buf, int32_t my_rank, void *const *peer_arenas /*[host]*/);

/*
 * Step 2 above.  x_local [dev] bf16 [T_local, H], the rank's own tokens in order; topk_idx,
 * topk_w [dev]: the table of all T tokens.  Asynchronous on `cuda_stream`.
 */
int ubep_dispatch_sharded(ubep_buffer_t *buf, const void *x_local /*[dev]*/, const int32_t *topk_idx /*[dev]*/,
                          const float *topk_w /*[dev]*/, int32_t T, void *cuda_stream);

/* Step 3 above: one small launch on `cuda_stream` after the rank's own ubep_dispatch_sharded. */
int ubep_wait_arrivals(ubep_buffer_t *buf, void *cuda_stream);

/*
 * out_local[t - t_begin] = bf16( sum_j topk_w[t][j] * y_r(j)[slot_row[t][j]] ) for the rank's
 * own tokens; same arithmetic as ubep_combine.  y_peers [dev]: R device pointers, entry r =
 * the expert-output buffer of rank r (bf16, laid out like the receive regions: [R, cap, H],
 * of which rank r fills region r) as this GPU addresses it.  topk_w [dev]: all T tokens.
 */
int ubep_combine_sharded(ubep_buffer_t *buf, const void *const *y_peers /*[dev]*/, const float *topk_w /*[dev]*/,
                         int32_t T, void *out_local /*[dev]*/, void *cuda_stream);

/* Device address and shape (unused dims = 1) of one arena array; valid until destroy. */
int ubep_view(ubep_buffer_t *buf, int which, void **dev_ptr /*[host]*/, int64_t shape[4] /*[host]*/);

/*
 * Synchronises the stream of the last call, copies the device status word to
 * *last_async_status ([host]; UBEP_OK or a UBEP_ERR_* code found on the device) and
 * clears it.
 */
int ubep_status(ubep_buffer_t *buf, int32_t *last_async_status /*[host]*/);

/* Number of non-empty dispatches issued through ubep_dispatch on this buffer so far
 * (graph replays are not counted; the device-side count is UBEP_VIEW_EPOCH). */
uint32_t ubep_epoch(const ubep_buffer_t *buf);

/* Kernels launched by this library since it was loaded (all buffers). */
uint64_t ubep_launch_count(void);

/*
 * Test hook for the bounded-wait path: the next ubep_dispatch skips the release store of
 * the readiness flag of token chunk `chunk` (-1 = none), so that the waits on it run out
 * after about a second, the kernel returns and ubep_status reports UBEP_ERR_TIMEOUT.
 */
int ubep_debug_withhold_flag(ubep_buffer_t *buf, int32_t chunk);

/*
 * Tracing (the paper reports per-task latency breakdowns, Sec. 5.3): when enabled, every
 * CTA of the following dispatches stamps the device nanosecond timer at its phase
 * boundaries into UBEP_VIEW_TRACE: 0 start, 1 counted, 2 all counts seen, 3 prefix sums
 * published, 4 all offsets seen, 5 rows assigned, 6 movers released, 7 first row in shared
 * memory, 8 last copy issued, 9 copies complete, 10 end.  Slots a CTA does not pass keep
 * their old value.
 */
int ubep_debug_trace(ubep_buffer_t *buf, int32_t enable);

/*
 * Warp-role split of the FP8 dispatch kernel (the paper's core-allocation question, Sec. 3.2
 * "most cores send tokens, a few compute token counts", and App. A / C: how many cores count and
 * how many send).  Of the CTA's 16 warps one loads rows and one issues the stores.
 *
 * ubep_debug_set_count_warps: n warps (the store issuer among them) form the count group that
 * computes the layout -- TokenCnt, the flag exchange, CalCumSum, row assignment -- while the
 * remaining 15 - n warps already quantise the rows the loader has fetched into a ring of
 * quantised rows that waits for the layout (1 <= n <= 13).  TokenCnt itself is done by all 15
 * warps first; the count group is what goes on through the flag exchange.  n = 0: all 15 warps
 * compute the layout and 14 of them quantise afterwards.  n = -1 (default): 8, or 0 when slices
 * are long enough for token stealing.  Applies to the PHASED and FUSED schedules; the flag-free
 * LOCAL schedule, whose layout waits for nobody, always runs as n = 0.
 * ubep_debug_set_quant_warps: at most n warps quantise (1 <= n <= 14, default 14), the rest idle.
 * ubep_debug_set_prefetch_rows: the loader fetches at most n rows before the layout is done
 * (default: as many as the rings hold).
 * Results never depend on any of them.
 */
int ubep_debug_set_quant_warps(ubep_buffer_t *buf, int32_t n);
int ubep_debug_set_count_warps(ubep_buffer_t *buf, int32_t n);
int ubep_debug_set_prefetch_rows(ubep_buffer_t *buf, int32_t n);

/*
 * Measurement aid: launches a kernel that does nothing (one small CTA per SM) on `cuda_stream`,
 * the ordinary way or, with ahead != 0, with programmatic stream serialization like the dispatch
 * and the small-batch combine kernels.  Timed in a chain it gives the floor that every kernel
 * boundary of a layer costs on this device.
 */
int ubep_debug_empty_launch(ubep_buffer_t *buf, int32_t ahead, void *cuda_stream);

/* Text of the last CUDA runtime error seen by this buffer's calls ("" if none). */
const char *ubep_last_cuda_error(const ubep_buffer_t *buf);

const char *ubep_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* UBEP_H */
