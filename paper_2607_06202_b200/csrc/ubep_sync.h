// Host-visible launchers of the readiness-protocol dispatch (ubep_sync.cu).
#pragma once

#include <cuda_runtime.h>

#include "ubep_common.cuh"

namespace ubep {

constexpr int kErrChecksum = -7;     // mirrors UBEP_ERR_CHECKSUM
constexpr int kSyncTimeSlots = 8;    // per-CTA time stamps of the last call

// Wire-buffer arrays and the protocol of one call.
struct SyncParams {
    int protocol;                   // UBEP_SYNC_*
    int tff_blocks;                 // 16-byte DataBlocks per row: ceil(rowB / 12)
    uint8_t* tff_wire;              // [R * cap][16 * tff_blocks]
    uint8_t* sp_wire;               // [R * cap][rowB]
    unsigned long long* checksum;   // [2][R]
    unsigned* announced;            // [2][R] senders that have added their marker sums
    unsigned* sw_rows;              // [2][R] rows whose stores have been fenced
    unsigned* seq_ctr;              // calls completed
    unsigned* seq_ticket;           // CTAs of the running call that have read seq_ctr
    unsigned* sp_dirty;             // != 0: a Sentinel Polling call gave up and may have left arrived blocks in the wire
    unsigned long long* times;      // [grid][kSyncTimeSlots]
};

// Dynamic shared memory the kernel needs beyond the dispatch plan's total.
int sync_extra_smem(const Params& p);

// whole_table: every CTA derives the layout from the whole routing table in shared memory; otherwise the
// count / prefix-sum launches (launch_count_scan) have run before over the same p.nchunks chunks.
cudaError_t launch_sync_dispatch(const Params& p, const SmemPlan& pl, const SyncParams& sp, bool whole_table,
                                 cudaStream_t st);

// Counts the 16-byte vectors of x that consist of 0xFFFF elements only.
cudaError_t launch_sentinel_scan(const void* x, long long n_vec, unsigned long long* count, int num_sms,
                                 cudaStream_t st);

}  // namespace ubep
