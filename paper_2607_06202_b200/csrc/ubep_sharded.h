// Host-visible launchers of the kernels for ranks on different GPUs (ubep_sharded.cu).
#pragma once

#include <cuda_runtime.h>

#include "ubep_common.cuh"

namespace ubep {

// Dynamic shared memory the sharded dispatch kernel needs beyond the dispatch plan's total.
int sharded_extra_smem(const Params& p);

// whole_table: every CTA derives the layout from the whole routing table in shared memory; otherwise the
// count / prefix-sum launches (launch_count_scan) have run before with p.nchunks = R * p.grid chunks.
cudaError_t launch_sharded_dispatch(const Params& p, const SmemPlan& pl, bool whole_table, cudaStream_t st);

// One CTA: waits until arrival[0] (rows announced) equals arrival[1] (rows expected).
cudaError_t launch_wait_arrivals(const unsigned* arrival, int32_t* status, cudaStream_t st);

// Combine of tokens [tok0, tok1): row `where` = rank * cap + row is read from y_peers[rank].
cudaError_t launch_sharded_combine(const uint16_t* const* y_peers, const int32_t* slot_pos, const float* topk_w,
                                   int tok0, int tok1, int H, int k, int cap, uint16_t* out_local, int num_sms,
                                   cudaStream_t st);

}  // namespace ubep
