// Host-visible launchers of the kernels in ubep_kernels.cu.
#pragma once

#include <cuda_runtime.h>

#include "ubep_common.cuh"

namespace ubep {

// Shared-memory plan of the dispatch kernel (ring depth, offsets, total); -1 if the
// bookkeeping of this call does not fit beside a four-row ring.
int plan_dispatch(const Params& p, int mode, int max_smem, SmemPlan* out);

cudaError_t launch_count_scan(const Params& p, const SmemPlan& pl, cudaStream_t st);
cudaError_t launch_dispatch(const Params& p, int mode, const SmemPlan& pl, cudaStream_t st, int* launches);
cudaError_t launch_combine(const uint16_t* y, const int32_t* slot_pos, const float* topk_w, int T, int H, int k,
                           uint16_t* out, int num_sms, bool ahead, cudaStream_t st);
cudaError_t launch_empty(int num_sms, bool ahead, cudaStream_t st);
cudaError_t launch_layout(const Params& p, int32_t* num_tokens_per_rank, int32_t* num_tokens_per_expert,
                          uint8_t* is_token_in_rank, int32_t* scratch_hist, unsigned* ticket, cudaStream_t st);

}  // namespace ubep
