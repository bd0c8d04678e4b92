// Host-visible launchers of the kernels in ubep_kernels.cu.
#pragma once

#include <cuda_runtime.h>

#include "ubep_common.cuh"

namespace ubep {

// Ring depth, stage size and dynamic shared memory of the dispatch kernel; -1 if the
// chunk's bookkeeping does not fit beside a four-row ring.
int plan_dispatch(const Params& p, int max_smem, int* stages, int* stage_bytes, size_t* smem);

cudaError_t launch_dispatch(const Params& p, int mode, int stages, int stage_bytes, size_t smem, cudaStream_t st,
                            int* launches);
cudaError_t launch_combine(const uint16_t* y, const int32_t* slot_pos, const float* topk_w, int T, int H, int k,
                           uint16_t* out, int num_sms, cudaStream_t st);
cudaError_t launch_layout(const Params& p, int32_t* num_tokens_per_rank, int32_t* num_tokens_per_expert,
                          uint8_t* is_token_in_rank, int32_t* scratch_hist, unsigned* ticket, cudaStream_t st);

}  // namespace ubep
