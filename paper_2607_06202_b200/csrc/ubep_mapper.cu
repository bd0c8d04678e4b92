// Token-level load partition of the hierarchical scheduler (Sec. 3.3 of the paper): the
// send sequence -- the experts in their re-mapped order, each with its token count -- is
// cut into equal contiguous slices, one per worker, and every worker finds where its slice
// starts with the quaternary prefix-sum search of Algorithm 1.
//
// One CTA builds the cumulative token counts C[0..n] of the re-mapped sequence in shared
// memory (block scan); one warp per worker then runs the search.  The three pivots of an
// iteration are evaluated side by side by three lanes (the paper evaluates them with one
// SIMD VectorCount); a ballot finds the quadrant.
//
// Reading of the printed algorithm: the loop runs while the window [lo, hi) holds more than
// one expert, gap = ceil((hi - lo) / 4), pivots lo + i * gap are clamped to hi, and the
// invariant C(lo) <= target < C(hi) is kept (as printed the gap never reaches 0 and pivots
// can pass the right end).
#include <cstdint>

#include "../../include/ubep.h"
#include "ubep_common.cuh"

namespace {

constexpr int kMapThreads = 1024;

__global__ void __launch_bounds__(kMapThreads) mapper_kernel(const int32_t* __restrict__ order,
                                                            const int32_t* __restrict__ counts, int n, int E,
                                                            int n_workers, int32_t* start_pos, int64_t* start_off,
                                                            int32_t* iters) {
    extern __shared__ long long cum[];   // cum[i] = tokens of the first i experts of the sequence
    __shared__ long long warp_tot[kMapThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // block-wide inclusive scan of counts[order[i]], kMapThreads entries per round
    long long carry = 0;
    if (tid == 0) cum[0] = 0;
    for (int base = 0; base < n; base += kMapThreads) {
        const int i = base + tid;
        long long v = 0;
        if (i < n) {
            const int e = order[i];
            if (e >= 0 && e < E) v = counts[e];   // ids out of range count as empty
        }
        long long incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long u = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += u;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        long long before = carry;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if (i < n) cum[i + 1] = before + incl;
        long long round_tot = 0;
        for (int w = 0; w < kMapThreads / 32; ++w) round_tot += warp_tot[w];
        carry += round_tot;
        __syncthreads();
    }
    const long long total = cum[n];
    for (int w = warp; w <= n_workers; w += kMapThreads / 32) {
        const long long target = (long long)w * total / n_workers;   // equal slices, sizes differ by <= 1
        int lo = 0, hi = n, it = 0;
        if (target >= total) {            // nothing left for this worker (also the closing entry w == n_workers)
            lo = n;
        } else {
            while (hi - lo > 1) {
                const int gap = (hi - lo + 3) / 4;
                // lane i in 1..3 evaluates pivot i; other lanes take the right end
                const int piv = min(lo + min(lane, 4) * gap, hi);
                const long long c = cum[piv];
                const unsigned below = __ballot_sync(0xffffffffu, lane >= 1 && lane <= 3 && target < c);
                // smallest q in 1..3 with target < C(pivot q), else 4
                const int q = below ? __ffs(below) - 1 : 4;
                const int new_lo = min(lo + (q - 1) * gap, hi);
                const int new_hi = q == 4 ? hi : min(lo + q * gap, hi);
                lo = new_lo;
                hi = new_hi;
                ++it;
            }
        }
        if (lane == 0) {
            start_pos[w] = lo;
            start_off[w] = lo < n ? target - cum[lo] : 0;
            if (iters) iters[w] = it;
        }
    }
}

}  // namespace

extern "C" int ubep_map_workers(const int32_t* order, const int32_t* counts, int32_t n, int32_t num_experts,
                                int32_t n_workers, int32_t* start_pos, int64_t* start_off, int32_t* iters,
                                void* cuda_stream) {
    if (!order || !counts || !start_pos || !start_off || n < 1 || num_experts < 1 || n_workers < 1) return UBEP_ERR_ARG;
    if ((size_t)(n + 1) * sizeof(long long) > 200 * 1024) return UBEP_ERR_ARG;
    const size_t smem = (size_t)(n + 1) * sizeof(long long);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(mapper_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return UBEP_ERR_CUDA;
    mapper_kernel<<<1, kMapThreads, smem, static_cast<cudaStream_t>(cuda_stream)>>>(
        order, counts, n, num_experts, n_workers, start_pos, start_off, iters);
    return cudaGetLastError() == cudaSuccess ? UBEP_OK : UBEP_ERR_CUDA;
}
