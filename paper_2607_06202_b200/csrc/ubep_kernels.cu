// Kernels of the dispatch / combine hot path for sm_100a.
//
//   count_kernel / scan_kernel        TokenCnt and CalCumSum as separate launches (the
//                                     bulk-synchronous pipeline; kernel boundaries = barriers)
//   dispatch_kernel<mode, fp8>        persistent CTA per token chunk: layout warps + a mover
//                                     warp that streams rows with TMA bulk copies; in fused
//                                     mode the layout steps are ordered by release/acquire
//                                     flags instead of launches (kernel decomposition)
//   combine_kernel<K>                 gather + fp32 weighted sum + one bf16 rounding
//   layout_kernel                     counts only (ubep_get_dispatch_layout)
#include <cuda_fp8.h>

#include "ubep_kernels.h"
#include "ubep_layout.cuh"

namespace ubep {

// --------------------------------------------------------------- phased: count / scan

__global__ void __launch_bounds__(32) count_kernel(const Params p) {
    extern __shared__ int sm_i[];
    count_chunk(p, blockIdx.x, sm_i, threadIdx.x);
}

__global__ void __launch_bounds__(256) scan_kernel(const Params p) {
    extern __shared__ int sm_i[];
    scan_rank(p, blockIdx.x, sm_i, threadIdx.x / 32, 8, threadIdx.x % 32, 1);
}

// ------------------------------------------------------------------ FP8 quantisation
// 8 consecutive bf16 channels per thread, 16 threads per 128-channel group.  All steps in
// fp32 without contraction: amax -> max(amax, 1e-4) -> scale = a / 448, inv = 448 / a,
// q = e4m3_rne_satfinite(x * inv).
__device__ __forceinline__ void quantize8(const uint4 in, bool valid, uint2& out, float& scale) {
    const uint32_t w[4] = {in.x, in.y, in.z, in.w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    float a = 0.0f;
    if (valid) {
#pragma unroll
        for (int i = 0; i < 8; ++i) a = fmaxf(a, fabsf(f[i]));
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    a = fmaxf(a, 1e-4f);
    scale = __fdiv_rn(a, 448.0f);
    const float inv = __fdiv_rn(448.0f, a);
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 v = make_float2(__fmul_rn(f[2 * i], inv), __fmul_rn(f[2 * i + 1], inv));
        q[i] = (uint32_t)__nv_cvt_float2_to_fp8x2(v, __NV_SATFINITE, __NV_E4M3);
    }
    out.x = q[0] | (q[1] << 16);
    out.y = q[2] | (q[3] << 16);
}

// --------------------------------------------------------------------- dispatch kernel
// Shared memory carve-up (dynamic): [stages * stage_bytes] row ring, then int arrays
// hist[B] (also scratch of scan_rank), arr[R], pos[chunk_slots].
template <int kMode, bool kFp8>
__global__ void __launch_bounds__(kThreads, 1) dispatch_kernel(const Params p, int stages, int stage_bytes) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t ready_bar;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c = blockIdx.x;
    const int t0 = (int)chunk_begin(c, p.T, p.nchunks), t1 = (int)chunk_begin(c + 1, p.T, p.nchunks);
    const int ntok = t1 - t0;
    int* hist = reinterpret_cast<int*>(smem + (size_t)stages * stage_bytes);
    int* arr = hist + p.B;
    int* pos = arr + p.R;
    volatile int* abortp = &abort_flag;
    int issued = 0;  // rows whose load thread 0 has started
    const unsigned epoch = current_epoch(p);

    constexpr int gn = kThreads - 32;  // layout group: warps 1..15
    constexpr int nw = kWarps - 1;
    const int gtid = tid - 32, gw = warp - 1;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], nw);
        }
        mbar_init(&ready_bar, 1);
        abort_flag = 0;
        mbar_fence_init();
    }
    for (int r = tid; r < p.R; r += kThreads) arr[r] = 0;
    // the arrival counters of the next call live in the other half; clear them now
    if (c == 0)
        for (int r = tid; r < p.R; r += kThreads) p.arrival[((epoch + 1) & 1) * p.R + r] = 0;
    __syncthreads();

    const unsigned row_in_bytes = (unsigned)p.H * 2u;

    if (warp == 0) {
        // ------------------------------------------------ mover warp (one elected thread)
        if (lane == 0) {
            bool ok = true;
            auto issue_load = [&](int n) {
                const int s = n % stages;
                mbar_arrive_expect_tx(&full_bar[s], row_in_bytes);
                bulk_load(smem + (size_t)s * stage_bytes, p.x + (size_t)(t0 + n) * p.H, row_in_bytes, &full_bar[s]);
            };
            if (!kFp8) {
                // loads run (stages - 3) rows ahead; up to 3 rows' stores stay in flight
                const int pf = stages - 3;
                for (; issued < min(pf, ntok); ++issued) issue_load(issued);
                ok = mbar_wait(&ready_bar, 0, abortp) && !*abortp;  // no rows without a layout
                for (int n = 0; ok && n < ntok; ++n) {
                    const int s = n % stages;
                    ok = mbar_wait(&full_bar[s], (n / stages) & 1, abortp);
                    if (!ok) break;
                    const uint8_t* src = smem + (size_t)s * stage_bytes;
                    for (int j = 0; j < p.k; ++j) {
                        const int where = pos[n * p.k + j];
                        if (where >= 0) bulk_store(p.recv_x + (size_t)where * p.rowB, src, (unsigned)p.rowB);
                    }
                    bulk_commit();
                    if (issued < ntok) {
                        bulk_wait_read<3>();
                        issue_load(issued);
                        ++issued;
                    }
                }
            } else {
                // loader only; the layout group quantises and stores, and frees the stages
                for (int n = 0; ok && n < ntok; ++n) {
                    const int s = n % stages;
                    if (n >= stages) ok = mbar_wait(&empty_bar[s], ((n / stages) - 1) & 1, abortp);
                    if (!ok) break;
                    issue_load(n);
                    issued = n + 1;
                }
            }
            if (!ok) {
                // a wait gave up: record it and let everybody leave
                report(p.status, kErrTimeout);
                abort_flag = 1;
            }
            bulk_wait_all<0>();
        }
    } else {
        // ------------------------------------------------------------- layout group
        bool ok = true;
        if (kMode == kModeFused) {
            if (gw == 0) count_chunk(p, c, hist, lane);
            group_sync(1, gn);
            if (gtid == 0 && c != p.withhold) {
                __threadfence();
                st_release(p.hist_flag + c, epoch);
            }
            // CalCumSum duty: this CTA serves rank c (and c + nchunks, ...)
            bool lost = false;  // a wait of this thread ran out
            for (int r = c; r < p.R; r += p.nchunks) {
                for (int cc = gtid; cc < p.nchunks; cc += gn)
                    if (!wait_flag(p.hist_flag + cc, epoch, abortp)) lost = true;
                if (group_or(1, gn, lost || *abortp)) { lost = true; break; }  // same answer for all
                scan_rank(p, r, hist, gw, nw, lane, 1);
                group_sync(1, gn);
                if (gtid == 0) {
                    __threadfence();
                    st_release(p.scan_flag + r, epoch);
                }
            }
            // every slot of this chunk may need any rank's bases
            if (!lost)
                for (int r = gtid; r < p.R; r += gn)
                    if (!wait_flag(p.scan_flag + r, epoch, abortp)) lost = true;
            ok = !group_or(1, gn, lost || *abortp);
            if (!ok && gtid == 0) {
                report(p.status, kErrTimeout);
                abort_flag = 1;
            }
        }
        if (ok) {
            finalize_chunk(p, c, pos, arr, gtid, gn);
            group_sync(1, gn);
            order_destinations(p, c, pos, ntok, gtid, gn);
            group_sync(1, gn);
        }
        if (gtid == 0) mbar_arrive(&ready_bar);
        if (kFp8 && ok) {
            const int nvec = p.H / 8;
            for (int n = 0; n < ntok; ++n) {
                const int s = n % stages;
                if (!mbar_wait(&full_bar[s], (n / stages) & 1, abortp)) break;
                const uint8_t* src = smem + (size_t)s * stage_bytes;
                for (int vb = gw * 32; vb < nvec; vb += gn) {
                    const int v = vb + lane;
                    const bool valid = v < nvec;
                    uint4 in = make_uint4(0, 0, 0, 0);
                    if (valid) in = *reinterpret_cast<const uint4*>(src + (size_t)v * 16);
                    uint2 q;
                    float scale;
                    quantize8(in, valid, q, scale);
                    if (valid) {
                        for (int j = 0; j < p.k; ++j) {
                            const int where = pos[n * p.k + j];
                            if (where < 0) continue;
                            *reinterpret_cast<uint2*>(p.recv_x + (size_t)where * p.rowB + (size_t)v * 8) = q;
                            if ((lane & 15) == 0) p.recv_scale[(size_t)where * p.G + (v >> 4)] = scale;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[s]);
            }
        }
    }
    __syncthreads();
    if (abort_flag) {
        // leaving early: the newest load of every ring stage may still be landing
        if (tid == 0)
            for (int n = max(0, issued - stages); n < issued; ++n)
                (void)mbar_wait(&full_bar[n % stages], (n / stages) & 1, nullptr);
        if (tid == 0) finish_dispatch(p, epoch);
        return;
    }
    // rows of this chunk have landed: add them to the per-region arrival counters
    {
        __threadfence();
        fence_proxy_async();
        for (int r = tid; r < p.R; r += kThreads)
            if (arr[r]) red_release_add(p.arrival + (epoch & 1) * p.R + r, (unsigned)arr[r]);
    }
    __syncthreads();
    if (tid == 0) finish_dispatch(p, epoch);
}

// ---------------------------------------------------------------------------- combine
// One thread per 16-byte vector of the output row: K independent 128-bit gathers, fp32
// fused multiply-adds in slot order, one round-to-nearest-even pack to bf16.
template <int K>
__global__ void __launch_bounds__(256) combine_kernel(const uint16_t* __restrict__ y,
                                                     const int32_t* __restrict__ slot_pos,
                                                     const float* __restrict__ topk_w, int T, int H, int k,
                                                     uint16_t* __restrict__ out) {
    const int nvec = H / 8;
    const int64_t total = (int64_t)T * nvec;
    const int kk = K > 0 ? K : k;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total;
         u += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(u / nvec), v = (int)(u - (int64_t)t * nvec);
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
        if (K > 0) {
            constexpr int KK = K > 0 ? K : 1;
            uint4 q[KK];
            float w[KK];
            int wh[KK];
#pragma unroll
            for (int j = 0; j < KK; ++j) {
                wh[j] = __ldg(slot_pos + (size_t)t * KK + j);
                w[j] = __ldg(topk_w + (size_t)t * KK + j);
            }
#pragma unroll
            for (int j = 0; j < KK; ++j) {
                q[j] = make_uint4(0, 0, 0, 0);
                if (wh[j] >= 0) q[j] = __ldg(reinterpret_cast<const uint4*>(y + (size_t)wh[j] * H) + v);
            }
#pragma unroll
            for (int j = 0; j < KK; ++j) {
                if (wh[j] < 0) continue;  // an empty slot contributes nothing
                const uint32_t ww[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[2 * i] = __fmaf_rn(w[j], __uint_as_float(ww[i] << 16), acc[2 * i]);
                    acc[2 * i + 1] = __fmaf_rn(w[j], __uint_as_float(ww[i] & 0xffff0000u), acc[2 * i + 1]);
                }
            }
        } else {
            for (int j = 0; j < kk; ++j) {
                const int where = __ldg(slot_pos + (size_t)t * kk + j);
                if (where < 0) continue;
                const float w = __ldg(topk_w + (size_t)t * kk + j);
                const uint4 q = __ldg(reinterpret_cast<const uint4*>(y + (size_t)where * H) + v);
                const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[2 * i] = __fmaf_rn(w, __uint_as_float(ww[i] << 16), acc[2 * i]);
                    acc[2 * i + 1] = __fmaf_rn(w, __uint_as_float(ww[i] & 0xffff0000u), acc[2 * i + 1]);
                }
            }
        }
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
            o[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        reinterpret_cast<uint4*>(out + (size_t)t * H)[v] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// ---------------------------------------------------------------- counts-only layout
// ubep_get_dispatch_layout: every CTA histograms its token chunk in shared memory, writes
// the chunk histogram to scratch, and the last CTA to finish (ticket) sums the chunks.
__global__ void __launch_bounds__(256) layout_kernel(const Params p, int32_t* num_tokens_per_rank,
                                                    int32_t* num_tokens_per_expert,
                                                    uint8_t* is_token_in_rank, int32_t* scratch_hist,
                                                    unsigned* ticket) {
    extern __shared__ int sm_i[];
    __shared__ bool last;
    const int B = p.B, k = p.k, R = p.R, n = gridDim.x, c = blockIdx.x;
    const int t0 = (int)chunk_begin(c, p.T, n), t1 = (int)chunk_begin(c + 1, p.T, n);
    for (int b = threadIdx.x; b < B; b += blockDim.x) sm_i[b] = 0;
    if (is_token_in_rank) {
        uint8_t* z = is_token_in_rank + (size_t)t0 * R;
        for (size_t i = threadIdx.x; i < (size_t)(t1 - t0) * R; i += blockDim.x) z[i] = 0;
    }
    __syncthreads();
    for (int t = t0 + threadIdx.x; t < t1; t += blockDim.x) {
        int seen[kMaxTopk];
        for (int j = 0; j < k; ++j) {
            const int e = resolve_expert(p, t, __ldg(p.topk_idx + (size_t)t * k + j));
            int r = -1;
            if (e >= 0) {
                atomicAdd(&sm_i[e], 1);
                r = e / p.L;
                bool first = true;
                for (int jj = 0; jj < j; ++jj) first = first && seen[jj] != r;
                if (first) {
                    atomicAdd(&sm_i[p.E + r], 1);
                    if (is_token_in_rank) is_token_in_rank[(size_t)t * R + r] = 1;
                }
            }
            seen[j] = r;
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < B; b += blockDim.x) scratch_hist[(size_t)c * B + b] = sm_i[b];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(ticket, 1u) == (unsigned)(n - 1);
    __syncthreads();
    if (!last) return;
    __threadfence();
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        int sum = 0;
        for (int cc = 0; cc < n; ++cc) sum += __ldcg(scratch_hist + (size_t)cc * B + b);
        if (b < p.E) {
            if (num_tokens_per_expert) num_tokens_per_expert[b] = sum;
        } else if (num_tokens_per_rank) {
            num_tokens_per_rank[b - p.E] = sum;
        }
    }
    if (threadIdx.x == 0) *ticket = 0;  // ready for the next call
}

// ------------------------------------------------------------------------- launchers

static size_t dispatch_smem_bytes(const Params& p, int stages, int stage_bytes) {
    const int chunk_tokens = (p.T + p.nchunks - 1) / p.nchunks;
    return (size_t)stages * stage_bytes + sizeof(int) * ((size_t)p.B + p.R + (size_t)chunk_tokens * p.k) + 16;
}

int plan_dispatch(const Params& p, int max_smem, int* stages, int* stage_bytes, size_t* smem) {
    const int sb = ((p.H * 2 + 127) / 128) * 128;
    const int chunk_tokens = (p.T + p.nchunks - 1) / p.nchunks;
    const size_t fixed = sizeof(int) * ((size_t)p.B + p.R + (size_t)chunk_tokens * p.k) + 16 + 1024;
    if (fixed + 4 * (size_t)sb > (size_t)max_smem) return -1;
    int st = (int)(((size_t)max_smem - fixed) / sb);
    if (st > kMaxStages) st = kMaxStages;
    *stages = st;
    *stage_bytes = sb;
    *smem = dispatch_smem_bytes(p, st, sb);
    return 0;
}

template <int kMode, bool kFp8>
static cudaError_t launch_dispatch_t(const Params& p, int stages, int stage_bytes, size_t smem, cudaStream_t st) {
    auto kern = dispatch_kernel<kMode, kFp8>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<p.nchunks, kThreads, smem, st>>>(p, stages, stage_bytes);
    return cudaGetLastError();
}

cudaError_t launch_dispatch(const Params& p, int mode, int stages, int stage_bytes, size_t smem, cudaStream_t st,
                            int* launches) {
    cudaError_t e;
    if (mode == kModePhased) {
        count_kernel<<<p.nchunks, 32, sizeof(int) * p.B, st>>>(p);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        scan_kernel<<<p.R, 256, sizeof(int) * (p.L + 1), st>>>(p);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        *launches = 3;
        return p.payload ? launch_dispatch_t<kModePhased, true>(p, stages, stage_bytes, smem, st)
                         : launch_dispatch_t<kModePhased, false>(p, stages, stage_bytes, smem, st);
    }
    *launches = 1;
    return p.payload ? launch_dispatch_t<kModeFused, true>(p, stages, stage_bytes, smem, st)
                     : launch_dispatch_t<kModeFused, false>(p, stages, stage_bytes, smem, st);
}

cudaError_t launch_combine(const uint16_t* y, const int32_t* slot_pos, const float* topk_w, int T, int H, int k,
                           uint16_t* out, int num_sms, cudaStream_t st) {
    const int64_t total = (int64_t)T * (H / 8);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)num_sms * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    switch (k) {
        case 1: combine_kernel<1><<<(int)blocks, 256, 0, st>>>(y, slot_pos, topk_w, T, H, k, out); break;
        case 2: combine_kernel<2><<<(int)blocks, 256, 0, st>>>(y, slot_pos, topk_w, T, H, k, out); break;
        case 4: combine_kernel<4><<<(int)blocks, 256, 0, st>>>(y, slot_pos, topk_w, T, H, k, out); break;
        case 8: combine_kernel<8><<<(int)blocks, 256, 0, st>>>(y, slot_pos, topk_w, T, H, k, out); break;
        default: combine_kernel<0><<<(int)blocks, 256, 0, st>>>(y, slot_pos, topk_w, T, H, k, out); break;
    }
    return cudaGetLastError();
}

cudaError_t launch_layout(const Params& p, int32_t* num_tokens_per_rank, int32_t* num_tokens_per_expert,
                          uint8_t* is_token_in_rank, int32_t* scratch_hist, unsigned* ticket, cudaStream_t st) {
    layout_kernel<<<p.nchunks, 256, sizeof(int) * p.B, st>>>(p, num_tokens_per_rank, num_tokens_per_expert,
                                                             is_token_in_rank, scratch_hist, ticket);
    return cudaGetLastError();
}

}  // namespace ubep
