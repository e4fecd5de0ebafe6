// LSE merge kernel: combines the partial results of the shard tasks of each merge group
// (the accumulation step of ring / all-gather context parallelism, paper Section II-B):
//     LSE = M + log sum_t exp(LSE_t - M),  M = max_t LSE_t
//     O   = sum_t exp(LSE_t - LSE) * O_t        (ascending shard order, bit-deterministic)
// HBM-bound: one warp per (query row, head), each lane owns head_dim/32 consecutive floats
// and reads them with one vector load per part.
#include <cuda_runtime.h>

#include "zl_device.h"
#include "zl_ptx.cuh"

namespace zl {

namespace {

constexpr int kMergeThreads = 256;

// Up to NP parts: the parts' LSEs are read once and kept in registers (weights e_t / z).
template <int D, int NP>
__device__ __forceinline__ float merge_small(const MergeParams& p, const MergeGroup& g, int row, int h, int lane,
                                             float (&acc)[D / 32]) {
    constexpr int V = D / 32;
    const float* lse_h = p.lse_partial + (int64_t)h * p.partial_rows + row;
    const int32_t* part = p.parts + g.part_begin;
    float lt[NP];
    float M = -INFINITY;
#pragma unroll
    for (int t = 0; t < NP; ++t) {
        lt[t] = (t < g.n_parts) ? __ldg(lse_h + part[t]) : -INFINITY;
        M = fmaxf(M, lt[t]);
    }
    float z = 0.f;
#pragma unroll
    for (int t = 0; t < NP; ++t) {
        lt[t] = (M == -INFINITY) ? 0.f : __expf(lt[t] - M);  // 0 for absent parts
        z += lt[t];
    }
    const float inv_z = (z > 0.f) ? 1.f / z : 0.f;
#pragma unroll
    for (int t = 0; t < NP; ++t) {
        if (t < g.n_parts) {
            const float w = lt[t] * inv_z;
            const float* src = p.o_partial + (((int64_t)part[t] + row) * p.n_heads + h) * D + lane * V;
            if constexpr (V == 4) {
                const float4 x = __ldcs(reinterpret_cast<const float4*>(src));
                acc[0] = fmaf(w, x.x, acc[0]); acc[1] = fmaf(w, x.y, acc[1]);
                acc[2] = fmaf(w, x.z, acc[2]); acc[3] = fmaf(w, x.w, acc[3]);
            } else {
                const float2 x = __ldcs(reinterpret_cast<const float2*>(src));
                acc[0] = fmaf(w, x.x, acc[0]); acc[1] = fmaf(w, x.y, acc[1]);
            }
        }
    }
    return (M == -INFINITY) ? -INFINITY : M + logf(z);
}

// NP = 4 or 8: every group has at most NP parts (chosen by the launcher); NP = 0: any number of parts.
template <int D, int NP>
__global__ void __launch_bounds__(kMergeThreads, 8) zl_merge_kernel(const MergeParams p) {  // 8 blocks = 64 warps per SM
    constexpr int V = D / 32;  // floats per lane: 4 (d=128) or 2 (d=64)
    const int lane = threadIdx.x & 31;
    const int warps_per_block = kMergeThreads / 32;
    const int64_t n_rows = p.row_prefix[p.n_groups];
    const int64_t n_units = n_rows * p.n_heads;
    for (int64_t u = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); u < n_units;
         u += (int64_t)gridDim.x * warps_per_block) {
        const int64_t r = u / p.n_heads;
        const int h = (int)(u - r * p.n_heads);
        // group of flat row r: binary search over the prefix sums
        int lo = 0, hi = p.n_groups;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.row_prefix[mid] <= r) lo = mid; else hi = mid;
        }
        const MergeGroup g = p.groups[lo];
        if (h < g.head_begin || h >= g.head_begin + g.head_count) continue;  // the group's tasks do not run this head
        const int row = (int)(r - p.row_prefix[lo]);
        float acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = 0.f;
        float L;
        if constexpr (NP > 0) {
            L = merge_small<D, NP>(p, g, row, h, lane, acc);
        } else {
            // any number of parts: three passes over the parts' LSEs
            float M = -INFINITY;
            for (int t = 0; t < g.n_parts; ++t) {
                const int64_t pr = (int64_t)p.parts[g.part_begin + t] + row;
                M = fmaxf(M, __ldg(p.lse_partial + (int64_t)h * p.partial_rows + pr));
            }
            float z = 0.f;
            for (int t = 0; t < g.n_parts; ++t) {
                const int64_t pr = (int64_t)p.parts[g.part_begin + t] + row;
                const float lt = __ldg(p.lse_partial + (int64_t)h * p.partial_rows + pr);
                z += (M == -INFINITY) ? 0.f : __expf(lt - M);
            }
            L = (M == -INFINITY) ? -INFINITY : M + logf(z);
            for (int t = 0; t < g.n_parts; ++t) {
                const int64_t pr = (int64_t)p.parts[g.part_begin + t] + row;
                const float lt = __ldg(p.lse_partial + (int64_t)h * p.partial_rows + pr);
                const float w = (L == -INFINITY) ? 0.f : __expf(lt - L);
                const float* src = p.o_partial + (pr * p.n_heads + h) * D + lane * V;
                if constexpr (V == 4) {
                    const float4 x = __ldcs(reinterpret_cast<const float4*>(src));
                    acc[0] = fmaf(w, x.x, acc[0]); acc[1] = fmaf(w, x.y, acc[1]);
                    acc[2] = fmaf(w, x.z, acc[2]); acc[3] = fmaf(w, x.w, acc[3]);
                } else {
                    const float2 x = __ldcs(reinterpret_cast<const float2*>(src));
                    acc[0] = fmaf(w, x.x, acc[0]); acc[1] = fmaf(w, x.y, acc[1]);
                }
            }
        }
        const int64_t qrow = (int64_t)g.q_off + row;
        __nv_bfloat16* dst = p.o + (qrow * p.n_heads + h) * D + lane * V;
        if constexpr (V == 4) {
            __nv_bfloat162 a = __floats2bfloat162_rn(acc[0], acc[1]);
            __nv_bfloat162 b = __floats2bfloat162_rn(acc[2], acc[3]);
            uint2 o2;
            o2.x = *reinterpret_cast<uint32_t*>(&a);
            o2.y = *reinterpret_cast<uint32_t*>(&b);
            *reinterpret_cast<uint2*>(dst) = o2;
        } else {
            *reinterpret_cast<__nv_bfloat162*>(dst) = __floats2bfloat162_rn(acc[0], acc[1]);
        }
        if (lane == 0) p.lse[(int64_t)h * p.total_q + qrow] = L;
    }
}

}  // namespace

cudaError_t launch_merge(int head_dim, const MergeParams& p, int max_parts, int n_sms, cudaStream_t stream) {
    if (p.n_groups == 0) return cudaSuccess;
    const int grid = n_sms * 8;  // 8 resident blocks of 256 threads per SM
    const int np = max_parts <= 4 ? 4 : (max_parts <= 8 ? 8 : 0);
    if (head_dim == 128) {
        if (np == 4) zl_merge_kernel<128, 4><<<grid, kMergeThreads, 0, stream>>>(p);
        else if (np == 8) zl_merge_kernel<128, 8><<<grid, kMergeThreads, 0, stream>>>(p);
        else zl_merge_kernel<128, 0><<<grid, kMergeThreads, 0, stream>>>(p);
    } else {
        if (np == 4) zl_merge_kernel<64, 4><<<grid, kMergeThreads, 0, stream>>>(p);
        else if (np == 8) zl_merge_kernel<64, 8><<<grid, kMergeThreads, 0, stream>>>(p);
        else zl_merge_kernel<64, 0><<<grid, kMergeThreads, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

// Self-test of the bounded wait: a barrier that never completes must time out, be reported through
// the status word, and leave the context usable.
namespace {
__global__ void zl_wait_selftest_kernel(int32_t* status, uint64_t limit_ns) {
    __shared__ uint64_t bar;
    __shared__ volatile int32_t abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!ptx::mbar_wait(&bar, 0, limit_ns, &abort_flag)) {
            if (atomicCAS(status, 0, (int)ZL_ERR_TIMEOUT) == 0) status[1] = 9001;
        }
    }
}
}  // namespace

cudaError_t launch_wait_selftest(int32_t* status, uint64_t limit_ns, cudaStream_t stream) {
    zl_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace zl
