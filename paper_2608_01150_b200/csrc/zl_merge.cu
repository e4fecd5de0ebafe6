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

constexpr int kHeadsPerUnit = 4;  // a warp merges this many heads of one query row before it looks up the next row

// One (row, head): LSE = M + log sum_t exp(LSE_t - M), O = sum_t exp(LSE_t - LSE) O_t in ascending part order.
// NP > 0: at most NP parts, whose LSEs are read once and kept in registers (weights e_t / z); when the group has
// exactly NP parts (the common case: one part per context-parallel chunk) all NP vector loads of the partial
// outputs are issued before the first use, so a warp keeps NP x 512 bytes in flight.  NP = 0: any number of
// parts, three passes over the parts' LSEs.
// `src0` points at this lane's floats of part row 0, head h; `lse_h` at lse_partial[h][row]; `slot` holds the
// parts' slot offsets (rows).
template <int D, int NP>
__device__ __forceinline__ float merge_one(const MergeParams& p, const MergeGroup& g, const int32_t* part,
                                           const int32_t (&slot)[NP > 0 ? NP : 1], const float* src0, const float* lse_h,
                                           float (&acc)[D / 32]) {
    constexpr int V = D / 32;
    const int64_t part_stride = (int64_t)p.n_heads * D;  // floats between consecutive rows of o_partial
    if constexpr (NP > 0) {
        const bool all_parts = g.n_parts == NP;  // warp-uniform
        float4 x4[NP];
        float2 x2[NP];
        if (all_parts) {
#pragma unroll
            for (int t = 0; t < NP; ++t) {
                const float* src = src0 + slot[t] * part_stride;
                if constexpr (V == 4) x4[t] = __ldcs(reinterpret_cast<const float4*>(src));
                else x2[t] = __ldcs(reinterpret_cast<const float2*>(src));
            }
        }
        float lt[NP];
        float M = -INFINITY;
#pragma unroll
        for (int t = 0; t < NP; ++t) {
            lt[t] = (t < g.n_parts) ? __ldg(lse_h + slot[t]) : -INFINITY;
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
                if (!all_parts) {
                    const float* src = src0 + slot[t] * part_stride;
                    if constexpr (V == 4) x4[t] = __ldcs(reinterpret_cast<const float4*>(src));
                    else x2[t] = __ldcs(reinterpret_cast<const float2*>(src));
                }
                if constexpr (V == 4) {
                    acc[0] = fmaf(w, x4[t].x, acc[0]); acc[1] = fmaf(w, x4[t].y, acc[1]);
                    acc[2] = fmaf(w, x4[t].z, acc[2]); acc[3] = fmaf(w, x4[t].w, acc[3]);
                } else {
                    acc[0] = fmaf(w, x2[t].x, acc[0]); acc[1] = fmaf(w, x2[t].y, acc[1]);
                }
            }
        }
        return (M == -INFINITY) ? -INFINITY : M + logf(z);
    } else {
        float M = -INFINITY;
        for (int t = 0; t < g.n_parts; ++t) M = fmaxf(M, __ldg(lse_h + part[t]));
        float z = 0.f;
        for (int t = 0; t < g.n_parts; ++t) z += (M == -INFINITY) ? 0.f : __expf(__ldg(lse_h + part[t]) - M);
        const float L = (M == -INFINITY) ? -INFINITY : M + logf(z);
        for (int t = 0; t < g.n_parts; ++t) {
            const float w = (L == -INFINITY) ? 0.f : __expf(__ldg(lse_h + part[t]) - L);
            const float* src = src0 + part[t] * part_stride;
            if constexpr (V == 4) {
                const float4 x = __ldcs(reinterpret_cast<const float4*>(src));
                acc[0] = fmaf(w, x.x, acc[0]); acc[1] = fmaf(w, x.y, acc[1]);
                acc[2] = fmaf(w, x.z, acc[2]); acc[3] = fmaf(w, x.w, acc[3]);
            } else {
                const float2 x = __ldcs(reinterpret_cast<const float2*>(src));
                acc[0] = fmaf(w, x.x, acc[0]); acc[1] = fmaf(w, x.y, acc[1]);
            }
        }
        return L;
    }
}

// NP = 4 or 8: every group has at most NP parts (chosen by the launcher); NP = 0: any number of parts.
// A unit of work is one query row and kHeadsPerUnit consecutive heads: the group lookup, the parts' slots and
// the row's base addresses are worked out once per unit (the kernel is bound by instruction issue, not by DRAM).
template <int D, int NP>
__global__ void __launch_bounds__(kMergeThreads, NP == 8 ? 3 : (NP == 4 ? 4 : 8)) zl_merge_kernel(const MergeParams p) {
    constexpr int V = D / 32;  // floats per lane: 4 (d=128) or 2 (d=64)
    const int lane = threadIdx.x & 31;
    const int warps_per_block = kMergeThreads / 32;
    const int64_t n_rows = p.row_prefix[p.n_groups];
    const int head_chunks = (p.n_heads + kHeadsPerUnit - 1) / kHeadsPerUnit;
    const int64_t n_units = n_rows * head_chunks;
    for (int64_t u = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); u < n_units;
         u += (int64_t)gridDim.x * warps_per_block) {
        const int64_t r = u / head_chunks;
        const int hc = (int)(u - r * head_chunks);
        // group of flat row r: binary search over the prefix sums
        int lo = 0, hi = p.n_groups;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.row_prefix[mid] <= r) lo = mid; else hi = mid;
        }
        const MergeGroup g = p.groups[lo];
        const int h_begin = max(hc * kHeadsPerUnit, g.head_begin);   // heads outside the group's range: no task runs them
        const int h_end = min(min((hc + 1) * kHeadsPerUnit, p.n_heads), g.head_begin + g.head_count);
        if (h_begin >= h_end) continue;
        const int row = (int)(r - p.row_prefix[lo]);
        const int32_t* part = p.parts + g.part_begin;
        int32_t slot[NP > 0 ? NP : 1];
        if constexpr (NP > 0) {
#pragma unroll
            for (int t = 0; t < NP; ++t) slot[t] = (t < g.n_parts) ? __ldg(part + t) : 0;
        }
        const int64_t qrow = (int64_t)g.q_off + row;
        for (int h = h_begin; h < h_end; ++h) {
            float acc[V];
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] = 0.f;
            const float* src0 = p.o_partial + ((int64_t)row * p.n_heads + h) * D + lane * V;
            const float* lse_h = p.lse_partial + (int64_t)h * p.partial_rows + row;
            const float L = merge_one<D, NP>(p, g, part, slot, src0, lse_h, acc);
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
}

}  // namespace

cudaError_t launch_merge(int head_dim, const MergeParams& p, int max_parts, int n_sms, cudaStream_t stream) {
    if (p.n_groups == 0) return cudaSuccess;
    const int grid = n_sms * 8;
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
