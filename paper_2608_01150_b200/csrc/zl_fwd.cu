// Forward kernel of the coalesced attention engine (sm_100a).
//
// One persistent launch walks a longest-first list of work items (task, head, query tile)
// that spans whole sequences and context-parallel shard tasks alike (paper Section IV-D:
// all whole sequences of a rank are packed into one block-diagonal attention call next to
// the rank's shards, without mixing attention across sequences).  Per item:
//   S = Q K^T on the tensor cores (tcgen05.mma, operands staged by TMA in 128B-swizzled
//   shared memory, accumulator in TMEM), online softmax in registers with one thread per
//   query row, P written back to TMEM as bf16, O += P V on the tensor cores.
// Whole-sequence tasks store final bf16 O and fp32 LSE; shard tasks store their partial
// result (normalised within their own K/V chunk) as fp32 O plus LSE for the merge kernel.
#include <cuda_runtime.h>

#include "zl_device.h"
#include "zl_ptx.cuh"

namespace zl {

using namespace ptx;

namespace {

constexpr int kFwdThreads = 192;  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: softmax
constexpr uint64_t kWaitLimitNs = 4000000000ull;

template <int D>
struct FwdSmem {
    static constexpr int kStages = (D == 128) ? 2 : 4;
    static constexpr int kTileBytes = kTileQ * D * 2;  // one 128-row tile of Q, K or V
    static constexpr int kBoxBytes = kTileQ * 128;     // one TMA box: 128 rows x 64 bf16
    static constexpr int kBoxes = D / 64;
    alignas(1024) uint8_t q[kTileBytes];
    alignas(1024) uint8_t k[kStages][kTileBytes];
    alignas(1024) uint8_t v[kStages][kTileBytes];
    alignas(8) uint64_t q_full, q_empty;
    uint64_t k_full[kStages], v_full[kStages], kv_empty[kStages];
    uint64_t s_full, p_full, pv_done;
    uint32_t tmem_base;
    volatile int32_t abort_flag;
};

__device__ __forceinline__ void report(int32_t* status, volatile int32_t* abort_flag, int where) {
    *abort_flag = 1;
    if (atomicCAS(status, 0, (int)ZL_ERR_TIMEOUT) == 0) status[1] = where;
}

// Wait used by a single elected thread.
#define ZL_WAIT(bar, parity, site)                                        \
    do {                                                                  \
        if (!mbar_wait((bar), (parity), kWaitLimitNs) || sm.abort_flag) { \
            report(p.status, &sm.abort_flag, 1000 + (site));              \
            goto teardown;                                                \
        }                                                                 \
    } while (0)
// Wait used by all 32 lanes of a warp: the outcome is made warp-uniform and the warp
// reconverges before the .sync.aligned TMEM instructions that follow.
#define ZL_WAIT_WARP(bar, parity, site)                                             \
    do {                                                                            \
        const bool ok_ = mbar_wait((bar), (parity), kWaitLimitNs) && !sm.abort_flag; \
        if (!__all_sync(0xffffffffu, ok_)) {                                        \
            report(p.status, &sm.abort_flag, 1000 + (site));                        \
            goto teardown;                                                          \
        }                                                                           \
    } while (0)

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
zl_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    using Smem = FwdSmem<D>;
    constexpr int kStages = Smem::kStages;
    constexpr int kBoxes = Smem::kBoxes;
    extern __shared__ uint8_t smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // TMEM columns: S [0,128), O [128,128+D), P (bf16 pairs) [256,320)
    constexpr uint32_t kColS = 0, kColO = 128, kColP = 256, kTmemCols = 512;

    if (threadIdx.x == 0) {
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.q_empty, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.k_full[s], 1);
            mbar_init(&sm.v_full[s], 1);
            mbar_init(&sm.kv_empty[s], 1);
        }
        mbar_init(&sm.s_full, 1);
        mbar_init(&sm.p_full, 128);
        mbar_init(&sm.pv_done, 1);
        sm.abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t q_cnt = 0, kv_cnt = 0;
            for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
                const WorkItem wi = p.items[it];
                const Task t = p.tasks[wi.unit];
                const int n_kv = (t.kv_len + kTileKV - 1) / kTileKV;
                if (n_kv == 0) continue;
                ZL_WAIT(&sm.q_empty, (q_cnt & 1) ^ 1, 1);
                mbar_arrive_expect_tx(&sm.q_full, Smem::kTileBytes);
                for (int b = 0; b < kBoxes; ++b)
                    tma_load_3d(sm.q + b * Smem::kBoxBytes, &tm_q, &sm.q_full, b * 64, wi.head, t.q_off + wi.row0);
                ++q_cnt;
                for (int j = 0; j < n_kv; ++j, ++kv_cnt) {
                    const int s = kv_cnt % kStages;
                    const uint32_t ph = (kv_cnt / kStages) & 1;
                    ZL_WAIT(&sm.kv_empty[s], ph ^ 1, 2);
                    mbar_arrive_expect_tx(&sm.k_full[s], Smem::kTileBytes);
                    for (int b = 0; b < kBoxes; ++b)
                        tma_load_3d(sm.k[s] + b * Smem::kBoxBytes, &tm_k, &sm.k_full[s], b * 64, wi.head,
                                    t.kv_off + j * kTileKV);
                    mbar_arrive_expect_tx(&sm.v_full[s], Smem::kTileBytes);
                    for (int b = 0; b < kBoxes; ++b)
                        tma_load_3d(sm.v[s] + b * Smem::kBoxBytes, &tm_v, &sm.v_full[s], b * 64, wi.head,
                                    t.kv_off + j * kTileKV);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(kTileQ, kTileKV, 0, 0);
            constexpr uint32_t idesc_o = make_idesc_bf16(kTileQ, D, 0, 1);
            uint32_t q_cnt = 0, kv_cnt = 0, p_cnt = 0;
            const uint32_t q_addr = smem_u32(sm.q);
            for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
                const WorkItem wi = p.items[it];
                const Task t = p.tasks[wi.unit];
                const int n_kv = (t.kv_len + kTileKV - 1) / kTileKV;
                if (n_kv == 0) continue;
                ZL_WAIT(&sm.q_full, q_cnt & 1, 11);
                ++q_cnt;
                auto issue_s = [&](uint32_t stage) {
                    const uint32_t k_addr = smem_u32(sm.k[stage]);
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t off = (ks / 4) * Smem::kBoxBytes + (ks % 4) * 32;
                        mma_ss(tmem + kColS, make_desc_sw128(q_addr + off, 16, 1024),
                               make_desc_sw128(k_addr + off, 16, 1024), idesc_s, ks > 0);
                    }
                    mma_commit(&sm.s_full);
                };
                ZL_WAIT(&sm.k_full[kv_cnt % kStages], (kv_cnt / kStages) & 1, 12);
                issue_s(kv_cnt % kStages);
                for (int j = 0; j < n_kv; ++j, ++kv_cnt) {
                    const uint32_t s = kv_cnt % kStages;
                    // P(j) written, S(j) fully read, O rescaled
                    ZL_WAIT(&sm.p_full, p_cnt & 1, 13);
                    ++p_cnt;
                    if (j + 1 < n_kv) {
                        const uint32_t nk = kv_cnt + 1;
                        ZL_WAIT(&sm.k_full[nk % kStages], (nk / kStages) & 1, 14);
                        issue_s(nk % kStages);
                    } else {
                        mma_commit(&sm.q_empty);  // all S MMAs of this item are done with Q
                    }
                    ZL_WAIT(&sm.v_full[s], (kv_cnt / kStages) & 1, 15);
                    tc_fence_after();
                    const uint32_t v_addr = smem_u32(sm.v[s]);
#pragma unroll
                    for (int ks = 0; ks < kTileKV / 16; ++ks) {
                        mma_ts(tmem + kColO, tmem + kColP + ks * 8,
                               make_desc_sw128(v_addr + ks * 2048, Smem::kBoxBytes, 1024), idesc_o,
                               j > 0 || ks > 0);
                    }
                    mma_commit(&sm.kv_empty[s]);
                    mma_commit(&sm.pv_done);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        const int quarter = warp & 3;              // TMEM lane quarter this warp may access
        const int row = quarter * 32 + lane;       // query row within the tile
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        uint32_t s_cnt = 0, pv_cnt = 0;
        const float sl2 = p.scale_log2;
        for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
            const WorkItem wi = p.items[it];
            const Task t = p.tasks[wi.unit];
            const int n_kv = (t.kv_len + kTileKV - 1) / kTileKV;
            float m = -INFINITY, l = 0.f;
            for (int j = 0; j < n_kv; ++j) {
                ZL_WAIT_WARP(&sm.s_full, s_cnt & 1, 21);
                ++s_cnt;
                tc_fence_after();
                float sv[kTileKV];
#pragma unroll
                for (int c = 0; c < kTileKV / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(lane_addr + kColS + c * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) sv[c * 32 + i] = __uint_as_float(r[i]);
                }
                const int valid = t.kv_len - j * kTileKV;  // columns of this tile inside the task
                if (valid < kTileKV) {
#pragma unroll
                    for (int c = 0; c < kTileKV; ++c)
                        if (c >= valid) sv[c] = -INFINITY;
                }
                float mx = sv[0];
#pragma unroll
                for (int c = 1; c < kTileKV; ++c) mx = fmaxf(mx, sv[c]);
                const float m_new = fmaxf(m, mx);
                const float alpha = ex2((m - m_new) * sl2);
                const float mb = m_new * sl2;
                float rs = 0.f;
                uint32_t pk[kTileKV / 2];
#pragma unroll
                for (int c = 0; c < kTileKV; c += 2) {
                    const float p0 = ex2(fmaf(sv[c], sl2, -mb));
                    const float p1 = ex2(fmaf(sv[c + 1], sl2, -mb));
                    rs += p0 + p1;
                    pk[c / 2] = pack_bf16(p0, p1);
                }
                l = l * alpha + rs;
                m = m_new;
                if (j > 0) {
                    // previous P V product must be complete before O is rescaled and P overwritten
                    ZL_WAIT_WARP(&sm.pv_done, pv_cnt & 1, 22);
                    ++pv_cnt;
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(lane_addr + kColO + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st_x32(lane_addr + kColO + c * 32, r);
                    }
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t r[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = pk[c * 32 + i];
                    tmem_st_x32(lane_addr + kColP + c * 32, r);
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&sm.p_full);
            }
            // ---- epilogue
            const bool row_ok = row < wi.rows;
            const float inv_l = (l > 0.f) ? 1.f / l : 0.f;
            const float lse = (l > 0.f) ? (m * sl2 + log2f(l)) * 0.6931471805599453f : -INFINITY;
            if (n_kv > 0) {
                ZL_WAIT_WARP(&sm.pv_done, pv_cnt & 1, 23);
                ++pv_cnt;
                tc_fence_after();
            }
            const int64_t grow = (int64_t)(t.partial_slot >= 0 ? t.partial_slot : t.q_off) + wi.row0 + row;
            if (t.partial_slot >= 0) {
                float* dst = p.o_partial + (grow * p.n_heads + wi.head) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    if (n_kv > 0) {
                        tmem_ld_x32(lane_addr + kColO + c * 32, r);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = 0;
                    }
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            float4 o4 = make_float4(__uint_as_float(r[i]) * inv_l, __uint_as_float(r[i + 1]) * inv_l,
                                                    __uint_as_float(r[i + 2]) * inv_l, __uint_as_float(r[i + 3]) * inv_l);
                            *reinterpret_cast<float4*>(dst + c * 32 + i) = o4;
                        }
                    }
                }
                if (row_ok) p.lse_partial[(int64_t)wi.head * p.partial_rows + grow] = lse;
            } else {
                __nv_bfloat16* dst = p.o + (grow * p.n_heads + wi.head) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    if (n_kv > 0) {
                        tmem_ld_x32(lane_addr + kColO + c * 32, r);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = 0;
                    }
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            uint4 o4;
                            o4.x = pack_bf16(__uint_as_float(r[i]) * inv_l, __uint_as_float(r[i + 1]) * inv_l);
                            o4.y = pack_bf16(__uint_as_float(r[i + 2]) * inv_l, __uint_as_float(r[i + 3]) * inv_l);
                            o4.z = pack_bf16(__uint_as_float(r[i + 4]) * inv_l, __uint_as_float(r[i + 5]) * inv_l);
                            o4.w = pack_bf16(__uint_as_float(r[i + 6]) * inv_l, __uint_as_float(r[i + 7]) * inv_l);
                            *reinterpret_cast<uint4*>(dst + c * 32 + i) = o4;
                        }
                    }
                }
                if (row_ok) p.lse[(int64_t)wi.head * p.total_q + grow] = lse;
            }
            tc_fence_before();
        }
    }

teardown:
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

cudaError_t launch_fwd(int head_dim, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                       const FwdParams& p, int grid, cudaStream_t stream) {
    if (p.n_items == 0) return cudaSuccess;
    if (head_dim == 128) {
        constexpr int smem = sizeof(FwdSmem<128>) + 1024;
        static bool configured = false;
        if (!configured) {
            cudaError_t e = cudaFuncSetAttribute(zl_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            configured = true;
        }
        zl_fwd_kernel<128><<<grid, kFwdThreads, smem, stream>>>(tq, tk, tv, p);
    } else {
        constexpr int smem = sizeof(FwdSmem<64>) + 1024;
        static bool configured = false;
        if (!configured) {
            cudaError_t e = cudaFuncSetAttribute(zl_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            configured = true;
        }
        zl_fwd_kernel<64><<<grid, kFwdThreads, smem, stream>>>(tq, tk, tv, p);
    }
    return cudaGetLastError();
}

}  // namespace zl
