// Backward kernels of the coalesced attention engine (sm_100a).
//
// Gradients of softmax attention for every task of a placement (whole sequences and
// context-parallel shard tasks, paper Section IV-D), for dL/dO = dO and no gradient
// through LSE.  With P = exp(scale * Q K^T - LSE) recomputed from the final LSE:
//     dV = P^T dO,   dS = P o (dO V^T - D),   dQ = scale * dS K,   dK = scale * dS^T Q,
//     D_i = sum_c dO_ic O_ic.
//
// Three launches:
//   pre   per 128-row query tile and head, a 4 KB "augmentation" tile holding -LSE/scale and
//         -D, each split into three bf16 pieces (the dQ accumulator is cleared by a memset node
//         before it).  The main kernel appends one extra K=16 MMA step to S^T and to dP^T whose
//         A operand is a tile of ones, so the tensor core itself produces S^T - LSE/scale and
//         dP^T - D: no per-column vector has to be broadcast from shared memory;
//   main  persistent; a CTA owns one 128-row key tile of one kv group and one head, keeps
//         K, V in shared memory and dK, dV in TMEM, and loops over every 128-row query tile
//         of every task that shares the key range.  Per tile it issues five tcgen05 MMAs
//         (S^T = K Q^T, dP^T = V dO^T, dV += P^T dO, dK += dS^T Q, dQ = dS K); dK/dV need no
//         atomics, dQ tiles are staged in shared memory and added into an fp32 accumulator by
//         the TMA (cp.reduce.async.bulk.tensor);
//   post  dQ accumulator * scale -> bf16.
#include <cuda_runtime.h>

#include "zl_device.h"
#include "zl_ptx.cuh"

namespace zl {

using namespace ptx;

namespace {

constexpr uint64_t kWaitLimitNs = 4000000000ull;

// ======================================================================= preprocess
constexpr int kPreThreads = 256;

__device__ __forceinline__ int find_q_group(const QGroup* g, int n, int slot_row) {
    int lo = 0, hi = n;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g[mid].slot <= slot_row) lo = mid; else hi = mid;
    }
    return lo;
}

// Splits x into three bf16 pieces whose sum reproduces x to about 24 bits.
__device__ __forceinline__ void split3(float x, __nv_bfloat16 (&h)[3]) {
    h[0] = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(h[0]);
    h[1] = __float2bfloat16_rn(r1);
    h[2] = __float2bfloat16_rn(r1 - __bfloat162float(h[1]));
}

// Augmentation tile layout (4 KB per 128 query rows, K-major without swizzle): element e (0..15)
// of row r lives at byte (e/8)*2048 + (r/8)*128 + (r%8)*16 + (e%8)*2.  Elements 0..2 hold the
// pieces of -LSE/scale, elements 8..10 the pieces of -D, everything else is zero.  Rows past the
// end of the query range get -1e30 and 0, which makes their P and dS vanish.
template <int D>
__global__ void __launch_bounds__(kPreThreads) zl_bwd_pre_kernel(const BwdParams p) {
    // One warp per (8 consecutive padded query rows, head): four lanes share a row, each reading a
    // quarter of its O and dO (16-byte loads), and the two 16-byte halves of the eight rows land in the
    // augmentation tile as two contiguous 128-byte stores.  A warp handles two such units per iteration and
    // issues all loads of both (O, dO and LSE: 8 KB + 64 B at d=128) before the first use.
    constexpr int kPerLane = D / 4;  // bf16 elements of one row handled by one lane
    constexpr int kVec = kPerLane / 8;
    constexpr int kUnits = 2;
    const int lane = threadIdx.x & 31;
    const int sub = lane >> 2, quarter = lane & 3;
    const int64_t n_units = (int64_t)(p.q_pad_total / 8) * p.n_heads;
    const int64_t stride = (int64_t)gridDim.x * (kPreThreads / 32);
    const float inv_scale = 1.f / p.scale;
    for (int64_t u0 = (int64_t)blockIdx.x * (kPreThreads / 32) + (threadIdx.x >> 5); u0 < n_units; u0 += kUnits * stride) {
        uint4 a[kUnits][kVec], b[kUnits][kVec];
        float lse[kUnits];
        bool live[kUnits], run[kUnits];
        int slot_row[kUnits], head[kUnits];
#pragma unroll
        for (int k = 0; k < kUnits; ++k) {
            const int64_t u = u0 + k * stride;
            run[k] = false;
            live[k] = false;
            lse[k] = 0.f;
            slot_row[k] = 0;
            head[k] = 0;
            if (u >= n_units) continue;
            const int row8 = (int)(u / p.n_heads);
            const int h = (int)(u - (int64_t)row8 * p.n_heads);
            // slots are padded to 128 rows: the eight rows belong to one query group
            const QGroup g = p.q_groups[find_q_group(p.q_groups, p.n_q_groups, row8 * 8)];
            if (h < g.head_begin || h >= g.head_begin + g.head_count) continue;  // warp-uniform: no task runs this head
            run[k] = true;
            head[k] = h;
            slot_row[k] = row8 * 8 + sub;
            const int r = slot_row[k] - g.slot;
            live[k] = r < g.q_len;
            if (live[k]) {
                const int64_t row = (int64_t)g.q_off + r;
                const uint4* po = reinterpret_cast<const uint4*>(p.o + (row * p.n_heads + h) * D + quarter * kPerLane);
                const uint4* pd = reinterpret_cast<const uint4*>(p.d_o + (row * p.n_heads + h) * D + quarter * kPerLane);
#pragma unroll
                for (int i = 0; i < kVec; ++i) { a[k][i] = __ldg(po + i); b[k][i] = __ldg(pd + i); }
                if (quarter == 0) lse[k] = __ldg(p.lse + (int64_t)h * p.total_q + row);
            }
        }
#pragma unroll
        for (int k = 0; k < kUnits; ++k) {
            if (!run[k]) continue;  // warp-uniform
            float acc = 0.f;
            if (live[k]) {
#pragma unroll
                for (int i = 0; i < kVec; ++i) {
                    const uint32_t aw[4] = {a[k][i].x, a[k][i].y, a[k][i].z, a[k][i].w};
                    const uint32_t bw[4] = {b[k][i].x, b[k][i].y, b[k][i].z, b[k][i].w};
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[w]));
                        const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[w]));
                        acc = fmaf(fa.x, fb.x, acc);
                        acc = fmaf(fa.y, fb.y, acc);
                    }
                }
            }
            acc += __shfl_xor_sync(0xffffffffu, acc, 1);
            acc += __shfl_xor_sync(0xffffffffu, acc, 2);
            // rows past the end of the query range: -1e30 and 0, which makes their P and dS vanish
            float xd = 0.f, xl = -1e30f;
            if (live[k]) {
                xd = -acc;
                const float l = lse[k];
                if (l > -INFINITY && l < INFINITY) xl = -l * inv_scale;
            }
            // lane quarter 0 writes elements 0..7 of its row (-LSE/scale pieces), quarter 1 elements 8..15 (-D pieces)
            if (quarter < 2) {
                __nv_bfloat16 hp[3];
                split3(quarter == 0 ? xl : xd, hp);
                uint4 val;
                val.x = (uint32_t)__bfloat16_as_ushort(hp[0]) | ((uint32_t)__bfloat16_as_ushort(hp[1]) << 16);
                val.y = (uint32_t)__bfloat16_as_ushort(hp[2]);
                val.z = 0u;
                val.w = 0u;
                const int tile = slot_row[k] / kTileQ, tr = slot_row[k] % kTileQ;
                uint8_t* base = p.aug + ((int64_t)head[k] * (p.q_pad_total / kTileQ) + tile) * 4096;
                *reinterpret_cast<uint4*>(base + quarter * 2048 + (tr / 8) * 128 + (tr % 8) * 16) = val;
            }
        }
    }
}

// ======================================================================= post
template <int D>
__global__ void __launch_bounds__(kPreThreads) zl_bwd_post_kernel(const BwdParams p) {
    // One warp per padded query row: every head of the row in batches of four, all four 16-byte loads
    // of a batch issued before the first conversion (2 KB in flight per warp at d=128).
    constexpr int V = D / 32;
    constexpr int kBatch = 4;
    const int lane = threadIdx.x & 31;
    for (int64_t slot_row = (int64_t)blockIdx.x * (kPreThreads / 32) + (threadIdx.x >> 5); slot_row < p.q_pad_total;
         slot_row += (int64_t)gridDim.x * (kPreThreads / 32)) {
        const QGroup g = p.q_groups[find_q_group(p.q_groups, p.n_q_groups, (int)slot_row)];
        const int r = (int)slot_row - g.slot;
        if (r >= g.q_len) continue;
        const float* src = p.dq_acc + slot_row * p.n_heads * D + lane * V;
        __nv_bfloat16* dst = p.dq + ((int64_t)g.q_off + r) * p.grad_row_stride + lane * V;
        const int h_end = g.head_begin + g.head_count;  // heads outside the group's range are left untouched
        for (int h0 = g.head_begin; h0 < h_end; h0 += kBatch) {
            if constexpr (V == 4) {
                float4 x[kBatch];
#pragma unroll
                for (int i = 0; i < kBatch; ++i)
                    if (h0 + i < h_end) x[i] = __ldcs(reinterpret_cast<const float4*>(src + (int64_t)(h0 + i) * D));
#pragma unroll
                for (int i = 0; i < kBatch; ++i)
                    if (h0 + i < h_end) {
                        uint2 o2;
                        o2.x = pack_bf16(x[i].x * p.scale, x[i].y * p.scale);
                        o2.y = pack_bf16(x[i].z * p.scale, x[i].w * p.scale);
                        *reinterpret_cast<uint2*>(dst + (int64_t)(h0 + i) * D) = o2;
                    }
            } else {
                float2 x[kBatch];
#pragma unroll
                for (int i = 0; i < kBatch; ++i)
                    if (h0 + i < h_end) x[i] = __ldcs(reinterpret_cast<const float2*>(src + (int64_t)(h0 + i) * D));
#pragma unroll
                for (int i = 0; i < kBatch; ++i)
                    if (h0 + i < h_end)
                        *reinterpret_cast<uint32_t*>(dst + (int64_t)(h0 + i) * D) = pack_bf16(x[i].x * p.scale, x[i].y * p.scale);
            }
        }
    }
}

// ======================================================================= main
// Warp roles (16 warps): warp 0 TMA producer, warp 1 MMA issuer, warps 2-3 idle,
// warps 4-7 and 8-11 two P/dS warpgroups (query columns 0-63 and 64-127 of every tile, one key
// row per thread), warps 12-15 dQ warpgroup (one query row per thread).
constexpr int kBwdThreads = 512;

template <int D>
struct BwdSmem {
    static constexpr int kTileBytes = 128 * D * 2;
    static constexpr int kBoxBytes = 128 * 128;
    static constexpr int kBoxes = D / 64;
    static constexpr int kDqChunkBytes = 128 * 32 * 4;  // 128 query rows x 32 fp32 columns
    alignas(1024) uint8_t k[kTileBytes];
    alignas(1024) uint8_t v[kTileBytes];
    alignas(1024) uint8_t q[2][kTileBytes];
    alignas(1024) uint8_t d_o[kTileBytes];
    alignas(1024) uint8_t ds[2 * kBoxBytes];            // dS^T tile: 128 key rows x 128 query columns, bf16
    alignas(1024) uint8_t dq_stage[kDqChunkBytes];      // one fp32 dQ chunk staged for the TMA reduce
    alignas(1024) uint8_t aug[2][4096];                 // per Q stage: bf16 pieces of -LSE/scale and -D
    alignas(1024) uint8_t ones[3][2048];                // [zeros][ones in elements 0..2][zeros]
    alignas(8) uint64_t kv_full, kv_empty;
    uint64_t q_full[2], q_empty[2], do_full, do_empty;
    uint64_t s_full, dp_full, p_full, ds_full, ds_free, dq_full, dq_empty, acc_full;
    uint32_t tmem_base;
    volatile int32_t abort_flag;
};

__device__ __forceinline__ void report(int32_t* status, volatile int32_t* abort_flag, int where) {
    *abort_flag = 1;
    if (atomicCAS(status, 0, (int)ZL_ERR_TIMEOUT) == 0) status[1] = where;
}

#define ZL_WAIT(bar, parity, site)                                        \
    do {                                                                  \
        if (!mbar_wait((bar), (parity), kWaitLimitNs, &sm.abort_flag)) { \
            report(p.status, &sm.abort_flag, 2000 + (site));              \
            goto teardown;                                                \
        }                                                                 \
    } while (0)
#define ZL_WAIT_WARP(bar, parity, site)                                              \
    do {                                                                             \
        const bool ok_ = mbar_wait((bar), (parity), kWaitLimitNs, &sm.abort_flag); \
        if (!__all_sync(0xffffffffu, ok_)) {                                         \
            report(p.status, &sm.abort_flag, 2000 + (site));                         \
            goto teardown;                                                           \
        }                                                                            \
    } while (0)

// Number of 128-row query tiles a kv group's CTA iterates over.
__device__ __forceinline__ int count_q_tiles(const BwdParams& p, const KvGroup& g) {
    int n = 0;
    for (int ti = 0; ti < g.n_tasks; ++ti)
        n += (p.tasks[p.kv_group_tasks[g.task_begin + ti]].q_len + kTileQ - 1) / kTileQ;
    return n;
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
zl_bwd_main_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                   const __grid_constant__ CUtensorMap tm_dq, const __grid_constant__ CUtensorMap tm_dk,
                   const __grid_constant__ CUtensorMap tm_dv, const BwdParams p) {
    using Smem = BwdSmem<D>;
    constexpr int kBoxes = Smem::kBoxes;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // TMEM columns: S^T / P^T [0,128), dP^T / dQ [128,256), dV [256,256+D), dK [384,384+D)
    constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384, kTmemCols = 512;

    if ((smem_u32(smem_raw) & 1023u) != 0) {  // swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0 && atomicCAS(p.status, 0, (int)ZL_ERR_CUDA) == 0) p.status[1] = 2999;
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(&sm.kv_full, 1);
        mbar_init(&sm.kv_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&sm.q_full[s], 1);
            mbar_init(&sm.q_empty[s], 1);
        }
        mbar_init(&sm.do_full, 1);
        mbar_init(&sm.do_empty, 1);
        mbar_init(&sm.s_full, 1);
        mbar_init(&sm.dp_full, 1);
        mbar_init(&sm.p_full, 256);
        mbar_init(&sm.ds_full, 256);
        mbar_init(&sm.ds_free, 1);
        mbar_init(&sm.dq_full, 1);
        mbar_init(&sm.dq_empty, 128);
        mbar_init(&sm.acc_full, 1);
        sm.abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_do);
        prefetch_tmap(&tm_dq);
        prefetch_tmap(&tm_dk);
        prefetch_tmap(&tm_dv);
    }
    // constant A operand of the augmentation steps: 128 rows x 8 bf16 per block
    for (int i = threadIdx.x; i < 3 * 2048 / 4; i += kBwdThreads) {
        const int blk = i / 512, w = i % 4;  // w: 32-bit word inside the row's 16 bytes
        uint32_t val = 0;
        if (blk == 1) val = (w == 0) ? 0x3F803F80u : (w == 1 ? 0x00003F80u : 0u);
        reinterpret_cast<uint32_t*>(&sm.ones[0][0])[i] = val;
    }
    fence_proxy_async_smem();
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp < 4) {
        reg_dec<104>();
        if (warp == 0 && lane == 0) {
            // -------------------------------------------------------------- TMA producer
            uint32_t item_cnt = 0, it_cnt = 0;
            for (int it = blockIdx.x; it < p.n_items; it += gridDim.x, ++item_cnt) {
                const WorkItem wi = p.items[it];
                const KvGroup g = p.kv_groups[wi.unit];
                ZL_WAIT(&sm.kv_empty, (item_cnt & 1) ^ 1, 1);
                mbar_arrive_expect_tx(&sm.kv_full, 2 * Smem::kTileBytes);
                for (int b = 0; b < kBoxes; ++b) {
                    tma_load_3d(sm.k + b * Smem::kBoxBytes, &tm_k, &sm.kv_full, b * 64, wi.head, g.kv_off + wi.row0);
                    tma_load_3d(sm.v + b * Smem::kBoxBytes, &tm_v, &sm.kv_full, b * 64, wi.head, g.kv_off + wi.row0);
                }
                for (int ti = 0; ti < g.n_tasks; ++ti) {
                    const Task t = p.tasks[p.kv_group_tasks[g.task_begin + ti]];
                    const int n_q = (t.q_len + kTileQ - 1) / kTileQ;
                    for (int qt = 0; qt < n_q; ++qt, ++it_cnt) {
                        const int s = it_cnt & 1;
                        ZL_WAIT(&sm.q_empty[s], ((it_cnt >> 1) & 1) ^ 1, 2);
                        mbar_arrive_expect_tx(&sm.q_full[s], Smem::kTileBytes + 4096);
                        for (int b = 0; b < kBoxes; ++b)
                            tma_load_3d(sm.q[s] + b * Smem::kBoxBytes, &tm_q, &sm.q_full[s], b * 64, wi.head,
                                        t.q_off + qt * kTileQ);
                        const int64_t tile = (int64_t)wi.head * (p.q_pad_total / kTileQ) + t.q_slot / kTileQ + qt;
                        bulk_load_1d(sm.aug[s], p.aug + tile * 4096, 4096, &sm.q_full[s]);
                        ZL_WAIT(&sm.do_empty, (it_cnt & 1) ^ 1, 3);
                        mbar_arrive_expect_tx(&sm.do_full, Smem::kTileBytes);
                        for (int b = 0; b < kBoxes; ++b)
                            tma_load_3d(sm.d_o + b * Smem::kBoxBytes, &tm_do, &sm.do_full, b * 64, wi.head,
                                        t.q_off + qt * kTileQ);
                    }
                }
            }
        } else if (warp == 1) {
            // -------------------------------------------------------------- MMA issuer
            // The whole warp runs this loop converged and one elected lane issues: descriptors
            // and barrier addresses then stay warp-uniform, which makes commits and satisfied
            // waits several times cheaper than from a single diverged thread.
            const bool mma_lane = elect_one();
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);   // S^T, dP^T: K-major x K-major
            constexpr uint32_t idesc_dv = make_idesc_bf16(128, D, 0, 1);    // A in TMEM / K-major smem, B MN-major
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, 1, 1);    // A MN-major smem, B MN-major
            // Descriptors are built once; stepping along K only adds a byte offset (>> 4) to the
            // start-address field, which cannot overflow for shared-memory addresses.
            const uint64_t dk_k = make_desc_sw128(smem_u32(sm.k), 16, 1024);                   // K tile, K-major
            const uint64_t dk_mn = make_desc_sw128(smem_u32(sm.k), Smem::kBoxBytes, 1024);     // K tile, MN-major
            const uint64_t dv_k = make_desc_sw128(smem_u32(sm.v), 16, 1024);
            const uint64_t ddo_k = make_desc_sw128(smem_u32(sm.d_o), 16, 1024);
            const uint64_t ddo_mn = make_desc_sw128(smem_u32(sm.d_o), Smem::kBoxBytes, 1024);
            const uint64_t dds_k = make_desc_sw128(smem_u32(sm.ds), 16, 1024);
            const uint64_t dds_mn = make_desc_sw128(smem_u32(sm.ds), Smem::kBoxBytes, 1024);
            const uint64_t dq_k0 = make_desc_sw128(smem_u32(sm.q[0]), 16, 1024);
            const uint64_t dq_mn0 = make_desc_sw128(smem_u32(sm.q[0]), Smem::kBoxBytes, 1024);
            const uint64_t daug0 = make_desc_noswizzle(smem_u32(sm.aug[0]), 2048, 128);
            const uint64_t dones_s = make_desc_noswizzle(smem_u32(&sm.ones[1][0]), 2048, 128);  // ones, then zeros
            const uint64_t dones_dp = make_desc_noswizzle(smem_u32(&sm.ones[0][0]), 2048, 128); // zeros, then ones
            constexpr uint32_t kQStageStep = Smem::kTileBytes >> 4, kAugStageStep = 4096 >> 4;
            // S^T = K Q^T - LSE/scale: the last step multiplies the ones block with the LSE pieces
            auto issue_s = [&](uint32_t stage) {
                const uint64_t dq = dq_k0 + stage * kQStageStep;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = ((ks / 4) * Smem::kBoxBytes + (ks % 4) * 32) >> 4;
                    if (mma_lane) mma_ss(tmem + kColS, dk_k + off, dq + off, idesc_s, ks > 0);
                }
                if (mma_lane) mma_ss(tmem + kColS, dones_s, daug0 + stage * kAugStageStep, idesc_s, true);
                if (mma_lane) mma_commit(&sm.s_full);
            };
            // dP^T = V dO^T - D: the ones sit in the second K chunk, where the tile holds the D pieces
            auto issue_dp = [&](uint32_t stage) {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = ((ks / 4) * Smem::kBoxBytes + (ks % 4) * 32) >> 4;
                    if (mma_lane) mma_ss(tmem + kColDP, dv_k + off, ddo_k + off, idesc_s, ks > 0);
                }
                if (mma_lane) mma_ss(tmem + kColDP, dones_dp, daug0 + stage * kAugStageStep, idesc_s, true);
                if (mma_lane) mma_commit(&sm.dp_full);
            };
            auto issue_dv = [&](bool acc) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // dV += P^T dO, K = 128 query rows
                    if (mma_lane) mma_ts(tmem + kColDV, tmem + kColS + (ks / 4) * 64 + (ks % 4) * 8, ddo_mn + ks * (2048 >> 4), idesc_dv,
                           acc || ks > 0);
                if (mma_lane) mma_commit(&sm.do_empty);
            };
            uint32_t item_cnt = 0, it_cnt = 0;
            for (int it = blockIdx.x; it < p.n_items; it += gridDim.x, ++item_cnt) {
                const WorkItem wi = p.items[it];
                const KvGroup g = p.kv_groups[wi.unit];
                const int n_it = count_q_tiles(p, g);
                ZL_WAIT_WARP(&sm.kv_full, item_cnt & 1, 11);
                // prologue: S, dP, dV of the item's first query tile and S of the second.
                // Steady-state order on the tensor pipe: dQ(i) dK(i) dP(i+1) dV(i+1) S(i+2).
                ZL_WAIT_WARP(&sm.q_full[it_cnt & 1], (it_cnt >> 1) & 1, 12);
                tc_fence_after();
                issue_s(it_cnt & 1);
                ZL_WAIT_WARP(&sm.do_full, it_cnt & 1, 13);
                ZL_WAIT_WARP(&sm.dq_empty, (it_cnt & 1) ^ 1, 14);  // previous dQ tile drained from the dP columns
                tc_fence_after();
                issue_dp(it_cnt & 1);
                ZL_WAIT_WARP(&sm.p_full, it_cnt & 1, 15);
                tc_fence_after();
                issue_dv(false);
                if (n_it > 1) {
                    const uint32_t n1 = it_cnt + 1;
                    ZL_WAIT_WARP(&sm.q_full[n1 & 1], (n1 >> 1) & 1, 16);
                    tc_fence_after();
                    issue_s(n1 & 1);  // overwrites P^T: ordered after dV on the tensor pipe
                }
                for (int i = 0; i < n_it; ++i, ++it_cnt) {
                    const uint64_t dq_mn = dq_mn0 + (it_cnt & 1) * kQStageStep;
                    ZL_WAIT_WARP(&sm.ds_full, it_cnt & 1, 17);
                    tc_fence_after();
                    {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)  // dQ = dS K, K = 128 key rows; lands in the dP columns
                            if (mma_lane) mma_ss(tmem + kColDP, dds_mn + ks * (2048 >> 4), dk_mn + ks * (2048 >> 4), idesc_dq, ks > 0);
                        if (mma_lane) mma_commit(&sm.dq_full);  // dQ first: its drain from TMEM runs under the dK MMAs
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {  // dK += dS^T Q, K = 128 query rows
                            const uint32_t off = ((ks / 4) * Smem::kBoxBytes + (ks % 4) * 32) >> 4;
                            if (mma_lane) mma_ss(tmem + kColDK, dds_k + off, dq_mn + ks * (2048 >> 4), idesc_dv, i > 0 || ks > 0);
                        }
                        if (mma_lane) mma_commit(&sm.q_empty[it_cnt & 1]);
                        if (mma_lane) mma_commit(&sm.ds_free);
                    }
                    if (i + 1 < n_it) {
                        const uint32_t n1 = it_cnt + 1, n2 = it_cnt + 2;
                        ZL_WAIT_WARP(&sm.do_full, n1 & 1, 18);
                        ZL_WAIT_WARP(&sm.dq_empty, it_cnt & 1, 19);
                        tc_fence_after();
                        issue_dp(n1 & 1);
                        ZL_WAIT_WARP(&sm.p_full, n1 & 1, 20);
                        tc_fence_after();
                        issue_dv(true);
                        if (i + 2 < n_it) {
                            ZL_WAIT_WARP(&sm.q_full[n2 & 1], (n2 >> 1) & 1, 16);
                            tc_fence_after();
                            issue_s(n2 & 1);
                        }
                    }
                }
                if (mma_lane) mma_commit(&sm.acc_full);
                if (mma_lane) mma_commit(&sm.kv_empty);
            }
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------------ P / dS warpgroups
        reg_inc<128>();
        const int wg = (warp - 4) >> 2;            // 0: query columns 0-63, 1: columns 64-127
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;       // key row within the tile
        const int col0 = wg * 64;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        const uint32_t ds_row_addr = smem_u32(sm.ds) + row * 128;
        const float sl2 = p.scale_log2;
        uint32_t item_cnt = 0, it_cnt = 0;
        const bool store_leader = (warp & 3) == 0 && lane == 0;  // one thread per warpgroup issues its TMA stores
        bool store_pending = false;
        for (int it = blockIdx.x; it < p.n_items; it += gridDim.x, ++item_cnt) {
            const WorkItem wi = p.items[it];
            const KvGroup g = p.kv_groups[wi.unit];
            const bool row_ok = row < wi.rows;
            for (int ti = 0; ti < g.n_tasks; ++ti) {
                const Task t = p.tasks[p.kv_group_tasks[g.task_begin + ti]];
                const int n_q = (t.q_len + kTileQ - 1) / kTileQ;
                for (int qt = 0; qt < n_q; ++qt, ++it_cnt) {
                    const int q_valid = min(kTileQ, t.q_len - qt * kTileQ);
                    const bool tile_full = (wi.rows == kTileKV) && (q_valid == kTileQ);  // warp-uniform
                    ZL_WAIT_WARP(&sm.s_full, it_cnt & 1, 22);
                    tc_fence_after();
                    uint32_t pk[32];  // P^T of this thread's row, bf16 pairs
                    {
                        uint32_t sr[2][32];
                        tmem_ld_x32(lane_addr + kColS + col0, sr[0]);
                        tmem_ld_x32(lane_addr + kColS + col0 + 32, sr[1]);
                        tmem_wait_ld();
                        if (tile_full) {
#pragma unroll
                            for (int c = 0; c < 2; ++c)
#pragma unroll
                                for (int i = 0; i < 32; i += 2)  // S^T already has -LSE/scale folded in
                                    pk[c * 16 + i / 2] = pack_bf16(ex2(__uint_as_float(sr[c][i]) * sl2),
                                                                   ex2(__uint_as_float(sr[c][i + 1]) * sl2));
                        } else {
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
#pragma unroll
                                for (int i = 0; i < 32; i += 2) {
                                    const int col = col0 + c * 32 + i;
                                    float p0 = ex2(__uint_as_float(sr[c][i]) * sl2);
                                    float p1 = ex2(__uint_as_float(sr[c][i + 1]) * sl2);
                                    p0 = (row_ok && col < q_valid) ? p0 : 0.f;  // select, never multiply
                                    p1 = (row_ok && col + 1 < q_valid) ? p1 : 0.f;
                                    pk[c * 16 + i / 2] = pack_bf16(p0, p1);
                                }
                            }
                        }
                        tmem_st_x32(lane_addr + kColS + col0, pk);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(&sm.p_full);

                    ZL_WAIT_WARP(&sm.dp_full, it_cnt & 1, 23);
                    if (it_cnt > 0) ZL_WAIT_WARP(&sm.ds_free, (it_cnt - 1) & 1, 24);  // dS buffer consumed by dK/dQ
                    if (store_pending) {
                        // this warpgroup's box of the dS tile staged the previous item's dK / dV tile
                        if (store_leader) bulk_wait_group_read<0>();
                        named_bar_sync(2 + wg, 128);
                        store_pending = false;
                    }
                    tc_fence_after();
                    {
                        uint32_t dr[2][32];
                        tmem_ld_x32(lane_addr + kColDP + col0, dr[0]);
                        tmem_ld_x32(lane_addr + kColDP + col0 + 32, dr[1]);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t dd[16];
                            if (tile_full) {
#pragma unroll
                                for (int i = 0; i < 32; i += 2)  // dS^T = P^T o (dP^T - D) in packed bf16 arithmetic
                                    dd[i / 2] = mul_bf16x2(pk[c * 16 + i / 2],
                                                           pack_bf16(__uint_as_float(dr[c][i]), __uint_as_float(dr[c][i + 1])));
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; i += 2) {
                                    const int col = col0 + c * 32 + i;
                                    float d0 = __uint_as_float(dr[c][i]), d1 = __uint_as_float(dr[c][i + 1]);
                                    d0 = (row_ok && col < q_valid) ? d0 : 0.f;  // P is already zero there; keep 0 * garbage out
                                    d1 = (row_ok && col + 1 < q_valid) ? d1 : 0.f;
                                    dd[i / 2] = mul_bf16x2(pk[c * 16 + i / 2], pack_bf16(d0, d1));
                                }
                            }
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4) {
                                const int c16 = (col0 >> 3) + c * 4 + k4;  // 16-byte chunk index along the query axis
                                const uint32_t addr = ds_row_addr + (c16 >> 3) * Smem::kBoxBytes + (((c16 & 7) ^ (row & 7)) << 4);
                                st_shared_v4(addr, dd[k4 * 4], dd[k4 * 4 + 1], dd[k4 * 4 + 2], dd[k4 * 4 + 3]);
                            }
                        }
                        tc_fence_before();
                        fence_proxy_async_smem();
                        mbar_arrive(&sm.ds_full);
                    }
                }
            }
            // ---- epilogue: warpgroup 0 stores dV, warpgroup 1 stores dK (scaled)
            ZL_WAIT_WARP(&sm.acc_full, item_cnt & 1, 25);
            tc_fence_after();
            const float sc = (wg == 0) ? 1.f : p.scale;
            const uint32_t col_acc = (wg == 0) ? kColDV : kColDK;
            if (wi.rows == kTileKV) {
                // full key tile: stage 64 columns at a time in this warpgroup's box of the (now idle) dS
                // tile and write them with one TMA store each -- coalesced, and the warpgroup moves on to
                // the next item while the copy engine drains the box
                const uint32_t box_addr = smem_u32(sm.ds) + wg * Smem::kBoxBytes + row * 128;
#pragma unroll
                for (int b = 0; b < kBoxes; ++b) {
                    if (b > 0) {
                        if (store_leader) bulk_wait_group_read<0>();
                        named_bar_sync(2 + wg, 128);
                    }
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(lane_addr + col_acc + b * 64 + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            const int i = k4 * 8;
                            st_shared_v4(box_addr + (((c * 4 + k4) ^ (row & 7)) << 4),
                                         pack_bf16(__uint_as_float(r[i]) * sc, __uint_as_float(r[i + 1]) * sc),
                                         pack_bf16(__uint_as_float(r[i + 2]) * sc, __uint_as_float(r[i + 3]) * sc),
                                         pack_bf16(__uint_as_float(r[i + 4]) * sc, __uint_as_float(r[i + 5]) * sc),
                                         pack_bf16(__uint_as_float(r[i + 6]) * sc, __uint_as_float(r[i + 7]) * sc));
                        }
                    }
                    fence_proxy_async_smem();
                    named_bar_sync(2 + wg, 128);
                    if (store_leader) {
                        tma_store_3d(wg == 0 ? &tm_dv : &tm_dk, sm.ds + wg * Smem::kBoxBytes, b * 64, wi.head,
                                     g.kv_off + wi.row0);
                        bulk_commit_group();
                    }
                }
                store_pending = true;
            } else {
                const int64_t grow = (int64_t)g.kv_off + wi.row0 + row;
                __nv_bfloat16* dst = (wg == 0 ? p.dv : p.dk) + grow * p.grad_row_stride + wi.head * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(lane_addr + col_acc + c * 32, r);
                    tmem_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            uint4 o4;
                            o4.x = pack_bf16(__uint_as_float(r[i]) * sc, __uint_as_float(r[i + 1]) * sc);
                            o4.y = pack_bf16(__uint_as_float(r[i + 2]) * sc, __uint_as_float(r[i + 3]) * sc);
                            o4.z = pack_bf16(__uint_as_float(r[i + 4]) * sc, __uint_as_float(r[i + 5]) * sc);
                            o4.w = pack_bf16(__uint_as_float(r[i + 6]) * sc, __uint_as_float(r[i + 7]) * sc);
                            *reinterpret_cast<uint4*>(dst + c * 32 + i) = o4;
                        }
                    }
                }
            }
            tc_fence_before();
        }
        if (store_leader) bulk_wait_group<0>();  // the last dK / dV stores have left shared memory and landed
    } else {
        // ------------------------------------------------------------------ dQ warpgroup (one query row per thread)
        reg_inc<152>();
        const int quarter = warp & 3;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        const bool leader = (lane == 0);  // per warp
        uint32_t it_cnt = 0, chunk_cnt = 0;
        for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
            const WorkItem wi = p.items[it];
            const KvGroup g = p.kv_groups[wi.unit];
            for (int ti = 0; ti < g.n_tasks; ++ti) {
                const Task t = p.tasks[p.kv_group_tasks[g.task_begin + ti]];
                const int n_q = (t.q_len + kTileQ - 1) / kTileQ;
                for (int qt = 0; qt < n_q; ++qt, ++it_cnt) {
                    ZL_WAIT_WARP(&sm.dq_full, it_cnt & 1, 31);
                    tc_fence_after();
                    {
                        // read the whole tile (frees the TMEM columns for the next dP^T), then stage
                        // 32-column chunks in swizzled shared memory and add them with the TMA
                        uint32_t r[D];
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t tmp[32];
                            tmem_ld_x32(lane_addr + kColDP + c * 32, tmp);
#pragma unroll
                            for (int i = 0; i < 32; ++i) r[c * 32 + i] = tmp[i];
                        }
                        tmem_wait_ld();
                        tc_fence_before();
                        mbar_arrive(&sm.dq_empty);
#pragma unroll
                        for (int c = 0; c < D / 32; ++c, ++chunk_cnt) {
                            // each warp stages its own 32 rows and adds them with its own reduce: no
                            // warpgroup barrier, and the four streams overlap in the copy engine
                            uint8_t* buf = sm.dq_stage + quarter * 4096;
                            if (chunk_cnt >= 1) {
                                if (leader) bulk_wait_group_read<0>();  // the previous reduce has read the buffer
                                __syncwarp();
                            }
                            const uint32_t row_addr = smem_u32(buf) + lane * 128;
#pragma unroll
                            for (int k4 = 0; k4 < 8; ++k4)
                                st_shared_v4(row_addr + ((k4 ^ (lane & 7)) << 4), r[c * 32 + k4 * 4], r[c * 32 + k4 * 4 + 1],
                                             r[c * 32 + k4 * 4 + 2], r[c * 32 + k4 * 4 + 3]);
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (leader) {
                                tma_reduce_add_3d(&tm_dq, buf, c * 32, wi.head, t.q_slot + qt * kTileQ + quarter * 32);
                                bulk_commit_group();
                            }
                        }
                    }
                }
            }
        }
        if (leader) bulk_wait_group<0>();
    }

teardown:
    // Also reached after an expired wait: bulk stores and reduces this thread has committed must have
    // finished reading shared memory before the CTA gives it up (a no-op on the normal path).
    bulk_wait_group<0>();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// The opt-in to large dynamic shared memory is a per-device attribute of the kernel.
constexpr int kMaxDevices = 64;

template <int D>
cudaError_t launch_main_t(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                          const CUtensorMap& tdo, const CUtensorMap& tdq, const CUtensorMap& tdk,
                          const CUtensorMap& tdv, const BwdParams& p, int grid, cudaStream_t stream) {
    constexpr int smem = sizeof(BwdSmem<D>);
    static bool configured[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices || !configured[dev]) {
        e = cudaFuncSetAttribute(zl_bwd_main_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < kMaxDevices) configured[dev] = true;
    }
    zl_bwd_main_kernel<D><<<grid, kBwdThreads, smem, stream>>>(tq, tk, tv, tdo, tdq, tdk, tdv, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_bwd_pre(int head_dim, const BwdParams& p, int n_sms, cudaStream_t stream) {
    if (p.q_pad_total == 0) return cudaSuccess;
    const int grid = n_sms * 2;  // what is resident at once (two units per warp in flight need 92 registers): no block waves
    if (head_dim == 128) zl_bwd_pre_kernel<128><<<grid, kPreThreads, 0, stream>>>(p);
    else zl_bwd_pre_kernel<64><<<grid, kPreThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_bwd_main(int head_dim, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                            const CUtensorMap& tdo, const CUtensorMap& tdq, const CUtensorMap& tdk,
                            const CUtensorMap& tdv, const BwdParams& p, int grid, cudaStream_t stream) {
    if (p.n_items == 0) return cudaSuccess;
    return head_dim == 128 ? launch_main_t<128>(tq, tk, tv, tdo, tdq, tdk, tdv, p, grid, stream)
                           : launch_main_t<64>(tq, tk, tv, tdo, tdq, tdk, tdv, p, grid, stream);
}

cudaError_t launch_bwd_post(int head_dim, const BwdParams& p, int n_sms, cudaStream_t stream) {
    if (p.q_pad_total == 0) return cudaSuccess;
    const int grid = n_sms * 8;
    if (head_dim == 128) zl_bwd_post_kernel<128><<<grid, kPreThreads, 0, stream>>>(p);
    else zl_bwd_post_kernel<64><<<grid, kPreThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace zl
