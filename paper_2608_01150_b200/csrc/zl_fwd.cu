// Forward kernel of the coalesced attention engine (sm_100a).
//
// One persistent launch walks a longest-first list of work items (task, head, 256-row query
// block) that spans whole sequences and context-parallel shard tasks alike (paper Section
// IV-D: all whole sequences of a rank are packed into one block-diagonal attention call next
// to the rank's shards, without mixing attention across sequences).
//
// A CTA keeps TWO 128-row query tiles in flight so that the softmax of one overlaps the
// tensor-core work of the other:
//   warp 0      TMA producer: Q tiles once per item, K/V tiles through a shared-memory ring
//   warp 1      MMA issuer:   S_x = Q_x K^T (tcgen05.mma, smem x smem -> TMEM) and
//                             O_x += P_x V  (P read from TMEM, V from smem) for x in {A, B}
//   warps 4-7   softmax of tile A, warps 8-11 softmax of tile B: one thread per query row,
//               online softmax with a lazily updated reference maximum, P written back over S
//               in TMEM as bf16, final normalisation and stores.
// Whole-sequence tasks store final bf16 O and fp32 LSE; shard tasks store their partial result
// (normalised within their own K/V chunk) as fp32 O plus LSE for the merge kernel.
#include <cuda_runtime.h>

#include "zl_device.h"
#include "zl_ptx.cuh"

namespace zl {

using namespace ptx;

namespace {

constexpr int kFwdThreads = 384;
constexpr uint64_t kWaitLimitNs = 4000000000ull;
// The reference maximum of a row is only raised when the tile maximum exceeds it by more than
// this many powers of two; until then exponentials stay below 2^8 and nothing is rescaled.
constexpr float kRescaleThresholdLog2 = 8.0f;

template <int D>
struct FwdSmem {
    static constexpr int kStages = (D == 128) ? 2 : 4;
    static constexpr int kTileBytes = kTileQ * D * 2;  // one 128-row tile of Q, K or V
    static constexpr int kBoxBytes = kTileQ * 128;     // one TMA box: 128 rows x 64 bf16
    static constexpr int kBoxes = D / 64;
    alignas(1024) uint8_t q[2][kTileBytes];
    alignas(1024) uint8_t k[kStages][kTileBytes];
    alignas(1024) uint8_t v[kStages][kTileBytes];
    alignas(1024) uint8_t o_stage[2][kBoxBytes];  // per softmax warpgroup: 128 rows x 128 bytes of O on their way out
    alignas(8) uint64_t q_full[2], q_empty;
    uint64_t kv_full[kStages], kv_empty[kStages];  // K and V of a stage travel together
    uint64_t s_full[2], p_half[2][2], o_full[2];  // p_half[tile][half of the key columns]
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
        if (!mbar_wait((bar), (parity), kWaitLimitNs, &sm.abort_flag)) { \
            report(p.status, &sm.abort_flag, 1000 + (site));              \
            goto teardown;                                                \
        }                                                                 \
    } while (0)
// Wait used by all 32 lanes of a warp: the outcome is made warp-uniform and the warp
// reconverges before the .sync.aligned TMEM instructions that follow.
#define ZL_WAIT_WARP(bar, parity, site)                                              \
    do {                                                                             \
        const bool ok_ = mbar_wait((bar), (parity), kWaitLimitNs, &sm.abort_flag); \
        if (!__all_sync(0xffffffffu, ok_)) {                                         \
            report(p.status, &sm.abort_flag, 1000 + (site));                         \
            goto teardown;                                                           \
        }                                                                            \
    } while (0)

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
zl_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
              const __grid_constant__ CUtensorMap tm_op, const FwdParams p) {
    using Smem = FwdSmem<D>;
    constexpr int kStages = Smem::kStages;
    constexpr int kBoxes = Smem::kBoxes;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // TMEM columns: S_A [0,128), S_B [128,256), O_A [256,256+D), O_B [384,384+D).  P_x (bf16
    // pairs) overwrites the first 64 columns of S_x once the row has been read.
    constexpr uint32_t kColS = 0, kColO = 256, kTmemCols = 512;

    if ((smem_u32(smem_raw) & 1023u) != 0) {  // swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0 && atomicCAS(p.status, 0, (int)ZL_ERR_CUDA) == 0) p.status[1] = 1999;
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(&sm.q_full[0], 1);
        mbar_init(&sm.q_full[1], 1);
        mbar_init(&sm.q_empty, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.kv_full[s], 1);
            mbar_init(&sm.kv_empty[s], 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(&sm.s_full[x], 1);
            mbar_init(&sm.p_half[x][0], 128);
            mbar_init(&sm.p_half[x][1], 128);
            mbar_init(&sm.o_full[x], 1);
        }
        sm.abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_o);
        prefetch_tmap(&tm_op);
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp < 4) {
        reg_dec<72>();
        if (warp == 0 && lane == 0) {
            // -------------------------------------------------------------- TMA producer
            uint32_t q_cnt = 0, qb_cnt = 0, kv_cnt = 0;
            for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
                const WorkItem wi = p.items[it];
                const Task t = p.tasks[wi.unit];
                const int n_kv = (t.kv_len + kTileKV - 1) / kTileKV;
                if (n_kv == 0) continue;
                const bool has_b = wi.rows > kTileQ;
                ZL_WAIT(&sm.q_empty, (q_cnt & 1) ^ 1, 1);
                ++q_cnt;
                mbar_arrive_expect_tx(&sm.q_full[0], Smem::kTileBytes);
                for (int b = 0; b < kBoxes; ++b)
                    tma_load_3d(sm.q[0] + b * Smem::kBoxBytes, &tm_q, &sm.q_full[0], b * 64, wi.head, t.q_off + wi.row0);
                for (int j = 0; j < n_kv; ++j, ++kv_cnt) {
                    const int s = kv_cnt % kStages;
                    const uint32_t ph = (kv_cnt / kStages) & 1;
                    ZL_WAIT(&sm.kv_empty[s], ph ^ 1, 2);
                    mbar_arrive_expect_tx(&sm.kv_full[s], 2 * Smem::kTileBytes);
                    for (int b = 0; b < kBoxes; ++b)
                        tma_load_3d(sm.k[s] + b * Smem::kBoxBytes, &tm_k, &sm.kv_full[s], b * 64, wi.head,
                                    t.kv_off + j * kTileKV);
                    if (j == 0 && has_b) {  // second query tile right after the first K tile
                        mbar_arrive_expect_tx(&sm.q_full[1], Smem::kTileBytes);
                        for (int b = 0; b < kBoxes; ++b)
                            tma_load_3d(sm.q[1] + b * Smem::kBoxBytes, &tm_q, &sm.q_full[1], b * 64, wi.head,
                                        t.q_off + wi.row0 + kTileQ);
                        ++qb_cnt;
                    }
                    for (int b = 0; b < kBoxes; ++b)
                        tma_load_3d(sm.v[s] + b * Smem::kBoxBytes, &tm_v, &sm.kv_full[s], b * 64, wi.head,
                                    t.kv_off + j * kTileKV);
                }
            }
        } else if (warp == 1) {
            // -------------------------------------------------------------- MMA issuer
            // The whole warp runs this loop converged and one elected lane issues, which keeps
            // descriptors and barrier addresses warp-uniform (cheaper commits and satisfied waits).
            const bool mma_lane = elect_one();
            constexpr uint32_t idesc_s = make_idesc_bf16(kTileQ, kTileKV, 0, 0);
            constexpr uint32_t idesc_o = make_idesc_bf16(kTileQ, D, 0, 1);
            const uint64_t dq0 = make_desc_sw128(smem_u32(sm.q[0]), 16, 1024);
            const uint64_t dk0 = make_desc_sw128(smem_u32(sm.k[0]), 16, 1024);
            const uint64_t dv0 = make_desc_sw128(smem_u32(sm.v[0]), Smem::kBoxBytes, 1024);  // V is the MN-major B operand
            constexpr uint32_t kTileStep = Smem::kTileBytes >> 4;
            // S_x = Q_x K^T
            auto issue_s = [&](int x, uint32_t stage) {
                const uint64_t dq = dq0 + x * kTileStep, dk = dk0 + stage * kTileStep;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = ((ks / 4) * Smem::kBoxBytes + (ks % 4) * 32) >> 4;
                    if (mma_lane) mma_ss(tmem + kColS + x * 128, dq + off, dk + off, idesc_s, ks > 0);
                }
                if (mma_lane) mma_commit(&sm.s_full[x]);
            };
            // O_x (+)= P_x V
            // (one half of the key columns: P arrives in two halves so that the first four K steps
            // run while the softmax warps still work on the second half)
            auto issue_pv = [&](int x, uint32_t stage, bool acc, int half) {
                const uint64_t dv = dv0 + stage * kTileStep;
#pragma unroll
                for (int ks = half * (kTileKV / 32); ks < (half + 1) * (kTileKV / 32); ++ks)
                    if (mma_lane) mma_ts(tmem + kColO + x * 128, tmem + kColS + x * 128 + ks * 8, dv + ks * (2048 >> 4), idesc_o,
                           acc || ks > 0);
            };
            uint32_t q_cnt = 0, qb_cnt = 0, kv_cnt = 0, pa_cnt = 0, pb_cnt = 0;
            for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
                const WorkItem wi = p.items[it];
                const Task t = p.tasks[wi.unit];
                const int n_kv = (t.kv_len + kTileKV - 1) / kTileKV;
                if (n_kv == 0) continue;
                const bool has_b = wi.rows > kTileQ;
                ZL_WAIT_WARP(&sm.q_full[0], q_cnt & 1, 11);
                ++q_cnt;
                ZL_WAIT_WARP(&sm.kv_full[kv_cnt % kStages], (kv_cnt / kStages) & 1, 12);
                tc_fence_after();
                issue_s(0, kv_cnt % kStages);
                if (has_b) {
                    ZL_WAIT_WARP(&sm.q_full[1], qb_cnt & 1, 13);
                    ++qb_cnt;
                    issue_s(1, kv_cnt % kStages);
                }
                if (n_kv == 1) if (mma_lane) mma_commit(&sm.q_empty);
                for (int j = 0; j < n_kv; ++j, ++kv_cnt) {
                    const uint32_t s = kv_cnt % kStages, nk = kv_cnt + 1, sn = nk % kStages;
                    const bool has_next = j + 1 < n_kv;
                    // tile A: P_A(j) is in TMEM (S_A(j) fully read, O_A rescaled if needed); K(j), V(j)
                    // were waited for when S(j) was issued
                    ZL_WAIT_WARP(&sm.p_half[0][0], pa_cnt & 1, 14);
                    tc_fence_after();
                    issue_pv(0, s, j > 0, 0);
                    ZL_WAIT_WARP(&sm.p_half[0][1], pa_cnt & 1, 15);
                    ++pa_cnt;
                    tc_fence_after();
                    issue_pv(0, s, true, 1);
                    if (!has_next) if (mma_lane) mma_commit(&sm.o_full[0]);
                    if (has_next) {
                        ZL_WAIT_WARP(&sm.kv_full[sn], (nk / kStages) & 1, 16);
                        issue_s(0, sn);  // overwrites P_A(j): ordered after P_A V on the tensor pipe
                    }
                    if (has_b) {
                        ZL_WAIT_WARP(&sm.p_half[1][0], pb_cnt & 1, 17);
                        tc_fence_after();
                        issue_pv(1, s, j > 0, 0);
                        ZL_WAIT_WARP(&sm.p_half[1][1], pb_cnt & 1, 18);
                        ++pb_cnt;
                        tc_fence_after();
                        issue_pv(1, s, true, 1);
                        if (!has_next) if (mma_lane) mma_commit(&sm.o_full[1]);
                    }
                    if (mma_lane) mma_commit(&sm.kv_empty[s]);  // S_A(j), S_B(j), P_A V(j), P_B V(j) are the stage's last readers
                    if (has_next) {
                        if (has_b) issue_s(1, sn);
                        if (j + 2 == n_kv) if (mma_lane) mma_commit(&sm.q_empty);  // last S of the item issued
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        reg_inc<216>();
        const int x = (warp - 4) >> 2;             // 0: tile A, 1: tile B
        const int quarter = warp & 3;              // TMEM lane quarter this warp may access
        const int row = quarter * 32 + lane;       // query row within the tile
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        const uint32_t col_s = kColS + x * 128, col_o = kColO + x * 128;
        uint32_t s_cnt = 0, o_cnt = 0;
        const bool store_leader = quarter == 0 && lane == 0;  // one thread per warpgroup issues its TMA stores
        bool store_pending = false;                            // this warpgroup's box may still be read by a store
        const float sl2 = p.scale_log2;
        for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
            const WorkItem wi = p.items[it];
            const int tile_rows = min(kTileQ, wi.rows - x * kTileQ);  // rows of this warpgroup's tile
            if (tile_rows <= 0) continue;
            const Task t = p.tasks[wi.unit];
            const int n_kv = (t.kv_len + kTileKV - 1) / kTileKV;
            float m_ref = -INFINITY, l = 0.f;  // reference maximum (raw score units) and row sum
            for (int j = 0; j < n_kv; ++j) {
                ZL_WAIT_WARP(&sm.s_full[x], s_cnt & 1, 21);
                ++s_cnt;
                tc_fence_after();
                float sv[kTileKV];
#pragma unroll
                for (int c = 0; c < kTileKV / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(lane_addr + col_s + c * 32, r);
#pragma unroll
                    for (int i = 0; i < 32; ++i) sv[c * 32 + i] = __uint_as_float(r[i]);
                }
                tmem_wait_ld();
                const int valid = t.kv_len - j * kTileKV;  // columns of this tile inside the task
                if (valid < kTileKV) {
#pragma unroll
                    for (int c = 0; c < kTileKV; ++c)
                        if (c >= valid) sv[c] = -INFINITY;  // select, never multiply
                }
                // four independent chains: a single running maximum is a 64-deep dependent chain
                float mx0 = max3(sv[0], sv[1], sv[2]), mx1 = max3(sv[3], sv[4], sv[5]);
                float mx2 = max3(sv[6], sv[7], sv[8]), mx3 = max3(sv[9], sv[10], sv[11]);
#pragma unroll
                for (int c = 12; c + 7 < kTileKV; c += 8) {
                    mx0 = max3(mx0, sv[c], sv[c + 1]);
                    mx1 = max3(mx1, sv[c + 2], sv[c + 3]);
                    mx2 = max3(mx2, sv[c + 4], sv[c + 5]);
                    mx3 = max3(mx3, sv[c + 6], sv[c + 7]);
                }
                // columns 124..127 remain (12 + 8 * 14 = 124)
                mx0 = max3(mx0, sv[kTileKV - 4], sv[kTileKV - 3]);
                mx1 = max3(mx1, sv[kTileKV - 2], sv[kTileKV - 1]);
                const float mx = fmaxf(max3(mx0, mx1, mx2), mx3);
                // lazy reference update: only when the tile maximum is far above the reference
                const bool raise = (mx - m_ref) * sl2 > kRescaleThresholdLog2;
                if (__any_sync(0xffffffffu, raise && j > 0)) {
                    // rescale O (the previous P V product is complete: S(j) was issued after it)
                    const float alpha = raise ? ex2((m_ref - mx) * sl2) : 1.f;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(lane_addr + col_o + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st_x32(lane_addr + col_o + c * 32, r);
                    }
                    l *= alpha;
                }
                if (raise) {
                    if (j == 0) l = 0.f;
                    m_ref = mx;
                }
                const float nmb = -m_ref * sl2;
                float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll
                for (int h = 0; h < 2; ++h) {  // P goes to the MMA warp in two halves of 64 key columns
                    uint32_t pk[kTileKV / 4];
#pragma unroll
                    for (int c = 0; c < kTileKV / 2; c += 2) {
                        const int cc = h * (kTileKV / 2) + c;
                        const float2 e = fma2(make_float2(sv[cc], sv[cc + 1]), make_float2(sl2, sl2), make_float2(nmb, nmb));
                        const float p0 = ex2(e.x), p1 = ex2(e.y);
                        sum2 = add2(sum2, make_float2(p0, p1));
                        pk[c / 2] = pack_bf16(p0, p1);
                    }
                    tmem_st_x32(lane_addr + col_s + h * 32, pk);
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(&sm.p_half[x][h]);
                }
                l += sum2.x + sum2.y;
            }
            // ---- epilogue
            const bool row_ok = row < tile_rows;
            const float inv_l = (l > 0.f) ? 1.f / l : 0.f;
            const float lse = (l > 0.f) ? (m_ref * sl2 + log2f(l)) * 0.6931471805599453f : -INFINITY;
            if (n_kv > 0) {
                ZL_WAIT_WARP(&sm.o_full[x], o_cnt & 1, 23);
                ++o_cnt;
                tc_fence_after();
            }
            const int64_t grow0 = (int64_t)(t.partial_slot >= 0 ? t.partial_slot : t.q_off) + wi.row0 + x * kTileQ;
            const int64_t grow = grow0 + row;
            if (tile_rows == kTileQ && n_kv > 0) {
                // full tile: stage 128 bytes per row at a time in this warpgroup's box and write each box
                // with one TMA store -- coalesced, and the warpgroup is free for the next item while the
                // copy engine drains the box
                const uint32_t box_row = smem_u32(sm.o_stage[x]) + row * 128;
                if (t.partial_slot >= 0) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {  // 32 fp32 columns per box
                        if (c > 0 || store_pending) {
                            if (store_leader) bulk_wait_group_read<0>();
                            named_bar_sync(2 + x, 128);
                        }
                        uint32_t r[32];
                        tmem_ld_x32(lane_addr + col_o + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int k4 = 0; k4 < 8; ++k4)
                            st_shared_v4(box_row + ((k4 ^ (row & 7)) << 4),
                                         __float_as_uint(__uint_as_float(r[k4 * 4]) * inv_l),
                                         __float_as_uint(__uint_as_float(r[k4 * 4 + 1]) * inv_l),
                                         __float_as_uint(__uint_as_float(r[k4 * 4 + 2]) * inv_l),
                                         __float_as_uint(__uint_as_float(r[k4 * 4 + 3]) * inv_l));
                        fence_proxy_async_smem();
                        named_bar_sync(2 + x, 128);
                        if (store_leader) {
                            tma_store_3d(&tm_op, sm.o_stage[x], c * 32, wi.head, (int32_t)grow0);
                            bulk_commit_group();
                        }
                    }
                    p.lse_partial[(int64_t)wi.head * p.partial_rows + grow] = lse;
                } else {
#pragma unroll
                    for (int b = 0; b < D / 64; ++b) {  // 64 bf16 columns per box
                        if (b > 0 || store_pending) {
                            if (store_leader) bulk_wait_group_read<0>();
                            named_bar_sync(2 + x, 128);
                        }
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t r[32];
                            tmem_ld_x32(lane_addr + col_o + b * 64 + c * 32, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4) {
                                const int i = k4 * 8;
                                st_shared_v4(box_row + (((c * 4 + k4) ^ (row & 7)) << 4),
                                             pack_bf16(__uint_as_float(r[i]) * inv_l, __uint_as_float(r[i + 1]) * inv_l),
                                             pack_bf16(__uint_as_float(r[i + 2]) * inv_l, __uint_as_float(r[i + 3]) * inv_l),
                                             pack_bf16(__uint_as_float(r[i + 4]) * inv_l, __uint_as_float(r[i + 5]) * inv_l),
                                             pack_bf16(__uint_as_float(r[i + 6]) * inv_l, __uint_as_float(r[i + 7]) * inv_l));
                            }
                        }
                        fence_proxy_async_smem();
                        named_bar_sync(2 + x, 128);
                        if (store_leader) {
                            tma_store_3d(&tm_o, sm.o_stage[x], b * 64, wi.head, (int32_t)grow0);
                            bulk_commit_group();
                        }
                    }
                    p.lse[(int64_t)wi.head * p.total_q + grow] = lse;
                }
                store_pending = true;
            } else if (t.partial_slot >= 0) {
                float* dst = p.o_partial + (grow * p.n_heads + wi.head) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    if (n_kv > 0) {
                        tmem_ld_x32(lane_addr + col_o + c * 32, r);
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
                        tmem_ld_x32(lane_addr + col_o + c * 32, r);
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
        if (store_leader) bulk_wait_group<0>();  // the last O stores have left shared memory and landed
    }

teardown:
    // Also reached after an expired wait: bulk stores this thread has committed must have finished
    // reading shared memory before the CTA gives it up (a no-op on the normal path).
    bulk_wait_group<0>();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

template <int D>
cudaError_t launch_t(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                     const CUtensorMap& top, const FwdParams& p, int grid, cudaStream_t stream) {
    constexpr int smem = sizeof(FwdSmem<D>);
    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    constexpr int kMaxDevices = 64;
    static bool configured[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices || !configured[dev]) {
        e = cudaFuncSetAttribute(zl_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < kMaxDevices) configured[dev] = true;
    }
    zl_fwd_kernel<D><<<grid, kFwdThreads, smem, stream>>>(tq, tk, tv, to, top, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd(int head_dim, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                       const CUtensorMap& to, const CUtensorMap& top, const FwdParams& p, int grid,
                       cudaStream_t stream) {
    if (p.n_items == 0) return cudaSuccess;
    return head_dim == 128 ? launch_t<128>(tq, tk, tv, to, top, p, grid, stream)
                           : launch_t<64>(tq, tk, tv, to, top, p, grid, stream);
}

}  // namespace zl
