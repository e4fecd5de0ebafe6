// Backward main kernel, CTA-pair form (sm_100a, head_dim 128).
//
// Same mathematics and the same three-launch structure as zl_bwd.cu (preprocess and dQ conversion
// are shared); this file replaces the main kernel by one that runs on clusters of two CTAs with
// tcgen05.mma.cta_group::2.  A pair owns two neighbouring 128-row key tiles of one kv group and one
// head -- CTA r holds tile r: K_r, V_r in shared memory, dK_r, dV_r in TMEM -- and both CTAs walk
// the same 128-row query tiles in lockstep.  Per query tile the leader CTA issues, for the pair:
//
//   S^T  = K Q^T  - LSE/scale   M = 256 keys, N = 128 queries   A = K_r,   B: 64 query rows from each CTA
//   dP^T = V dO^T - D           M = 256,      N = 128           A = V_r,   B: 64 dO rows from each CTA
//   dV  += P^T dO               M = 256,      N = 128 (d)       A = P^T in TMEM, B: 64 columns of dO from each CTA
//   dK  += dS^T Q               M = 256,      N = 128 (d)       A = dS^T in TMEM, B: 64 columns of Q from each CTA
//   dQ   = dS K                 M = 128 queries (64 per CTA), N = 128 (d), K = 256 keys
//
// Why a pair.  With one CTA per key tile every B operand is read from shared memory once per CTA and
// every (query tile, key tile) adds a 64 KB fp32 dQ tile into the accumulator; that kernel is bound
// by shared-memory bandwidth and by the bulk reduce.  In the pair each CTA supplies half of every B
// operand, dS^T feeds the dK MMA from TMEM, and dQ is summed over the pair's 256 keys inside the tensor
// core: each P/dS thread stores its 64-query row of dS in its own CTA's shared memory -- into the dQ
// operand itself when these are the queries this CTA reduces, else into an outgoing box that one lane
// per warp sends to the partner with a bulk copy -- so a CTA ends up with dS of 64 queries x 256 keys
// and reduces a 32 KB dQ tile: half the reduce bytes, half the staging.
//
// Crossing the pair takes about a thousand cycles, so dQ is kept off the loop-carried chain
// dP^T(i) -> dS(i) -> dK(i) -> dP^T(i+1): its result lands in the upper half of the S^T columns, which
// are free once the P/dS warps have read S^T(i+1), instead of the dP^T columns, and the tensor pipe runs
// dK(i) dP^T(i+1) dQ(i) dV(i+1) S^T(i+2).
//
// Both CTAs run the same roles: warp 0 and warp 2 TMA producers, warp 1 MMA issuer (leader only), warp 3
// second MMA issuer for dQ in the leader and relay in the partner (it tells the leader that the leader's
// dS rows have landed there), warps 4-11 P/dS (one key row per thread), warps 12-15 dQ drain + reduce.  Signals that the leader's
// MMA warp waits for live in the leader's shared memory: the partner's TMA loads count their bytes
// there and the partner's warps arrive there through the cluster address space; MMA completions are
// committed to the barrier at the same offset in both CTAs.
#include <cuda_runtime.h>

#include "zl_device.h"
#include "zl_ptx.cuh"

namespace zl {

using namespace ptx;

namespace {

constexpr uint64_t kWaitLimitNs = 4000000000ull;
constexpr int kPairThreads = 512;
constexpr int D = 128;

struct PairSmem {
    static constexpr int kTileBytes = 128 * D * 2;  // 128 rows x 128 bf16
    static constexpr int kBoxBytes = 128 * 128;     // 128 rows x 64 bf16
    static constexpr int kHalfBoxBytes = 64 * 128;  // 64 rows x 64 bf16
    alignas(1024) uint8_t k[kTileBytes];            // own key tile, d 0-63 | d 64-127: A of S^T (K-major)
    alignas(1024) uint8_t v[kTileBytes];            // own value tile: A of dP^T
    alignas(1024) uint8_t kx[2][kBoxBytes];         // keys of tile 0 | tile 1 of the pair, this CTA's half of d: B of dQ
    alignas(1024) uint8_t q_r[2][kHalfBoxBytes];    // this CTA's 64 query rows, d 0-63 | d 64-127: B of S^T
    alignas(1024) uint8_t q_c[kBoxBytes];           // all 128 query rows, this CTA's half of d: B of dK
    alignas(1024) uint8_t do_r[2][kHalfBoxBytes];   // B of dP^T
    alignas(1024) uint8_t do_c[kBoxBytes];          // B of dV
    alignas(1024) uint8_t ds[2][kBoxBytes];         // dS, keys of tile 0 | tile 1 x this CTA's 64 queries: A of dQ
    alignas(1024) uint8_t ds_out[4][4096];          // per warp of the other warpgroup: dS rows on their way to the partner
    alignas(1024) uint8_t dq_stage[4][2048];        // per dQ warp: 32 rows x 16 fp32 columns on their way to the reduce
    alignas(1024) uint8_t aug_s[2048];              // [pieces of -LSE/scale of this CTA's 64 queries | zeros]
    alignas(1024) uint8_t aug_d[2048];              // [pieces of -D | zeros]
    alignas(1024) uint8_t ones[2][2048];            // [ones in elements 0..2][zeros]
    // K, V and the K columns for dQ are filled and released separately: K is free after the item's last S^T, V after
    // its last dP^T, the K columns after its last dQ, and the next item's tiles are loaded as soon as each one is
    alignas(8) uint64_t k_full, k_empty, v_full, v_empty, kx_full, kx_empty;
    uint64_t qr_full, qr_empty, qc_full, qc_empty;
    uint64_t dor_full, dor_empty, doc_full, doc_empty;  // dO rows + D pieces (B of dP^T) and dO columns (B of dV) have different lifetimes
    uint64_t s_full, dp_full, p_full, dst_full, ds_full, ds_free, dq_full, acc_full;
    uint64_t dq_empty[2];  // dQ tile g drained from TMEM: barrier g & 1 (two waiters, one of which may be two tiles behind)
    uint64_t s_read;      // every P/dS warp of both CTAs has read its S^T columns
    uint64_t sp_read[4];  // per lane quarter: warpgroup 0 has read its S^T columns
    uint64_t dp_read[4];  // per lane quarter: warpgroup 0 has read its dP^T columns
    uint64_t ds_land;     // partner CTA only: the leader's dS rows have landed in this CTA
    uint32_t tmem_base;
    volatile int32_t abort_flag;
};

static_assert(sizeof(PairSmem) <= 227 * 1024, "shared memory of the pair kernel");

// Out of line, like the slow halves of the waits: the kernel has some sixty wait sites and its loops should stay in
// the instruction cache.
__device__ __noinline__ void report(int32_t* status, volatile int32_t* abort_flag, int where) {
    *abort_flag = 1;
    if (atomicCAS(status, 0, (int)ZL_ERR_TIMEOUT) == 0) status[1] = where;
}

// Bounded waits: the first try is inline, the timed loop out of line -- the kernel has some sixty wait sites and its
// loops should stay in the instruction cache.  The loop gives up when the limit has passed or another role of the CTA
// has given up; the acquire has cluster scope, which barriers the partner CTA arrives on need.
__device__ __noinline__ bool pair_wait_slow(uint64_t* bar, uint32_t parity, const volatile int32_t* abort_flag) {
    const uint64_t t0 = globaltimer();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((++spins & 0xFF) == 0) {
            if (*abort_flag) return false;
            if (globaltimer() - t0 > kWaitLimitNs) return false;
        }
    }
}
__device__ __forceinline__ bool pair_wait(uint64_t* bar, uint32_t parity, const volatile int32_t* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return pair_wait_slow(bar, parity, abort_flag);
}
__device__ __forceinline__ bool pair_wait_cluster(uint64_t* bar, uint32_t parity, const volatile int32_t* abort_flag) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    return pair_wait_slow(bar, parity, abort_flag);
}

#define ZL_WAIT(bar, parity, site)                                        \
    do {                                                                  \
        if (!pair_wait((bar), (parity), &sm.abort_flag)) {               \
            report(p.status, &sm.abort_flag, 3000 + (site));              \
            goto teardown;                                                \
        }                                                                 \
    } while (0)
#define ZL_WAIT_WARP(bar, parity, site)                                              \
    do {                                                                             \
        const bool ok_ = pair_wait((bar), (parity), &sm.abort_flag);                 \
        if (!__all_sync(0xffffffffu, ok_)) {                                         \
            report(p.status, &sm.abort_flag, 3000 + (site));                         \
            goto teardown;                                                           \
        }                                                                            \
    } while (0)
// the same for barriers the partner CTA arrives on
#define ZL_WAIT_WARP_CL(bar, parity, site)                                                    \
    do {                                                                                      \
        const bool ok_ = pair_wait_cluster((bar), (parity), &sm.abort_flag);                  \
        if (!__all_sync(0xffffffffu, ok_)) {                                                  \
            report(p.status, &sm.abort_flag, 3000 + (site));                                  \
            goto teardown;                                                                    \
        }                                                                                     \
    } while (0)

__device__ __forceinline__ int count_q_tiles(const BwdParams&, const KvGroup& g) { return g.n_q_tiles; }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
zl_bwd_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_q64,
                   const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_do, const __grid_constant__ CUtensorMap tm_do64,
                   const __grid_constant__ CUtensorMap tm_dq, const __grid_constant__ CUtensorMap tm_aug,
                   const __grid_constant__ CUtensorMap tm_dk32, const __grid_constant__ CUtensorMap tm_dv32,
                   const BwdParams p) {
    using Smem = PairSmem;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();   // 0: leader, holds key tile 0 of every item; 1: key tile 1
    const int n_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;

    // TMEM columns (per CTA): S^T [0,128), then P^T as bf16 pairs [0,64) and the CTA's 64 x 128 dQ tile as
    // 128 lanes x 64 columns [64,128); dP^T [128,256), then dS^T as bf16 pairs [128,192); dV [256,384); dK [384,512)
    constexpr uint32_t kColS = 0, kColDQ = 64, kColDP = 128, kColDS = 128, kColDV = 256, kColDK = 384, kTmemCols = 512;

    const bool misaligned = (smem_u32(smem_raw) & 1023u) != 0;  // identical in both CTAs: same kernel, same offsets
    if (misaligned) {
        if (threadIdx.x == 0 && atomicCAS(p.status, 0, (int)ZL_ERR_CUDA) == 0) p.status[1] = 3999;
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(&sm.k_full, 1);
        mbar_init(&sm.k_empty, 1);
        mbar_init(&sm.v_full, 1);
        mbar_init(&sm.v_empty, 1);
        mbar_init(&sm.kx_full, 1);
        mbar_init(&sm.kx_empty, 1);
        mbar_init(&sm.qr_full, 1);
        mbar_init(&sm.qr_empty, 1);
        mbar_init(&sm.qc_full, 1);
        mbar_init(&sm.qc_empty, 1);
        mbar_init(&sm.dor_full, 1);
        mbar_init(&sm.dor_empty, 1);
        mbar_init(&sm.doc_full, 1);
        mbar_init(&sm.doc_empty, 1);
        mbar_init(&sm.s_full, 1);
        mbar_init(&sm.dp_full, 1);
        mbar_init(&sm.p_full, 16);    // one arrival per P/dS warp of both CTAs
        mbar_init(&sm.dst_full, 16);  // dS^T in TMEM (A of dK)
        mbar_init(&sm.ds_full, 9);    // dS in shared memory (A of dQ): the eight warps that store in place and the
                                      // relay arrive; the rows the partner sends to the leader are counted in bytes
        mbar_init(&sm.ds_land, 1);
        mbar_init(&sm.ds_free, 1);
        mbar_init(&sm.dq_full, 1);
        mbar_init(&sm.dq_empty[0], 8);   // one arrival per dQ warp of both CTAs
        mbar_init(&sm.dq_empty[1], 8);
        mbar_init(&sm.acc_full, 1);
        mbar_init(&sm.s_read, 16);
        for (int i = 0; i < 4; ++i) { mbar_init(&sm.dp_read[i], 1); mbar_init(&sm.sp_read[i], 1); }
        sm.abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_q64);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_do);
        prefetch_tmap(&tm_do64);
        prefetch_tmap(&tm_dq);
        prefetch_tmap(&tm_aug);
    }
    // constant operands: the ones blocks of the augmentation steps and the zero halves of the augmentation tiles
    for (int i = threadIdx.x; i < 2 * 2048 / 4; i += kPairThreads) {
        const int blk = i / 512, w = i % 4;
        uint32_t val = 0;
        if (blk == 0) val = (w == 0) ? 0x3F803F80u : (w == 1 ? 0x00003F80u : 0u);
        reinterpret_cast<uint32_t*>(&sm.ones[0][0])[i] = val;
    }
    for (int i = threadIdx.x; i < 1024 / 4; i += kPairThreads) {
        reinterpret_cast<uint32_t*>(sm.aug_s + 1024)[i] = 0u;
        reinterpret_cast<uint32_t*>(sm.aug_d + 1024)[i] = 0u;
    }
    fence_proxy_async_smem();
    if (warp == 1) {
        tmem_alloc_pair(&sm.tmem_base, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive();   // the partner's barriers are initialised before anything is sent to them
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp < 4) {
        // (no register reallocation: every role fits the 128 registers the launch bounds give)
        if (warp == 0 && lane == 0) {
            // -------------------------------------------------------------- TMA producer: K, V, Q rows, dO
            // Transaction bytes of both CTAs are counted on the leader's barrier, which the leader's
            // producer arms for the pair.
            const uint32_t k_full_l = map_to_cta(smem_u32(&sm.k_full), 0);
            const uint32_t v_full_l = map_to_cta(smem_u32(&sm.v_full), 0);
            const uint32_t qr_full_l = map_to_cta(smem_u32(&sm.qr_full), 0);
            const uint32_t dor_full_l = map_to_cta(smem_u32(&sm.dor_full), 0);
            const uint32_t doc_full_l = map_to_cta(smem_u32(&sm.doc_full), 0);
            uint32_t item_cnt = 0, it_cnt = 0;
            #pragma unroll 1
            for (int it = cluster_id; it < p.n_items; it += n_clusters, ++item_cnt) {
                const WorkItem wi = p.items[it];
                const KvGroup g = p.kv_groups[wi.unit];
                const int key0 = g.kv_off + wi.row0;   // first key row of the pair
                ZL_WAIT(&sm.k_empty, (item_cnt & 1) ^ 1, 1);
                if (rank == 0) mbar_arrive_expect_tx(&sm.k_full, 2 * Smem::kTileBytes);
                for (int b = 0; b < 2; ++b)
                    tma_load_3d_pair(sm.k + b * Smem::kBoxBytes, &tm_k, k_full_l, b * 64, wi.head, key0 + 128 * (int)rank);
                ZL_WAIT(&sm.v_empty, (item_cnt & 1) ^ 1, 6);
                if (rank == 0) mbar_arrive_expect_tx(&sm.v_full, 2 * Smem::kTileBytes);
                for (int b = 0; b < 2; ++b)
                    tma_load_3d_pair(sm.v + b * Smem::kBoxBytes, &tm_v, v_full_l, b * 64, wi.head, key0 + 128 * (int)rank);
                #pragma unroll 1
                for (int ti = 0; ti < g.n_tasks; ++ti) {
                    const Task t = p.tasks[p.kv_group_tasks[g.task_begin + ti]];
                    const int n_q = (t.q_len + kTileQ - 1) / kTileQ;
                    #pragma unroll 1
                    for (int qt = 0; qt < n_q; ++qt, ++it_cnt) {
                        const int q0 = t.q_off + qt * kTileQ;
                        const int aug_row = (wi.head * (p.q_pad_total / kTileQ) + t.q_slot / kTileQ + qt) * 4 + (int)rank;
                        ZL_WAIT(&sm.qr_empty, (it_cnt & 1) ^ 1, 2);
                        if (rank == 0) mbar_arrive_expect_tx(&sm.qr_full, 2 * (2 * Smem::kHalfBoxBytes + 1024));
                        for (int b = 0; b < 2; ++b)
                            tma_load_3d_pair(sm.q_r[b], &tm_q64, qr_full_l, b * 64, wi.head, q0 + 64 * (int)rank);
                        tma_load_2d_pair(sm.aug_s, &tm_aug, qr_full_l, 0, aug_row);
                        ZL_WAIT(&sm.dor_empty, (it_cnt & 1) ^ 1, 3);
                        if (rank == 0) mbar_arrive_expect_tx(&sm.dor_full, 2 * (2 * Smem::kHalfBoxBytes + 1024));
                        for (int b = 0; b < 2; ++b)
                            tma_load_3d_pair(sm.do_r[b], &tm_do64, dor_full_l, b * 64, wi.head, q0 + 64 * (int)rank);
                        tma_load_2d_pair(sm.aug_d, &tm_aug, dor_full_l, 0, aug_row + 2);
                        ZL_WAIT(&sm.doc_empty, (it_cnt & 1) ^ 1, 7);
                        if (rank == 0) mbar_arrive_expect_tx(&sm.doc_full, 2 * Smem::kBoxBytes);
                        tma_load_3d_pair(sm.do_c, &tm_do, doc_full_l, 64 * (int)rank, wi.head, q0);
                    }
                }
            }
        } else if (warp == 2 && lane == 0) {
            // -------------------------------------------------------------- TMA producer: Q columns (B of dK)
            // Its buffer is released two MMAs later than the Q rows; a producer of its own keeps that wait
            // from delaying the other loads.
            const uint32_t qc_full_l = map_to_cta(smem_u32(&sm.qc_full), 0);
            const uint32_t kx_full_l = map_to_cta(smem_u32(&sm.kx_full), 0);
            uint32_t item_cnt = 0, it_cnt = 0;
            #pragma unroll 1
            for (int it = cluster_id; it < p.n_items; it += n_clusters, ++item_cnt) {
                const WorkItem wi = p.items[it];
                const KvGroup g = p.kv_groups[wi.unit];
                // the K columns for dQ are the last buffer of the previous item to come free (after its last dQ), and
                // dQ is the last MMA group of a tile to need its operand: loaded here, off the other producer's path
                ZL_WAIT(&sm.kx_empty, (item_cnt & 1) ^ 1, 8);
                if (rank == 0) mbar_arrive_expect_tx(&sm.kx_full, 2 * 2 * Smem::kBoxBytes);
                for (int b = 0; b < 2; ++b)
                    tma_load_3d_pair(sm.kx[b], &tm_k, kx_full_l, 64 * (int)rank, wi.head, g.kv_off + wi.row0 + 128 * b);
                #pragma unroll 1
                for (int ti = 0; ti < g.n_tasks; ++ti) {
                    const Task t = p.tasks[p.kv_group_tasks[g.task_begin + ti]];
                    const int n_q = (t.q_len + kTileQ - 1) / kTileQ;
                    #pragma unroll 1
                    for (int qt = 0; qt < n_q; ++qt, ++it_cnt) {
                        ZL_WAIT(&sm.qc_empty, (it_cnt & 1) ^ 1, 4);
                        if (rank == 0) mbar_arrive_expect_tx(&sm.qc_full, 2 * Smem::kBoxBytes);
                        tma_load_3d_pair(sm.q_c, &tm_q, qc_full_l, 64 * (int)rank, wi.head, t.q_off + qt * kTileQ);
                    }
                }
            }
        } else if (warp == 3 && lane == 0 && rank == 1) {
            // -------------------------------------------------------------- relay (partner CTA)
            // The leader's MMA warp cannot wait on a barrier of this CTA: when the dS rows the leader sent
            // have landed here, tell the leader.
            const uint32_t ds_full_l = map_to_cta(smem_u32(&sm.ds_full), 0);
            uint32_t it_cnt = 0;
            #pragma unroll 1
            for (int it = cluster_id; it < p.n_items; it += n_clusters) {
                const KvGroup g = p.kv_groups[p.items[it].unit];
                const int n_it = count_q_tiles(p, g);
                #pragma unroll 1
                for (int i = 0; i < n_it; ++i, ++it_cnt) {
                    mbar_arrive_expect_tx(&sm.ds_land, Smem::kBoxBytes);
                    ZL_WAIT(&sm.ds_land, it_cnt & 1, 5);
                    mbar_arrive_cluster(ds_full_l);
                }
            }
        } else if (warp == 1 && rank == 0) {
            // -------------------------------------------------------------- MMA issuer (leader CTA)
            const bool mma_lane = elect_one();
            constexpr uint32_t idesc_s = make_idesc_bf16(256, 128, 0, 0);    // S^T, dP^T: K-major x K-major
            constexpr uint32_t idesc_kv = make_idesc_bf16(256, 128, 0, 1);   // dV, dK: A in TMEM, B MN-major
            const uint64_t dk_k = make_desc_sw128(smem_u32(sm.k), 16, 1024);
            const uint64_t dv_k = make_desc_sw128(smem_u32(sm.v), 16, 1024);
            const uint64_t dqr_k = make_desc_sw128(smem_u32(sm.q_r[0]), 16, 1024);
            const uint64_t ddor_k = make_desc_sw128(smem_u32(sm.do_r[0]), 16, 1024);
            const uint64_t dqc_mn = make_desc_sw128(smem_u32(sm.q_c), Smem::kBoxBytes, 1024);
            const uint64_t ddoc_mn = make_desc_sw128(smem_u32(sm.do_c), Smem::kBoxBytes, 1024);
            const uint64_t daug_s = make_desc_noswizzle(smem_u32(sm.aug_s), 1024, 128);
            const uint64_t daug_d = make_desc_noswizzle(smem_u32(sm.aug_d), 1024, 128);
            const uint64_t dones = make_desc_noswizzle(smem_u32(&sm.ones[0][0]), 2048, 128);  // ones, then zeros
            // S^T = K Q^T - LSE/scale (last step: ones block x LSE pieces)
            auto issue_s = [&]() {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t offa = ((ks / 4) * Smem::kBoxBytes + (ks % 4) * 32) >> 4;
                    const uint32_t offb = ((ks / 4) * Smem::kHalfBoxBytes + (ks % 4) * 32) >> 4;
                    if (mma_lane) mma_ss_pair(tmem + kColS, dk_k + offa, dqr_k + offb, idesc_s, ks > 0);
                }
                if (mma_lane) mma_ss_pair(tmem + kColS, dones, daug_s, idesc_s, true);
                if (mma_lane) mma_commit_pair(&sm.s_full);
                if (mma_lane) mma_commit_pair(&sm.qr_empty);
            };
            auto issue_dp = [&]() {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t offa = ((ks / 4) * Smem::kBoxBytes + (ks % 4) * 32) >> 4;
                    const uint32_t offb = ((ks / 4) * Smem::kHalfBoxBytes + (ks % 4) * 32) >> 4;
                    if (mma_lane) mma_ss_pair(tmem + kColDP, dv_k + offa, ddor_k + offb, idesc_s, ks > 0);
                }
                if (mma_lane) mma_ss_pair(tmem + kColDP, dones, daug_d, idesc_s, true);
                if (mma_lane) mma_commit_pair(&sm.dp_full);
                if (mma_lane) mma_commit_pair(&sm.dor_empty);
            };
            auto issue_dv = [&](bool acc) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // dV += P^T dO, K = 128 query rows
                    if (mma_lane) mma_ts_pair(tmem + kColDV, tmem + kColS + ks * 8, ddoc_mn + ks * (2048 >> 4), idesc_kv,
                                              acc || ks > 0);
                if (mma_lane) mma_commit_pair(&sm.doc_empty);
            };
            uint32_t item_cnt = 0, it_base = 0;  // it_base: query tiles of earlier items
            uint32_t dq_waited = 0;  // dQ tiles known to be drained from TMEM in both CTAs
            #pragma unroll 1
            for (int it = cluster_id; it < p.n_items; it += n_clusters, ++item_cnt) {
                const WorkItem wi = p.items[it];
                const KvGroup g = p.kv_groups[wi.unit];
                const int n_it = count_q_tiles(p, g);
                // Order of this warp's MMAs: dK(i) dP(i+1) dV(i+1) S(i+2); dQ(i) comes from the second issuer.  The
                // two steps before the item's first tile (i = -2, -1) are the prologue: S(0), then dP(0) dV(0) S(1).
                // S^T(x) overwrites the columns of dQ(x-2) (dQ(x-1) is only issued once S^T(x) has been read); the
                // first S^T of an item follows the previous item's last dQ, which cannot wait for it: the P/dS warps
                // read that S^T only after their epilogue, and the epilogue stages in the boxes the last dQ reads.
                #pragma unroll 1
                for (int i = -2; i < n_it; ++i) {
                    if (i >= 0) {
                        // dK needs dS^T in TMEM only
                        const uint32_t c = it_base + i;
                        ZL_WAIT_WARP_CL(&sm.dst_full, c & 1, 17);
                        ZL_WAIT_WARP_CL(&sm.qc_full, c & 1, 18);
                        tc_fence_after();
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)  // dK += dS^T Q, K = 128 query rows, dS^T from TMEM
                            if (mma_lane) mma_ts_pair(tmem + kColDK, tmem + kColDS + ks * 8, dqc_mn + ks * (2048 >> 4), idesc_kv,
                                                      i > 0 || ks > 0);
                        if (mma_lane) mma_commit_pair(&sm.qc_empty);
                    }
                    if (i + 1 >= 0 && i + 1 < n_it) {
                        // dP^T of the next tile right behind it (it overwrites dS^T: ordered after dK on the tensor pipe)
                        const uint32_t c = it_base + i + 1;
                        ZL_WAIT_WARP_CL(&sm.dor_full, c & 1, 19);
                        if (i + 1 == 0) ZL_WAIT_WARP_CL(&sm.v_full, item_cnt & 1, 12);
                        tc_fence_after();
                        issue_dp();
                        if (i + 1 == n_it - 1 && mma_lane) mma_commit_pair(&sm.v_empty);  // the item's last dP^T: V may go
                        ZL_WAIT_WARP_CL(&sm.p_full, c & 1, 21);
                        ZL_WAIT_WARP_CL(&sm.doc_full, c & 1, 29);
                        tc_fence_after();
                        issue_dv(i + 1 > 0);
                    }
                    if (i + 2 < n_it) {
                        const uint32_t c = it_base + i + 2;
                        const uint32_t drained = it_base + (i + 1 > 0 ? i + 1 : 0);  // dQ tiles that must have left TMEM
                        ZL_WAIT_WARP_CL(&sm.qr_full, c & 1, 22);
                        if (i + 2 == 0) ZL_WAIT_WARP_CL(&sm.k_full, item_cnt & 1, 11);
                        while (dq_waited < drained) { ZL_WAIT_WARP_CL(&sm.dq_empty[dq_waited & 1], (dq_waited >> 1) & 1, 25); ++dq_waited; }
                        tc_fence_after();
                        issue_s();  // overwrites P^T: ordered after dV on the tensor pipe
                        if (i + 2 == n_it - 1 && mma_lane) mma_commit_pair(&sm.k_empty);  // the item's last S^T: K may go
                    }
                }
                it_base += n_it;
                if (mma_lane) mma_commit_pair(&sm.acc_full);
            }
        } else if (warp == 3 && rank == 0) {
            // -------------------------------------------------------------- second MMA issuer (leader CTA): dQ
            // dQ(i) depends on nothing the other MMAs produce in TMEM and nothing depends on it but the drain, so
            // it has a queue of its own: it goes out when the dS rows that cross the pair have landed and S^T(i+1)
            // has been read in both CTAs (its result takes the upper half of those columns), behind dQ(i-1)'s drain.
            const bool mma_lane = elect_one();
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, 128, 1, 1);   // A MN-major, B MN-major
            const uint64_t dds_mn = make_desc_sw128(smem_u32(sm.ds[0]), Smem::kBoxBytes, 1024);
            const uint64_t dkx_mn = make_desc_sw128(smem_u32(sm.kx[0]), Smem::kBoxBytes, 1024);
            uint32_t item_cnt = 0, it_cnt = 0;
            #pragma unroll 1
            for (int it = cluster_id; it < p.n_items; it += n_clusters, ++item_cnt) {
                const KvGroup g = p.kv_groups[p.items[it].unit];
                const int n_it = count_q_tiles(p, g);
                ZL_WAIT_WARP_CL(&sm.kx_full, item_cnt & 1, 51);  // the K columns of this item are in place
                #pragma unroll 1
                for (int i = 0; i < n_it; ++i, ++it_cnt) {
                    ZL_WAIT_WARP_CL(&sm.ds_full, it_cnt & 1, 52);
                    if (i + 1 < n_it) ZL_WAIT_WARP_CL(&sm.s_read, (it_cnt + 1) & 1, 53);
                    if (it_cnt > 0) ZL_WAIT_WARP_CL(&sm.dq_empty[(it_cnt - 1) & 1], ((it_cnt - 1) >> 1) & 1, 54);
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 16; ++ks)  // dQ = dS K over the pair's 256 keys; 64 query rows per CTA
                        if (mma_lane) mma_ss_pair(tmem + kColDQ, dds_mn + ks * (2048 >> 4), dkx_mn + ks * (2048 >> 4),
                                                  idesc_dq, ks > 0);
                    if (mma_lane) mma_commit_pair(&sm.dq_full);
                    if (mma_lane) mma_commit_pair(&sm.ds_free);
                }
                // the K columns may be replaced when this item's last dQ has run
                if (mma_lane) mma_commit_pair(&sm.kx_empty);
            }
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------------ P / dS warpgroups

        const int wg = (warp - 4) >> 2;            // 0: query columns 0-63, 1: columns 64-127
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;       // key row within this CTA's tile
        const int col0 = wg * 64;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        // this thread's 64 values of dS belong to the dQ rows that CTA `wg` reduces: they go to that CTA's
        // slot for the keys of this CTA's tile -- directly when that is this CTA, else through the outgoing box
        const bool ds_local = (uint32_t)wg == rank;   // warp-uniform
        const uint32_t ds_row_dst = ds_local ? smem_u32(sm.ds[rank]) + row * 128 : smem_u32(sm.ds_out[quarter]) + lane * 128;
        const uint32_t ds_remote_dst = map_to_cta(smem_u32(sm.ds[rank]) + quarter * 4096, (uint32_t)wg);
        const uint32_t s_read_l = map_to_cta(smem_u32(&sm.s_read), 0);
        const uint32_t ds_remote_bar = map_to_cta(smem_u32(wg == 0 ? &sm.ds_full : &sm.ds_land), (uint32_t)wg);
        const uint32_t p_full_l = map_to_cta(smem_u32(&sm.p_full), 0);
        const uint32_t ds_full_l = map_to_cta(smem_u32(&sm.ds_full), 0);
        const uint32_t dst_full_l = map_to_cta(smem_u32(&sm.dst_full), 0);
        const float sl2 = p.scale_log2;
        uint32_t item_cnt = 0, it_cnt = 0;
        bool store_pending = false;  // warp-uniform
        // The item after this one is fetched while this one runs: at an item boundary these warps are on the critical
        // path (epilogue, then the next item's first P), and two dependent loads from global memory are ~1,200 cycles.
        WorkItem wi_cur = p.items[min(cluster_id, p.n_items - 1)];
        KvGroup g_cur = p.kv_groups[wi_cur.unit];
        #pragma unroll 1
        for (int it = cluster_id; it < p.n_items; it += n_clusters, ++item_cnt) {
            const WorkItem wi = wi_cur;
            const KvGroup g = g_cur;
            const bool has_next = it + n_clusters < p.n_items;
            if (has_next) wi_cur = p.items[it + n_clusters];
            const int rows_here = min(kTileKV, wi.rows - kTileKV * (int)rank);  // key rows of this CTA's tile (may be <= 0)
            const bool row_ok = row < rows_here;
            const float row_bias = row_ok ? 0.f : -INFINITY;
            const int n_it = count_q_tiles(p, g);
            {
                #pragma unroll 1
                for (int i = 0; i < n_it; ++i, ++it_cnt) {
                    ZL_WAIT_WARP(&sm.s_full, it_cnt & 1, 31);
                    tc_fence_after();
                    uint32_t pk[32];  // P^T of this thread's row, bf16 pairs
                    {
                        uint32_t sr[2][32];
                        tmem_ld_x32(lane_addr + kColS + col0, sr[0]);
                        tmem_ld_x32(lane_addr + kColS + col0 + 32, sr[1]);
                        tmem_wait_ld();
                        // S^T has been read: the upper half of its columns may take a dQ tile, and warpgroup 1 may
                        // put its P^T into the columns [32,64) that warpgroup 0 has just read
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive_cluster(s_read_l);
                            if (wg == 0) mbar_arrive(&sm.sp_read[quarter]);
                        }
                        // S^T already has -LSE/scale folded in; query columns past the end of the task carry -1e30
                        // there (preprocess kernel) and key rows past the end of the item get -inf here, so their
                        // P is exactly zero without a second code path
#pragma unroll
                        for (int c = 0; c < 2; ++c)
#pragma unroll
                            for (int i = 0; i < 32; i += 2)
                                pk[c * 16 + i / 2] = pack_bf16(ex2(fmaf(__uint_as_float(sr[c][i]), sl2, row_bias)),
                                                               ex2(fmaf(__uint_as_float(sr[c][i + 1]), sl2, row_bias)));
                        if (wg == 1) {
                            ZL_WAIT_WARP(&sm.sp_read[quarter], it_cnt & 1, 36);
                            tc_fence_after();
                        }
                        tmem_st_x32(lane_addr + kColS + wg * 32, pk);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(p_full_l);

                    ZL_WAIT_WARP(&sm.dp_full, it_cnt & 1, 32);
                    tc_fence_after();
                    {
                        uint32_t dr[2][32];
                        tmem_ld_x32(lane_addr + kColDP + col0, dr[0]);
                        tmem_ld_x32(lane_addr + kColDP + col0 + 32, dr[1]);
                        tmem_wait_ld();
                        // dS^T goes back into the dP^T columns [128,192): warpgroup 1 writes columns that
                        // warpgroup 0 reads, so it waits for the warp of warpgroup 0 that shares its lanes
                        if (wg == 0) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&sm.dp_read[quarter]);
                        }
                        uint32_t dd[32];
                        // dS^T = P^T o (dP^T - D) in packed bf16 arithmetic; where P is zero by masking, dP^T - D is
                        // finite (rows of other sequences or the zero fill of the loads), so the product is zero
#pragma unroll
                        for (int c = 0; c < 2; ++c)
#pragma unroll
                            for (int i = 0; i < 32; i += 2)
                                dd[c * 16 + i / 2] = mul_bf16x2(pk[c * 16 + i / 2],
                                                                pack_bf16(__uint_as_float(dr[c][i]), __uint_as_float(dr[c][i + 1])));
                        // A operand of dK first (dS^T as bf16 pairs in TMEM): the dK MMAs start while the rows for
                        // the dQ operand are still being stored and sent
                        if (wg == 1) {
                            ZL_WAIT_WARP(&sm.dp_read[quarter], it_cnt & 1, 35);
                            tc_fence_after();
                        }
                        tmem_st_x32(lane_addr + kColDS + wg * 32, dd);
                        tmem_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(dst_full_l);
                        // A operand of dQ: one 128-byte row (this key, 64 queries), in place or in the outgoing box
                        // (same swizzle: the box is copied to the same offset modulo 1024 in the partner), once the
                        // dQ MMAs of the previous tile have consumed the boxes in both CTAs
                        if (it_cnt > 0) ZL_WAIT_WARP(&sm.ds_free, (it_cnt - 1) & 1, 33);
                        if (store_pending) {  // the previous item's last gradient store still reads this warp's box
                            if (lane == 0) bulk_wait_group_read<0>();
                            __syncwarp();
                            store_pending = false;
                        }
#pragma unroll
                        for (int c16 = 0; c16 < 8; ++c16)
                            st_shared_v4(ds_row_dst + ((c16 ^ (row & 7)) << 4), dd[c16 * 4], dd[c16 * 4 + 1], dd[c16 * 4 + 2],
                                         dd[c16 * 4 + 3]);
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            if (!ds_local) bulk_copy_to_cta(ds_remote_dst, sm.ds_out[quarter], 4096, ds_remote_bar);
                            // the leader's first warp also announces the bytes the partner sends to the leader
                            else if (rank == 0 && warp == 4) mbar_arrive_expect_tx(&sm.ds_full, Smem::kBoxBytes);
                            else mbar_arrive_cluster(ds_full_l);
                        }
                    }
                }
            }
            // ---- epilogue: warpgroup 0 stores dV, warpgroup 1 stores dK (scaled), one key row per thread
            if (has_next) g_cur = p.kv_groups[wi_cur.unit];  // arrives under the epilogue
            ZL_WAIT_WARP(&sm.acc_full, item_cnt & 1, 34);
            tc_fence_after();
            const float sc = (wg == 0) ? 1.f : p.scale;
            const uint32_t col_acc = (wg == 0) ? kColDV : kColDK;
            const int64_t grow = (int64_t)g.kv_off + wi.row0 + kTileKV * (int)rank + row;
            if (quarter * 32 + 32 <= rows_here) {
                // all 32 rows of this warp are inside the item: stage 64 columns at a time in the 4 KB of the dS
                // operand that only this warp writes (its rows of the in-place box, or its outgoing box) and
                // write each with one TMA store -- coalesced, and the warp moves on while the copy engine drains
                // the box.  The last dQ MMAs read that box and are not covered by acc_full (another thread
                // issued them): wait for them here, as the next hand-over would.
                ZL_WAIT_WARP(&sm.ds_free, (it_cnt - 1) & 1, 42);
                const uint32_t box = ds_local ? smem_u32(sm.ds[rank]) + quarter * 4096 : smem_u32(sm.ds_out[quarter]);
                const uint32_t box_row = box + lane * 128;
#pragma unroll 1
                for (int b = 0; b < 2; ++b) {
                    if (b > 0) {
                        if (lane == 0) bulk_wait_group_read<0>();
                        __syncwarp();
                    }
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(lane_addr + col_acc + b * 64 + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            const int i = k4 * 8;
                            st_shared_v4(box_row + (((c * 4 + k4) ^ (lane & 7)) << 4),
                                         pack_bf16(__uint_as_float(r[i]) * sc, __uint_as_float(r[i + 1]) * sc),
                                         pack_bf16(__uint_as_float(r[i + 2]) * sc, __uint_as_float(r[i + 3]) * sc),
                                         pack_bf16(__uint_as_float(r[i + 4]) * sc, __uint_as_float(r[i + 5]) * sc),
                                         pack_bf16(__uint_as_float(r[i + 6]) * sc, __uint_as_float(r[i + 7]) * sc));
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                                     ::"l"(reinterpret_cast<uint64_t>(wg == 0 ? &tm_dv32 : &tm_dk32)), "r"(box), "r"(b * 64),
                                       "r"(wi.head), "r"((int)(grow - lane)) : "memory");
                        bulk_commit_group();
                    }
                }
                store_pending = true;
            } else {
                __nv_bfloat16* dst = (wg == 0 ? p.dv : p.dk) + grow * p.grad_row_stride + wi.head * D;
#pragma unroll 1
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
    } else {
        // ------------------------------------------------------------------ dQ warpgroup
        // The CTA's dQ tile (its 64 query rows x 128 columns) sits in TMEM as 128 lanes x 64 columns: lanes
        // 0-63 hold columns 0-63 of rows 0-63, lanes 64-127 columns 64-127.  Warp w drains lanes 32w..32w+31.

        const int quarter = warp & 3;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        const bool leader = (lane == 0);
        const uint32_t dq_empty_l[2] = {map_to_cta(smem_u32(&sm.dq_empty[0]), 0), map_to_cta(smem_u32(&sm.dq_empty[1]), 0)};
        const int row_in_tile = 64 * (int)rank + 32 * (quarter & 1);  // first query row of this warp's 32 rows
        const int col_base = 64 * (quarter >> 1);
        uint8_t* buf = sm.dq_stage[quarter];
        const uint32_t row_addr = smem_u32(buf) + lane * 64;  // 64-byte rows, 64-byte swizzle
        uint32_t it_cnt = 0, chunk_cnt = 0;
        #pragma unroll 1
        for (int it = cluster_id; it < p.n_items; it += n_clusters) {
            const WorkItem wi = p.items[it];
            const KvGroup g = p.kv_groups[wi.unit];
            #pragma unroll 1
            for (int ti = 0; ti < g.n_tasks; ++ti) {
                const Task t = p.tasks[p.kv_group_tasks[g.task_begin + ti]];
                const int n_q = (t.q_len + kTileQ - 1) / kTileQ;
                #pragma unroll 1
                for (int qt = 0; qt < n_q; ++qt, ++it_cnt) {
                    ZL_WAIT_WARP(&sm.dq_full, it_cnt & 1, 41);
                    tc_fence_after();
                    uint32_t r[64];
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t tmp[32];
                        tmem_ld_x32(lane_addr + kColDQ + c * 32, tmp);
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[c * 32 + i] = tmp[i];
                    }
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (leader) mbar_arrive_cluster(dq_empty_l[it_cnt & 1]);  // the columns may take the next S^T or dQ tile
#pragma unroll
                    for (int c = 0; c < 4; ++c, ++chunk_cnt) {
                        if (chunk_cnt >= 1) {
                            if (leader) bulk_wait_group_read<0>();  // the previous reduce has read the buffer
                            __syncwarp();
                        }
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4)
                            st_shared_v4(row_addr + ((k4 ^ ((lane >> 1) & 3)) << 4), r[c * 16 + k4 * 4], r[c * 16 + k4 * 4 + 1],
                                         r[c * 16 + k4 * 4 + 2], r[c * 16 + k4 * 4 + 3]);
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (leader) {
                            tma_reduce_add_3d(&tm_dq, buf, col_base + c * 16, wi.head, t.q_slot + qt * kTileQ + row_in_tile);
                            bulk_commit_group();
                        }
                    }
                }
            }
        }
        if (leader) bulk_wait_group<0>();
    }

teardown:
    // Also reached after an expired wait.  Bulk reduces this thread has committed must have finished reading
    // shared memory, and neither CTA may leave while the partner can still address its shared memory or TMEM.
    bulk_wait_group<0>();
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_pair(tmem, kTmemCols);
    }
}

}  // namespace

cudaError_t launch_bwd_pair(const CUtensorMap& tq, const CUtensorMap& tq64, const CUtensorMap& tk, const CUtensorMap& tv,
                            const CUtensorMap& tdo, const CUtensorMap& tdo64, const CUtensorMap& tdq,
                            const CUtensorMap& taug, const CUtensorMap& tdk32, const CUtensorMap& tdv32, const BwdParams& p,
                            int n_clusters, cudaStream_t stream) {
    if (p.n_items == 0) return cudaSuccess;
    constexpr int smem = sizeof(PairSmem);
    constexpr int kMaxDevices = 64;
    static bool configured[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices || !configured[dev]) {
        e = cudaFuncSetAttribute(zl_bwd_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < kMaxDevices) configured[dev] = true;
    }
    zl_bwd_pair_kernel<<<2 * n_clusters, kPairThreads, smem, stream>>>(tq, tq64, tk, tv, tdo, tdo64, tdq, taug, tdk32, tdv32, p);
    return cudaGetLastError();
}

}  // namespace zl
