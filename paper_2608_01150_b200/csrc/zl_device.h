// Kernel parameter blocks and launch entry points shared by the C-ABI layer and the kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "zl_internal.h"

namespace zl {

struct FwdParams {
    const Task* tasks;
    const WorkItem* items;
    int32_t n_items;
    int32_t n_heads;
    int32_t total_q;
    int32_t partial_rows;
    float scale_log2;  // scale * log2(e)
    __nv_bfloat16* o;
    float* lse;
    float* o_partial;
    float* lse_partial;
    int32_t* status;  // [0] = code, [1] = where
};

struct MergeParams {
    const MergeGroup* groups;
    const int32_t* parts;       // partial slot row offsets
    const int32_t* row_prefix;  // n_groups + 1
    int32_t n_groups;
    int32_t n_heads;
    int32_t total_q;
    int32_t partial_rows;
    const float* o_partial;
    const float* lse_partial;
    __nv_bfloat16* o;
    float* lse;
};

struct BwdParams {
    const Task* tasks;
    const WorkItem* items;       // (kv group, head, first key row, rows)
    const KvGroup* kv_groups;
    const int32_t* kv_group_tasks;
    const QGroup* q_groups;
    int32_t n_items;
    int32_t n_q_groups;
    int32_t n_heads;
    int32_t total_q;
    int32_t q_pad_total;
    float scale;
    float scale_log2;
    const __nv_bfloat16* o;
    const __nv_bfloat16* d_o;
    const float* lse;
    __nv_bfloat16* dq;
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    int64_t grad_row_stride;  // elements between token rows of dq, dk, dv (H*d, or 3*H*d when packed)
    float* dq_acc;  // [q_pad_total, H, d]
    uint8_t* aug;   // [H, q_pad_total / 128] tiles of 4 KB: bf16 splits of -lse/scale and -rowsum(dO o O)
    int32_t* status;
};

cudaError_t launch_bwd_pre(int head_dim, const BwdParams& p, int n_sms, cudaStream_t stream);
cudaError_t launch_bwd_main(int head_dim, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                            const CUtensorMap& tdo, const CUtensorMap& tdq, const CUtensorMap& tdk,
                            const CUtensorMap& tdv, const BwdParams& p, int grid, cudaStream_t stream);
// CTA-pair form of the main kernel (head_dim 128): `p.items` is the pair item list, `tq64` / `tdo64` are maps
// with 64-row boxes, `taug` views the augmentation tiles as rows of 1 KB, `tdk32` / `tdv32` are the gradient maps
// with 32-row boxes (one warp's rows).
cudaError_t launch_bwd_pair(const CUtensorMap& tq, const CUtensorMap& tq64, const CUtensorMap& tk, const CUtensorMap& tv,
                            const CUtensorMap& tdo, const CUtensorMap& tdo64, const CUtensorMap& tdq,
                            const CUtensorMap& taug, const CUtensorMap& tdk32, const CUtensorMap& tdv32, const BwdParams& p,
                            int n_clusters, cudaStream_t stream);
cudaError_t launch_bwd_post(int head_dim, const BwdParams& p, int n_sms, cudaStream_t stream);

cudaError_t launch_fwd(int head_dim, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                       const CUtensorMap& to, const CUtensorMap& top, const FwdParams& p, int grid,
                       cudaStream_t stream);
// `max_parts`: the largest number of parts of any merge group (selects a register-resident variant).
cudaError_t launch_merge(int head_dim, const MergeParams& p, int max_parts, int n_sms, cudaStream_t stream);
cudaError_t launch_wait_selftest(int32_t* status, uint64_t limit_ns, cudaStream_t stream);

}  // namespace zl
