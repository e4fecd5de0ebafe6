// Internal definitions shared by the host scheduler and the kernels of libzellige.
#pragma once

#include <cstdint>
#include <vector>

#include "zellige.h"

namespace zl {

constexpr int kTileQ = 128;   // query rows per MMA tile (TMEM lanes)
constexpr int kTileKV = 128;  // key rows per MMA tile
constexpr int kFwdBlockQ = 2 * kTileQ;  // query rows per forward work item: two tiles in flight per CTA

// One attention task on the device: whole sequence or shard.
struct alignas(32) Task {
    int32_t q_off, q_len, kv_off, kv_len;
    int32_t partial_slot;  // first row of the task's slot in o_partial, -1 for a whole sequence
    int32_t q_slot;        // first row of the task's query range in the padded backward scratch
    int32_t kv_group;      // -1 if kv_len == 0
    int32_t q_group;       // index of the distinct query range (dQ accumulation unit)
};

// (task | kv group, head, first row relative to the task's query range | group's key range, rows)
struct alignas(16) WorkItem {
    int32_t unit, head, row0, rows;
};

// Shard tasks that share a query range and a head range; they are merged for heads
// [head_begin, head_begin + head_count) only.
struct alignas(32) MergeGroup {
    int32_t q_off, q_len;
    int32_t part_begin, n_parts;  // range in the merge part list (partial slot row offsets)
    int32_t head_begin, head_count;
    int32_t pad_[2];
};

// A distinct (query range, head range): rows [slot, slot + pad128(q_len)) of the backward scratch
// arrays, of which only the heads of the range are used.
struct alignas(32) QGroup {
    int32_t q_off, q_len, slot, pad;
    int32_t head_begin, head_count;
    int32_t pad_[2];
};

struct alignas(16) KvGroup {
    int32_t kv_off, kv_len;
    int32_t task_begin, n_tasks;  // range in the kv-group task list
    int32_t n_q_tiles;            // 128-row query tiles of all its tasks together
    int32_t pad_[3];
};

// One attention problem of a placement as the builder receives it: a whole sequence (q range ==
// kv range, final after the forward launch) or a shard (one query chunk x one K/V chunk), over the
// heads [head_begin, head_begin + head_count).
struct InputTask {
    int32_t q_off, q_len, kv_off, kv_len, seq_id;
    int32_t head_begin, head_count;
    int32_t shard_idx;  // index into the caller's shard array, -1 for a whole sequence
};

// Everything zl_build_tasks derives from a placement, on the host.
struct Schedule {
    int32_t n_heads = 0, head_dim = 0, total_q = 0, total_kv = 0;
    std::vector<Task> tasks;
    std::vector<int32_t> task_head_begin, task_head_count;  // per task (host only: items carry their head)
    std::vector<int32_t> whole_to_task;     // per input whole sequence: task index or -1 (empty sequence)
    std::vector<int32_t> shard_to_task;     // per input shard: task index or -1 (q_len == 0)
    std::vector<int32_t> shard_slot_off;    // per input shard: slot row offset (or 0)
    std::vector<int32_t> shard_slot_rows;   // per input shard: padded slot rows (0 if skipped)
    std::vector<MergeGroup> merge_groups;
    std::vector<int32_t> merge_parts;       // slot row offsets, ascending shard order per group
    std::vector<int32_t> merge_row_prefix;  // n_merge_groups+1 prefix sums of q_len
    std::vector<QGroup> q_groups;
    int64_t q_pad_total = 0;                // rows of the padded backward scratch arrays
    std::vector<KvGroup> kv_groups;
    std::vector<int32_t> kv_group_tasks;
    std::vector<WorkItem> fwd_items;
    std::vector<WorkItem> bwd_items;
    std::vector<WorkItem> bwd_pair_items;   // (kv group, head, first key row, rows <= 256): two key tiles per CTA pair
    // Launch phases: the work lists are grouped by phase and a phased launch walks one group.  Forward phases are
    // per task, backward phases per kv group; one phase (the whole list) until zl_set_fwd_phases / zl_set_bwd_phases.
    std::vector<int32_t> fwd_task_phase, bwd_group_phase;
    std::vector<int32_t> fwd_phase_begin, bwd_phase_begin, bwd_pair_phase_begin;  // n_phases + 1 offsets into the lists
    int64_t partial_rows = 0;
    int32_t n_fused_ranges = 0;             // shard query ranges lowered to one final task (chunk fusion)
    size_t bwd_workspace_bytes = 0;
    // byte offsets inside the backward workspace
    size_t ws_dq_acc_off = 0, ws_aug_off = 0;
};

// Validates the placement and fills `s`.  Pure host code, no CUDA.
// `in`: whole sequences first (in placement order), then shards (in the caller's order); `n_shards` is
// the size of the caller's shard array.  `flags`: ZL_BUILD_* bits of zl_build_tasks_ex.
zl_status build_schedule(const std::vector<InputTask>& in, int32_t n_shards, int32_t total_q, int32_t total_kv,
                         int32_t n_heads, int32_t head_dim, uint32_t flags, Schedule* s);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace zl
