// Host scheduler of libzellige: lowers a placement (whole sequences + shard descriptors, each
// over a range of heads) into task tables and longest-first work lists.  Pure host code.
//
// Paper Section IV-D: the engine "lowers the placement into a rank-local schedule" and packs
// all whole sequences of a rank into one block-diagonal call beside the rank's shards; its
// second coalescing mode batches Ulysses sequences, which hold all tokens of a sequence for a
// subset of the heads.  The paper orders segments by decreasing split degree so that
// collectives line up across ranks; on one GPU there are no collectives, and the order that
// matters is the one that keeps a long sequence from finishing last, so items are sorted
// longest-first.
#include <algorithm>
#include <map>
#include <tuple>
#include <utility>

#include "zl_internal.h"

namespace zl {

namespace {

struct Range {
    int64_t off, len;
    bool operator<(const Range& o) const { return std::tie(off, len) < std::tie(o.off, o.len); }
    bool operator==(const Range& o) const { return off == o.off && len == o.len; }
};

using HeadRange = std::pair<int32_t, int32_t>;  // [first, second)

// Ranges must be pairwise identical or disjoint.
bool identical_or_disjoint(std::vector<Range> r) {
    std::sort(r.begin(), r.end());
    r.erase(std::unique(r.begin(), r.end()), r.end());
    for (size_t i = 1; i < r.size(); ++i)
        if (r[i - 1].off + r[i - 1].len > r[i].off) return false;
    return true;
}

// Head by head, the ranges of the tasks that cover the head must be pairwise identical or disjoint,
// and tasks with an identical range must cover the same heads (they form one accumulation group:
// a range claimed by two different head sets would be written by two groups).  Empty ranges are
// ignored.  The heads are walked as the elementary intervals between the tasks' range ends.
bool ranges_consistent(const std::vector<Range>& rng, const std::vector<HeadRange>& heads) {
    std::vector<int32_t> cuts;
    for (size_t i = 0; i < rng.size(); ++i)
        if (rng[i].len > 0) { cuts.push_back(heads[i].first); cuts.push_back(heads[i].second); }
    std::sort(cuts.begin(), cuts.end());
    cuts.erase(std::unique(cuts.begin(), cuts.end()), cuts.end());
    for (size_t c = 0; c + 1 < cuts.size(); ++c) {
        const int32_t a = cuts[c], b = cuts[c + 1];
        std::vector<Range> sel;
        std::map<Range, HeadRange> owner;
        for (size_t i = 0; i < rng.size(); ++i) {
            if (rng[i].len == 0 || heads[i].first > a || heads[i].second < b) continue;
            sel.push_back(rng[i]);
            auto it = owner.emplace(rng[i], heads[i]);
            if (!it.second && it.first->second != heads[i]) return false;
        }
        if (!identical_or_disjoint(std::move(sel))) return false;
    }
    return true;
}

using GroupKey = std::tuple<int64_t, int64_t, int32_t, int32_t>;  // range offset, length, head range

}  // namespace

zl_status build_schedule(const std::vector<InputTask>& in, int32_t n_shards, int32_t total_q, int32_t total_kv,
                         int32_t n_heads, int32_t head_dim, uint32_t flags, Schedule* s) {
    if (!s || n_shards < 0 || total_q < 0 || total_kv < 0 || n_heads <= 0) return ZL_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return ZL_ERR_UNSUPPORTED;

    *s = Schedule();
    s->n_heads = n_heads; s->head_dim = head_dim; s->total_q = total_q; s->total_kv = total_kv;

    // ---- per-descriptor checks; the whole region ends where the last whole sequence ends
    int64_t whole_end = 0;
    for (const InputTask& t : in) {
        if (t.q_len < 0 || t.kv_len < 0 || t.q_off < 0 || t.kv_off < 0) return ZL_ERR_INVALID_ARG;
        if ((int64_t)t.q_off + t.q_len > total_q || (int64_t)t.kv_off + t.kv_len > total_kv) return ZL_ERR_INVALID_ARG;
        if (t.head_begin < 0 || t.head_count < 1 || (int64_t)t.head_begin + t.head_count > n_heads)
            return ZL_ERR_INVALID_ARG;
        if (t.shard_idx >= n_shards) return ZL_ERR_INVALID_ARG;
        if (t.shard_idx < 0 && t.q_len > 0) whole_end = std::max<int64_t>(whole_end, (int64_t)t.q_off + t.q_len);
    }
    const size_t n_in = in.size();
    std::vector<bool> live(n_in, false);  // contributes a task (or part of a fused one)
    for (size_t i = 0; i < n_in; ++i) {
        const InputTask& t = in[i];
        if (t.q_len == 0) continue;
        if (t.shard_idx >= 0 && (t.q_off < whole_end || (t.kv_len > 0 && t.kv_off < whole_end))) return ZL_ERR_OVERLAP;
        live[i] = true;
    }

    std::vector<Range> q_rng(n_in), kv_rng(n_in);
    std::vector<HeadRange> heads(n_in);
    for (size_t i = 0; i < n_in; ++i) {
        q_rng[i] = live[i] ? Range{in[i].q_off, in[i].q_len} : Range{0, 0};
        kv_rng[i] = live[i] ? Range{in[i].kv_off, in[i].kv_len} : Range{0, 0};
        heads[i] = {in[i].head_begin, in[i].head_begin + in[i].head_count};
    }
    if (!ranges_consistent(q_rng, heads) || !ranges_consistent(kv_rng, heads)) return ZL_ERR_OVERLAP;
    // the same (query range, key range) twice on a common head
    {
        std::map<std::tuple<int64_t, int64_t, int64_t, int64_t>, std::vector<HeadRange>> seen;
        for (size_t i = 0; i < n_in; ++i) {
            if (!live[i] || in[i].kv_len == 0) continue;
            auto& v = seen[std::make_tuple(q_rng[i].off, q_rng[i].len, kv_rng[i].off, kv_rng[i].len)];
            for (const HeadRange& h : v)
                if (h.first < heads[i].second && heads[i].first < h.second) return ZL_ERR_OVERLAP;
            v.push_back(heads[i]);
        }
    }

    // ---- optional fusion of local chunks: a (query range, head range) whose non-empty key chunks, sorted
    // by offset, tile one contiguous interval needs no partials and no merge -- it is exact attention
    // over the interval, i.e. one task that is final after the forward launch.  Done for all such
    // ranges or for none: the fused intervals must still be consistent with every other key range.
    std::vector<int32_t> fuse_leader(n_in, -1);  // per input: first input of its fused range, or -1
    std::vector<Range> fuse_union(n_in, Range{0, 0});
    if (flags & ZL_BUILD_FUSE_LOCAL_CHUNKS) {
        std::map<GroupKey, std::vector<int32_t>> by_q;
        for (size_t i = 0; i < n_in; ++i)
            if (live[i] && in[i].shard_idx >= 0)
                by_q[GroupKey(q_rng[i].off, q_rng[i].len, heads[i].first, heads[i].second)].push_back((int32_t)i);
        std::vector<Range> eff_kv = kv_rng;
        for (auto& kvp : by_q) {
            std::vector<Range> chunks;
            for (int32_t i : kvp.second)
                if (in[i].kv_len > 0) chunks.push_back(kv_rng[i]);
            std::sort(chunks.begin(), chunks.end());
            bool contiguous = chunks.size() >= 2;
            for (size_t c = 1; c < chunks.size() && contiguous; ++c)
                contiguous = chunks[c - 1].off + chunks[c - 1].len == chunks[c].off;
            if (!contiguous) continue;
            const Range u{chunks.front().off, chunks.back().off + chunks.back().len - chunks.front().off};
            for (int32_t i : kvp.second) {
                fuse_leader[i] = kvp.second.front();
                fuse_union[i] = u;
                eff_kv[i] = (i == kvp.second.front()) ? u : Range{0, 0};
            }
        }
        if (!ranges_consistent(eff_kv, heads)) std::fill(fuse_leader.begin(), fuse_leader.end(), -1);
    }

    // ---- tasks: whole sequences in placement order, then shards in the caller's order
    s->whole_to_task.clear();
    s->shard_to_task.assign(n_shards, -1);
    s->shard_slot_off.assign(n_shards, 0);
    s->shard_slot_rows.assign(n_shards, 0);
    std::map<GroupKey, int32_t> merge_index;          // (query range, head range) -> merge group
    std::vector<std::vector<int32_t>> merge_members;  // task indices per group
    std::vector<int32_t> merge_seq;
    auto push_task = [&](const Task& t, const InputTask& src) {
        s->tasks.push_back(t);
        s->task_head_begin.push_back(src.head_begin);
        s->task_head_count.push_back(src.head_count);
    };
    for (size_t i = 0; i < n_in; ++i) {
        if (in[i].shard_idx < 0) s->whole_to_task.push_back(live[i] ? (int32_t)s->tasks.size() : -1);
        if (!live[i]) continue;
        const InputTask& d = in[i];
        Task t{};
        t.q_off = d.q_off; t.q_len = d.q_len; t.kv_off = d.kv_off; t.kv_len = d.kv_len;
        t.partial_slot = -1; t.q_slot = 0; t.kv_group = -1; t.q_group = -1;
        if (d.shard_idx < 0) {  // whole sequence: final after the forward launch
            push_task(t, d);
            continue;
        }
        if (fuse_leader[i] >= 0) {
            // fused query range: its first shard carries the task over the whole interval, final
            // after the forward launch; the other shards of the range add nothing
            if (fuse_leader[i] != (int32_t)i) {
                if (in[fuse_leader[i]].seq_id != d.seq_id) return ZL_ERR_INVALID_ARG;
                s->shard_to_task[d.shard_idx] = s->shard_to_task[in[fuse_leader[i]].shard_idx];
                continue;
            }
            t.kv_off = (int32_t)fuse_union[i].off; t.kv_len = (int32_t)fuse_union[i].len;
            s->shard_to_task[d.shard_idx] = (int32_t)s->tasks.size();
            push_task(t, d);
            ++s->n_fused_ranges;
            continue;
        }
        const GroupKey mk(d.q_off, d.q_len, d.head_begin, d.head_begin + d.head_count);
        auto it = merge_index.find(mk);
        if (it == merge_index.end()) {
            it = merge_index.emplace(mk, (int32_t)merge_members.size()).first;
            merge_members.emplace_back();
            merge_seq.push_back(d.seq_id);
        } else if (merge_seq[it->second] != d.seq_id) {
            return ZL_ERR_INVALID_ARG;
        }
        // slot padded to whole query tiles so a full-tile store of a ragged last tile can
        // never reach another task's slot
        const int32_t padded = (int32_t)align_up((size_t)d.q_len, kTileQ);
        t.partial_slot = (int32_t)s->partial_rows;
        s->shard_slot_off[d.shard_idx] = t.partial_slot;
        s->shard_slot_rows[d.shard_idx] = padded;
        s->partial_rows += padded;
        if (s->partial_rows > INT32_MAX) return ZL_ERR_INVALID_ARG;
        s->shard_to_task[d.shard_idx] = (int32_t)s->tasks.size();
        merge_members[it->second].push_back((int32_t)s->tasks.size());
        push_task(t, d);
    }

    // merge groups, in order of first appearance; parts in ascending shard order
    s->merge_row_prefix.push_back(0);
    for (size_t g = 0; g < merge_members.size(); ++g) {
        const int32_t t0i = merge_members[g][0];
        const Task& t0 = s->tasks[t0i];
        MergeGroup mg{};
        mg.q_off = t0.q_off; mg.q_len = t0.q_len;
        mg.part_begin = (int32_t)s->merge_parts.size(); mg.n_parts = (int32_t)merge_members[g].size();
        mg.head_begin = s->task_head_begin[t0i]; mg.head_count = s->task_head_count[t0i];
        for (int32_t ti : merge_members[g]) s->merge_parts.push_back(s->tasks[ti].partial_slot);
        s->merge_groups.push_back(mg);
        s->merge_row_prefix.push_back(s->merge_row_prefix.back() + t0.q_len);
    }

    // query groups (distinct query range x head range) and kv groups (distinct key range x head range)
    {
        std::map<GroupKey, int32_t> qg, kg;
        std::vector<std::vector<int32_t>> kmembers;
        for (size_t ti = 0; ti < s->tasks.size(); ++ti) {
            Task& t = s->tasks[ti];
            const int32_t hb = s->task_head_begin[ti], he = hb + s->task_head_count[ti];
            const GroupKey qk(t.q_off, t.q_len, hb, he);
            auto qi = qg.find(qk);
            if (qi == qg.end()) {
                qi = qg.emplace(qk, (int32_t)s->q_groups.size()).first;
                const int32_t pad = (int32_t)align_up((size_t)t.q_len, kTileQ);
                QGroup g{};
                g.q_off = t.q_off; g.q_len = t.q_len; g.slot = (int32_t)s->q_pad_total; g.pad = pad;
                g.head_begin = hb; g.head_count = he - hb;
                s->q_groups.push_back(g);
                s->q_pad_total += pad;
                if (s->q_pad_total > INT32_MAX) return ZL_ERR_INVALID_ARG;
            }
            t.q_group = qi->second;
            t.q_slot = s->q_groups[qi->second].slot;
            if (t.kv_len == 0) continue;
            const GroupKey kk(t.kv_off, t.kv_len, hb, he);
            auto ki = kg.find(kk);
            if (ki == kg.end()) {
                ki = kg.emplace(kk, (int32_t)kmembers.size()).first;
                kmembers.emplace_back();
            }
            t.kv_group = ki->second;
            kmembers[ki->second].push_back((int32_t)ti);
        }
        for (size_t g = 0; g < kmembers.size(); ++g) {
            const Task& t0 = s->tasks[kmembers[g][0]];
            KvGroup kgp{t0.kv_off, t0.kv_len, (int32_t)s->kv_group_tasks.size(), (int32_t)kmembers[g].size(), 0, {0, 0, 0}};
            for (int32_t ti : kmembers[g]) {
                s->kv_group_tasks.push_back(ti);
                kgp.n_q_tiles += (s->tasks[ti].q_len + kTileQ - 1) / kTileQ;
            }
            s->kv_groups.push_back(kgp);
        }
    }

    // forward work list: (task, head of the task's range, query block), longest-first
    for (size_t ti = 0; ti < s->tasks.size(); ++ti) {
        const Task& t = s->tasks[ti];
        for (int32_t h = s->task_head_begin[ti]; h < s->task_head_begin[ti] + s->task_head_count[ti]; ++h)
            for (int32_t r = 0; r < t.q_len; r += kFwdBlockQ)
                s->fwd_items.push_back({(int32_t)ti, h, r, std::min(kFwdBlockQ, t.q_len - r)});
    }
    std::stable_sort(s->fwd_items.begin(), s->fwd_items.end(), [&](const WorkItem& a, const WorkItem& b) {
        const int32_t ka = s->tasks[a.unit].kv_len, kb = s->tasks[b.unit].kv_len;
        if (ka != kb) return ka > kb;
        if (a.rows != b.rows) return a.rows > b.rows;
        return std::tie(a.unit, a.head, a.row0) < std::tie(b.unit, b.head, b.row0);
    });

    // backward work list: (kv group, head of the group's range, key tile); cost = total query rows served
    std::vector<int64_t> group_cost(s->kv_groups.size(), 0);
    for (size_t g = 0; g < s->kv_groups.size(); ++g)
        for (int32_t j = 0; j < s->kv_groups[g].n_tasks; ++j)
            group_cost[g] += s->tasks[s->kv_group_tasks[s->kv_groups[g].task_begin + j]].q_len;
    for (size_t g = 0; g < s->kv_groups.size(); ++g) {
        const int32_t t0 = s->kv_group_tasks[s->kv_groups[g].task_begin];
        for (int32_t h = s->task_head_begin[t0]; h < s->task_head_begin[t0] + s->task_head_count[t0]; ++h)
            for (int32_t r = 0; r < s->kv_groups[g].kv_len; r += kTileKV)
                s->bwd_items.push_back({(int32_t)g, h, r, std::min(kTileKV, s->kv_groups[g].kv_len - r)});
    }
    auto bwd_order = [&](const WorkItem& a, const WorkItem& b) {
        if (group_cost[a.unit] != group_cost[b.unit]) return group_cost[a.unit] > group_cost[b.unit];
        if (a.rows != b.rows) return a.rows > b.rows;
        return std::tie(a.unit, a.head, a.row0) < std::tie(b.unit, b.head, b.row0);
    };
    std::stable_sort(s->bwd_items.begin(), s->bwd_items.end(), bwd_order);
    // the same list in units of two key tiles, for the CTA-pair form of the main kernel
    for (size_t g = 0; g < s->kv_groups.size(); ++g) {
        const int32_t t0 = s->kv_group_tasks[s->kv_groups[g].task_begin];
        for (int32_t h = s->task_head_begin[t0]; h < s->task_head_begin[t0] + s->task_head_count[t0]; ++h)
            for (int32_t r = 0; r < s->kv_groups[g].kv_len; r += 2 * kTileKV)
                s->bwd_pair_items.push_back({(int32_t)g, h, r, std::min(2 * kTileKV, s->kv_groups[g].kv_len - r)});
    }
    std::stable_sort(s->bwd_pair_items.begin(), s->bwd_pair_items.end(), bwd_order);

    // one launch phase until the caller says otherwise
    s->fwd_task_phase.assign(s->tasks.size(), 0);
    s->bwd_group_phase.assign(s->kv_groups.size(), 0);
    s->fwd_phase_begin = {0, (int32_t)s->fwd_items.size()};
    s->bwd_phase_begin = {0, (int32_t)s->bwd_items.size()};
    s->bwd_pair_phase_begin = {0, (int32_t)s->bwd_pair_items.size()};

    // backward workspace over the padded query slots: fp32 dQ accumulator [q_pad, H, d], then one
    // 4 KB "augmentation" tile per (head, 128-row query tile) holding -LSE/scale and -D split
    // into bf16 pieces (see the backward preprocess kernel)
    s->ws_dq_acc_off = 0;
    s->ws_aug_off = align_up((size_t)s->q_pad_total * n_heads * head_dim * sizeof(float), 256);
    s->bwd_workspace_bytes = s->ws_aug_off + align_up((size_t)(s->q_pad_total / kTileQ) * n_heads * 4096, 256);
    return ZL_OK;
}

}  // namespace zl
