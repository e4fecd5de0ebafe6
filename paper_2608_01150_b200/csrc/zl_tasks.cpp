// Host scheduler of libzellige: lowers a placement (whole sequences + shard descriptors)
// into task tables and longest-first work lists.  Pure host code.
//
// Paper Section IV-D: the engine "lowers the placement into a rank-local schedule" and packs
// all whole sequences of a rank into one block-diagonal call beside the rank's shards.  The
// paper orders segments by decreasing split degree so that collectives line up across
// ranks; on one GPU there are no collectives, and the order that matters is the one that
// keeps a long sequence from finishing last, so items are sorted longest-first.
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

// Ranges must be pairwise identical or disjoint.
bool identical_or_disjoint(std::vector<Range> r) {
    std::sort(r.begin(), r.end());
    r.erase(std::unique(r.begin(), r.end()), r.end());
    for (size_t i = 1; i < r.size(); ++i)
        if (r[i - 1].off + r[i - 1].len > r[i].off) return false;
    return true;
}

}  // namespace

zl_status build_schedule(const int32_t* cu, int32_t n_whole, const zl_shard_desc* shards,
                         int32_t n_shards, int32_t total_q, int32_t total_kv, int32_t n_heads,
                         int32_t head_dim, uint32_t flags, Schedule* s) {
    if (!s || n_whole < 0 || n_shards < 0 || total_q < 0 || total_kv < 0 || n_heads <= 0)
        return ZL_ERR_INVALID_ARG;
    if ((n_whole > 0 && !cu) || (n_shards > 0 && !shards)) return ZL_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return ZL_ERR_UNSUPPORTED;

    *s = Schedule();
    s->n_heads = n_heads; s->head_dim = head_dim; s->total_q = total_q; s->total_kv = total_kv;

    int64_t whole_end = 0;
    if (n_whole > 0) {
        if (cu[0] != 0) return ZL_ERR_INVALID_ARG;
        for (int i = 0; i < n_whole; ++i)
            if (cu[i + 1] < cu[i]) return ZL_ERR_INVALID_ARG;
        whole_end = cu[n_whole];
        if (whole_end > total_q || whole_end > total_kv) return ZL_ERR_INVALID_ARG;
    }

    std::vector<Range> q_ranges, kv_ranges;
    // whole sequences
    for (int i = 0; i < n_whole; ++i) {
        const int32_t len = cu[i + 1] - cu[i];
        if (len == 0) continue;
        Task t{};
        t.q_off = cu[i]; t.q_len = len; t.kv_off = cu[i]; t.kv_len = len;
        t.partial_slot = -1; t.q_slot = 0; t.kv_group = -1; t.q_group = -1;
        s->tasks.push_back(t);
        q_ranges.push_back({cu[i], len});
        kv_ranges.push_back({cu[i], len});
    }
    // Optional fusion of local chunks: a query range whose non-empty key chunks, sorted by offset,
    // tile one contiguous interval needs no partials and no merge -- it is exact attention over
    // the interval, i.e. one task that is final after the forward launch.  Done for all such
    // ranges or for none: the fused intervals must still be identical-or-disjoint with every other
    // key range of the placement.
    std::vector<int32_t> fuse_leader(n_shards, -1);  // per shard: first shard of its fused range, or -1
    std::vector<Range> fuse_union(n_shards, Range{0, 0});
    if ((flags & ZL_BUILD_FUSE_LOCAL_CHUNKS) && n_shards > 0) {
        std::map<std::pair<int64_t, int64_t>, std::vector<int32_t>> by_q;
        bool sane = true;
        for (int i = 0; i < n_shards && sane; ++i) {
            const zl_shard_desc& d = shards[i];
            if (d.q_len < 0 || d.kv_len < 0 || d.q_off < 0 || d.kv_off < 0) sane = false;
            else if (d.q_len > 0) by_q[{d.q_off, d.q_len}].push_back(i);
        }
        std::vector<Range> all_kv;
        for (int i = 0; i < n_whole; ++i)
            if (cu[i + 1] > cu[i]) all_kv.push_back({cu[i], cu[i + 1] - cu[i]});
        for (auto& kvp : by_q) {
            if (!sane) break;
            std::vector<Range> chunks;
            for (int32_t i : kvp.second)
                if (shards[i].kv_len > 0) chunks.push_back({shards[i].kv_off, shards[i].kv_len});
            std::sort(chunks.begin(), chunks.end());
            bool contiguous = chunks.size() >= 2;
            for (size_t c = 1; c < chunks.size() && contiguous; ++c)
                contiguous = chunks[c - 1].off + chunks[c - 1].len == chunks[c].off;
            if (contiguous) {
                const Range u{chunks.front().off, chunks.back().off + chunks.back().len - chunks.front().off};
                for (int32_t i : kvp.second) { fuse_leader[i] = kvp.second.front(); fuse_union[i] = u; }
                all_kv.push_back(u);
            } else {
                for (const Range& c : chunks) all_kv.push_back(c);
            }
        }
        if (!sane || !identical_or_disjoint(all_kv)) std::fill(fuse_leader.begin(), fuse_leader.end(), -1);
    }

    // shards
    s->shard_to_task.assign(n_shards, -1);
    s->shard_slot_off.assign(n_shards, 0);
    s->shard_slot_rows.assign(n_shards, 0);
    std::map<std::pair<int64_t, int64_t>, int32_t> merge_index;  // q range -> merge group
    std::vector<std::vector<int32_t>> merge_members;             // task indices per group
    std::vector<int32_t> merge_seq;
    std::vector<std::tuple<int64_t, int64_t, int64_t, int64_t>> seen_pairs;
    for (int i = 0; i < n_shards; ++i) {
        const zl_shard_desc& d = shards[i];
        if (d.q_len < 0 || d.kv_len < 0 || d.q_off < 0 || d.kv_off < 0) return ZL_ERR_INVALID_ARG;
        if ((int64_t)d.q_off + d.q_len > total_q || (int64_t)d.kv_off + d.kv_len > total_kv)
            return ZL_ERR_INVALID_ARG;
        if (d.q_len == 0) continue;
        if (d.q_off < whole_end || (d.kv_len > 0 && d.kv_off < whole_end)) return ZL_ERR_OVERLAP;
        if (d.kv_len > 0) {
            auto key = std::make_tuple((int64_t)d.q_off, (int64_t)d.q_len, (int64_t)d.kv_off, (int64_t)d.kv_len);
            if (std::find(seen_pairs.begin(), seen_pairs.end(), key) != seen_pairs.end())
                return ZL_ERR_OVERLAP;
            seen_pairs.push_back(key);
            kv_ranges.push_back({d.kv_off, d.kv_len});
        }
        q_ranges.push_back({d.q_off, d.q_len});
        Task t{};
        t.q_off = d.q_off; t.q_len = d.q_len; t.kv_off = d.kv_off; t.kv_len = d.kv_len;
        t.kv_group = -1; t.q_group = -1; t.q_slot = 0;
        if (fuse_leader[i] >= 0) {
            // fused query range: its first shard carries the task over the whole interval, final
            // after the forward launch; the other shards of the range add nothing
            if (d.kv_len > 0) kv_ranges.back() = fuse_union[i];
            if (fuse_leader[i] != i) {
                if (shards[fuse_leader[i]].seq_id != d.seq_id) return ZL_ERR_INVALID_ARG;
                s->shard_to_task[i] = s->shard_to_task[fuse_leader[i]];
                continue;
            }
            t.kv_off = (int32_t)fuse_union[i].off; t.kv_len = (int32_t)fuse_union[i].len;
            t.partial_slot = -1;
            s->shard_to_task[i] = (int32_t)s->tasks.size();
            s->tasks.push_back(t);
            ++s->n_fused_ranges;
            continue;
        }
        auto mk = std::make_pair((int64_t)d.q_off, (int64_t)d.q_len);
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
        s->shard_slot_off[i] = t.partial_slot;
        s->shard_slot_rows[i] = padded;
        s->partial_rows += padded;
        s->shard_to_task[i] = (int32_t)s->tasks.size();
        merge_members[it->second].push_back((int32_t)s->tasks.size());
        s->tasks.push_back(t);
    }
    if (!identical_or_disjoint(q_ranges) || !identical_or_disjoint(kv_ranges)) return ZL_ERR_OVERLAP;
    if (s->partial_rows > INT32_MAX) return ZL_ERR_INVALID_ARG;

    // merge groups, in order of first appearance; parts in ascending shard order
    s->merge_row_prefix.push_back(0);
    for (size_t g = 0; g < merge_members.size(); ++g) {
        const Task& t0 = s->tasks[merge_members[g][0]];
        MergeGroup mg{t0.q_off, t0.q_len, (int32_t)s->merge_parts.size(), (int32_t)merge_members[g].size()};
        for (int32_t ti : merge_members[g]) s->merge_parts.push_back(s->tasks[ti].partial_slot);
        s->merge_groups.push_back(mg);
        s->merge_row_prefix.push_back(s->merge_row_prefix.back() + t0.q_len);
    }

    // query groups (distinct query ranges) and kv groups (distinct key ranges)
    {
        std::map<std::pair<int64_t, int64_t>, int32_t> qg, kg;
        std::vector<std::vector<int32_t>> kmembers;
        for (size_t ti = 0; ti < s->tasks.size(); ++ti) {
            Task& t = s->tasks[ti];
            auto qk = std::make_pair((int64_t)t.q_off, (int64_t)t.q_len);
            auto qi = qg.find(qk);
            if (qi == qg.end()) {
                qi = qg.emplace(qk, (int32_t)s->q_groups.size()).first;
                const int32_t pad = (int32_t)align_up((size_t)t.q_len, kTileQ);
                s->q_groups.push_back({t.q_off, t.q_len, (int32_t)s->q_pad_total, pad});
                s->q_pad_total += pad;
            }
            t.q_group = qi->second;
            t.q_slot = s->q_groups[qi->second].slot;
            if (t.kv_len == 0) continue;
            auto kk = std::make_pair((int64_t)t.kv_off, (int64_t)t.kv_len);
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
            KvGroup kgp{t0.kv_off, t0.kv_len, (int32_t)s->kv_group_tasks.size(), (int32_t)kmembers[g].size()};
            for (int32_t ti : kmembers[g]) s->kv_group_tasks.push_back(ti);
            s->kv_groups.push_back(kgp);
        }
    }

    // forward work list: (task, head, query block), longest-first
    for (size_t ti = 0; ti < s->tasks.size(); ++ti) {
        const Task& t = s->tasks[ti];
        for (int32_t h = 0; h < n_heads; ++h)
            for (int32_t r = 0; r < t.q_len; r += kFwdBlockQ)
                s->fwd_items.push_back({(int32_t)ti, h, r, std::min(kFwdBlockQ, t.q_len - r)});
    }
    std::stable_sort(s->fwd_items.begin(), s->fwd_items.end(), [&](const WorkItem& a, const WorkItem& b) {
        const int32_t ka = s->tasks[a.unit].kv_len, kb = s->tasks[b.unit].kv_len;
        if (ka != kb) return ka > kb;
        if (a.rows != b.rows) return a.rows > b.rows;
        return std::tie(a.unit, a.head, a.row0) < std::tie(b.unit, b.head, b.row0);
    });

    // backward work list: (kv group, head, key tile); cost = total query rows served
    std::vector<int64_t> group_cost(s->kv_groups.size(), 0);
    for (size_t g = 0; g < s->kv_groups.size(); ++g)
        for (int32_t j = 0; j < s->kv_groups[g].n_tasks; ++j)
            group_cost[g] += s->tasks[s->kv_group_tasks[s->kv_groups[g].task_begin + j]].q_len;
    for (size_t g = 0; g < s->kv_groups.size(); ++g)
        for (int32_t h = 0; h < n_heads; ++h)
            for (int32_t r = 0; r < s->kv_groups[g].kv_len; r += kTileKV)
                s->bwd_items.push_back({(int32_t)g, h, r, std::min(kTileKV, s->kv_groups[g].kv_len - r)});
    std::stable_sort(s->bwd_items.begin(), s->bwd_items.end(), [&](const WorkItem& a, const WorkItem& b) {
        if (group_cost[a.unit] != group_cost[b.unit]) return group_cost[a.unit] > group_cost[b.unit];
        if (a.rows != b.rows) return a.rows > b.rows;
        return std::tie(a.unit, a.head, a.row0) < std::tie(b.unit, b.head, b.row0);
    });

    // backward workspace over the padded query slots: fp32 dQ accumulator [q_pad, H, d], then one
    // 4 KB "augmentation" tile per (head, 128-row query tile) holding -LSE/scale and -D split
    // into bf16 pieces (see the backward preprocess kernel)
    if (s->q_pad_total > INT32_MAX) return ZL_ERR_INVALID_ARG;
    s->ws_dq_acc_off = 0;
    s->ws_aug_off = align_up((size_t)s->q_pad_total * n_heads * head_dim * sizeof(float), 256);
    s->bwd_workspace_bytes = s->ws_aug_off + align_up((size_t)(s->q_pad_total / kTileQ) * n_heads * 4096, 256);
    return ZL_OK;
}

}  // namespace zl
