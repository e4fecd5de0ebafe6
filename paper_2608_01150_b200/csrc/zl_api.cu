// C-ABI layer of libzellige: handle management, TMA descriptor encoding, kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <tuple>

#include "zl_device.h"

using namespace zl;

struct zl_tasks {
    Schedule sched;
    int device = -1;           // -1: host-only handle (no CUDA device present)
    int n_sms = 0;
    uint8_t* d_tables = nullptr;  // one allocation holding every device table
    Task* d_tasks = nullptr;
    WorkItem* d_fwd_items = nullptr;
    WorkItem* d_bwd_items = nullptr;
    WorkItem* d_bwd_pair_items = nullptr;
    int bwd_kernel = 0;           // 0: library default, 1: one CTA per key tile, 2: CTA pairs (head_dim 128)
    int sm_margin = 0;            // SMs the persistent kernels leave free (for communication kernels running beside them)
    MergeGroup* d_merge_groups = nullptr;
    int32_t* d_merge_parts = nullptr;
    int32_t* d_merge_prefix = nullptr;
    QGroup* d_q_groups = nullptr;
    KvGroup* d_kv_groups = nullptr;
    int32_t* d_kv_group_tasks = nullptr;
    int32_t* d_status = nullptr;
    // optional per-kernel event timing (measurement only)
    mutable bool timing = false;
    mutable std::vector<cudaEvent_t> ev_start[ZL_K_COUNT], ev_stop[ZL_K_COUNT];
    mutable int ev_used[ZL_K_COUNT] = {0, 0, 0, 0, 0};
};

namespace {

std::atomic<int64_t> g_launches{0};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Tensor map over a packed [rows, H, d] bf16 tensor: box = 64 columns x 1 head x box_rows rows,
// 128-byte swizzle, zero fill outside the tensor.
// `row_stride` (elements) is the distance between token rows: H*d, or 3*H*d for a view into packed QKV.
bool make_tmap(CUtensorMap* m, const void* base, int64_t rows, int n_heads, int head_dim, int box_rows,
               int64_t row_stride) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)n_heads, (cuuint64_t)(rows > 0 ? rows : 1)};
    cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)row_stride * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

constexpr int kMaxTimedLaunches = 1024;
constexpr bool kDefaultBwdPair = true;   // which backward main kernel a handle uses unless zl_set_bwd_kernel chose one

// Brackets one kernel launch with events when timing is enabled on the handle.
struct LaunchTimer {
    const zl_tasks* t;
    int id;
    cudaStream_t cs;
    cudaEvent_t stop = nullptr;
    LaunchTimer(const zl_tasks* t_, int id_, cudaStream_t cs_) : t(t_), id(id_), cs(cs_) {
        if (!t->timing || t->ev_used[id] >= kMaxTimedLaunches) return;
        const int i = t->ev_used[id];
        if ((int)t->ev_start[id].size() <= i) {
            cudaEvent_t a, b;
            if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
            t->ev_start[id].push_back(a);
            t->ev_stop[id].push_back(b);
        }
        cudaEventRecord(t->ev_start[id][i], cs);
        stop = t->ev_stop[id][i];
        t->ev_used[id] = i + 1;
    }
    ~LaunchTimer() { if (stop) cudaEventRecord(stop, cs); }
};

// Tensor map over the fp32 dQ accumulator [rows, H, d]: box = 32 columns x 1 head x box_rows rows with 128-byte
// swizzle, or (box_cols = 16) 16 columns with 64-byte swizzle.
bool make_tmap_f32_acc(CUtensorMap* m, const void* base, int64_t rows, int n_heads, int head_dim, int box_rows = 32,
                       int box_cols = 32) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)n_heads, (cuuint64_t)(rows > 0 ? rows : 1)};
    cuuint64_t strides[2] = {(cuuint64_t)head_dim * 4, (cuuint64_t)head_dim * 4 * n_heads};
    cuuint32_t box[3] = {(cuuint32_t)box_cols, 1, (cuuint32_t)box_rows};  // one warp's 32 rows (dQ) or a 128-row tile
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, box_cols == 16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The augmentation tiles of the backward workspace as a 2-D array of 1 KB rows (256 x 32-bit): row
// tile * 4 + chunk * 2 + half holds one K chunk of one 64-row half of a tile.
bool make_tmap_aug_rows(CUtensorMap* m, const void* base, int64_t n_tiles) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {256, (cuuint64_t)(n_tiles > 0 ? n_tiles * 4 : 1)};
    cuuint64_t strides[1] = {1024};
    cuuint32_t box[2] = {256, 1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Launches go to the current device: it has to be the one the handle's tables live on.
bool on_handle_device(const zl_tasks* t) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == t->device;
}

template <class T>
size_t place(size_t& off, size_t count) {
    off = align_up(off, 256);
    const size_t at = off;
    off += count * sizeof(T);
    return at;
}

}  // namespace

extern "C" {

const char* zl_status_str(zl_status s) {
    switch (s) {
        case ZL_OK: return "ZL_OK";
        case ZL_ERR_INVALID_ARG: return "ZL_ERR_INVALID_ARG";
        case ZL_ERR_OVERLAP: return "ZL_ERR_OVERLAP";
        case ZL_ERR_UNSUPPORTED: return "ZL_ERR_UNSUPPORTED";
        case ZL_ERR_WORKSPACE: return "ZL_ERR_WORKSPACE";
        case ZL_ERR_CUDA: return "ZL_ERR_CUDA";
        case ZL_ERR_TIMEOUT: return "ZL_ERR_TIMEOUT";
    }
    return "ZL_ERR_UNKNOWN";
}

int64_t zl_launch_count(void) { return g_launches.load(); }

zl_status zl_build_tasks(const int32_t* cu_seqlens, int32_t n_whole, const zl_shard_desc* shards,
                         int32_t n_shards, int32_t total_q, int32_t total_kv, int32_t n_heads,
                         int32_t head_dim, void* stream, zl_tasks** out) {
    return zl_build_tasks_ex(cu_seqlens, n_whole, shards, n_shards, total_q, total_kv, n_heads, head_dim, 0u,
                             stream, out);
}

zl_status zl_build_tasks_ex(const int32_t* cu_seqlens, int32_t n_whole, const zl_shard_desc* shards,
                            int32_t n_shards, int32_t total_q, int32_t total_kv, int32_t n_heads,
                            int32_t head_dim, uint32_t flags, void* stream, zl_tasks** out) {
    if (!out) return ZL_ERR_INVALID_ARG;
    *out = nullptr;
    if (n_whole < 0 || (n_whole > 0 && !cu_seqlens)) return ZL_ERR_INVALID_ARG;
    std::vector<zl_whole_desc> whole;
    if (n_whole > 0) {
        if (cu_seqlens[0] != 0) return ZL_ERR_INVALID_ARG;
        for (int i = 0; i < n_whole; ++i) {
            if (cu_seqlens[i + 1] < cu_seqlens[i]) return ZL_ERR_INVALID_ARG;
            whole.push_back({cu_seqlens[i], cu_seqlens[i + 1] - cu_seqlens[i], 0, n_heads});
        }
    }
    return zl_build_tasks_heads(whole.data(), n_whole, shards, nullptr, n_shards, total_q, total_kv, n_heads,
                                head_dim, flags, stream, out);
}

zl_status zl_build_tasks_heads(const zl_whole_desc* whole, int32_t n_whole, const zl_shard_desc* shards,
                               const zl_head_range* shard_heads, int32_t n_shards, int32_t total_q,
                               int32_t total_kv, int32_t n_heads, int32_t head_dim, uint32_t flags,
                               void* stream, zl_tasks** out) {
    if (!out) return ZL_ERR_INVALID_ARG;
    *out = nullptr;
    if (flags & ~ZL_BUILD_FUSE_LOCAL_CHUNKS) return ZL_ERR_INVALID_ARG;
    if (n_whole < 0 || n_shards < 0 || (n_whole > 0 && !whole) || (n_shards > 0 && !shards)) return ZL_ERR_INVALID_ARG;
    std::vector<InputTask> in;
    in.reserve((size_t)n_whole + n_shards);
    for (int i = 0; i < n_whole; ++i) {
        const zl_whole_desc& w = whole[i];
        if (w.off < 0 || w.len < 0 || (int64_t)w.off + w.len > std::min(total_q, total_kv)) return ZL_ERR_INVALID_ARG;
        in.push_back({w.off, w.len, w.off, w.len, 0, w.head_begin, w.head_count, -1});
    }
    for (int i = 0; i < n_shards; ++i) {
        const zl_shard_desc& d = shards[i];
        const zl_head_range hr = shard_heads ? shard_heads[i] : zl_head_range{0, n_heads};
        in.push_back({d.q_off, d.q_len, d.kv_off, d.kv_len, d.seq_id, hr.head_begin, hr.head_count, i});
    }
    zl_tasks* h = new (std::nothrow) zl_tasks();
    if (!h) return ZL_ERR_INVALID_ARG;
    zl_status st = build_schedule(in, n_shards, total_q, total_kv, n_heads, head_dim, flags, &h->sched);
    if (st != ZL_OK) { delete h; return st; }

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) {
        cudaGetLastError();  // host-only handle: inspection works, launches return ZL_ERR_CUDA
        *out = h;
        return ZL_OK;
    }
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        delete h; return ZL_ERR_CUDA;
    }
    if (prop.major != 10) { delete h; return ZL_ERR_UNSUPPORTED; }
    h->device = dev;
    h->n_sms = prop.multiProcessorCount;

    const Schedule& s = h->sched;
    size_t off = 0;
    const size_t o_tasks = place<Task>(off, s.tasks.size());
    const size_t o_fwd = place<WorkItem>(off, s.fwd_items.size());
    const size_t o_bwd = place<WorkItem>(off, s.bwd_items.size());
    const size_t o_bwd2 = place<WorkItem>(off, s.bwd_pair_items.size());
    const size_t o_mg = place<MergeGroup>(off, s.merge_groups.size());
    const size_t o_mp = place<int32_t>(off, s.merge_parts.size());
    const size_t o_mr = place<int32_t>(off, s.merge_row_prefix.size());
    const size_t o_qg = place<QGroup>(off, s.q_groups.size());
    const size_t o_kg = place<KvGroup>(off, s.kv_groups.size());
    const size_t o_kt = place<int32_t>(off, s.kv_group_tasks.size());
    const size_t o_st = place<int32_t>(off, 2);
    const size_t total = align_up(off, 256);

    std::vector<uint8_t> host(total, 0);
    auto put = [&](size_t at, const void* src, size_t bytes) { if (bytes) std::memcpy(host.data() + at, src, bytes); };
    put(o_tasks, s.tasks.data(), s.tasks.size() * sizeof(Task));
    put(o_fwd, s.fwd_items.data(), s.fwd_items.size() * sizeof(WorkItem));
    put(o_bwd, s.bwd_items.data(), s.bwd_items.size() * sizeof(WorkItem));
    put(o_bwd2, s.bwd_pair_items.data(), s.bwd_pair_items.size() * sizeof(WorkItem));
    put(o_mg, s.merge_groups.data(), s.merge_groups.size() * sizeof(MergeGroup));
    put(o_mp, s.merge_parts.data(), s.merge_parts.size() * sizeof(int32_t));
    put(o_mr, s.merge_row_prefix.data(), s.merge_row_prefix.size() * sizeof(int32_t));
    put(o_qg, s.q_groups.data(), s.q_groups.size() * sizeof(QGroup));
    put(o_kg, s.kv_groups.data(), s.kv_groups.size() * sizeof(KvGroup));
    put(o_kt, s.kv_group_tasks.data(), s.kv_group_tasks.size() * sizeof(int32_t));

    if (cudaMalloc(&h->d_tables, total) != cudaSuccess) { delete h; return ZL_ERR_CUDA; }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // pageable source: the copy is staged before the call returns, so `host` may go away
    if (cudaMemcpyAsync(h->d_tables, host.data(), total, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaStreamSynchronize(cs) != cudaSuccess) {
        cudaFree(h->d_tables); delete h; return ZL_ERR_CUDA;
    }
    h->d_tasks = reinterpret_cast<Task*>(h->d_tables + o_tasks);
    h->d_fwd_items = reinterpret_cast<WorkItem*>(h->d_tables + o_fwd);
    h->d_bwd_items = reinterpret_cast<WorkItem*>(h->d_tables + o_bwd);
    h->d_bwd_pair_items = reinterpret_cast<WorkItem*>(h->d_tables + o_bwd2);
    h->d_merge_groups = reinterpret_cast<MergeGroup*>(h->d_tables + o_mg);
    h->d_merge_parts = reinterpret_cast<int32_t*>(h->d_tables + o_mp);
    h->d_merge_prefix = reinterpret_cast<int32_t*>(h->d_tables + o_mr);
    h->d_q_groups = reinterpret_cast<QGroup*>(h->d_tables + o_qg);
    h->d_kv_groups = reinterpret_cast<KvGroup*>(h->d_tables + o_kg);
    h->d_kv_group_tasks = reinterpret_cast<int32_t*>(h->d_tables + o_kt);
    h->d_status = reinterpret_cast<int32_t*>(h->d_tables + o_st);
    *out = h;
    return ZL_OK;
}

zl_status zl_tasks_get_info(const zl_tasks* t, zl_tasks_info* info) {
    if (!t || !info) return ZL_ERR_INVALID_ARG;
    const Schedule& s = t->sched;
    info->n_tasks = (int32_t)s.tasks.size();
    info->n_merge_groups = (int32_t)s.merge_groups.size();
    info->n_kv_groups = (int32_t)s.kv_groups.size();
    info->n_fwd_items = (int32_t)s.fwd_items.size();
    info->n_bwd_items = (int32_t)s.bwd_items.size();
    info->n_fused_ranges = s.n_fused_ranges;
    info->partial_rows = s.partial_rows;
    info->o_partial_bytes = (size_t)s.partial_rows * s.n_heads * s.head_dim * sizeof(float);
    info->lse_partial_bytes = (size_t)s.partial_rows * s.n_heads * sizeof(float);
    info->bwd_workspace_bytes = s.bwd_workspace_bytes;
    return ZL_OK;
}

zl_status zl_tasks_get_partial_slot(const zl_tasks* t, int32_t shard_idx, int64_t* row_off, int64_t* rows_padded) {
    if (!t || !row_off || !rows_padded) return ZL_ERR_INVALID_ARG;
    if (shard_idx < 0 || shard_idx >= (int32_t)t->sched.shard_to_task.size()) return ZL_ERR_INVALID_ARG;
    *row_off = t->sched.shard_slot_off[shard_idx];
    *rows_padded = t->sched.shard_slot_rows[shard_idx];
    return ZL_OK;
}

static zl_status copy_items(const std::vector<WorkItem>& v, int32_t* items, int32_t capacity, int32_t* count) {
    if (!count) return ZL_ERR_INVALID_ARG;
    *count = (int32_t)v.size();
    if (!items) return ZL_OK;
    if (capacity < (int32_t)v.size()) return ZL_ERR_INVALID_ARG;
    if (!v.empty()) std::memcpy(items, v.data(), v.size() * sizeof(WorkItem));
    return ZL_OK;
}

zl_status zl_tasks_get_fwd_items(const zl_tasks* t, int32_t* items, int32_t capacity, int32_t* count) {
    if (!t) return ZL_ERR_INVALID_ARG;
    return copy_items(t->sched.fwd_items, items, capacity, count);
}

zl_status zl_tasks_get_bwd_items(const zl_tasks* t, int32_t* items, int32_t capacity, int32_t* count) {
    if (!t) return ZL_ERR_INVALID_ARG;
    return copy_items(t->sched.bwd_items, items, capacity, count);
}

void zl_free_tasks(zl_tasks* t) {
    if (!t) return;
    for (int k = 0; k < ZL_K_COUNT; ++k) {
        for (cudaEvent_t e : t->ev_start[k]) cudaEventDestroy(e);
        for (cudaEvent_t e : t->ev_stop[k]) cudaEventDestroy(e);
    }
    if (t->d_tables) cudaFree(t->d_tables);
    delete t;
}

}  // extern "C"

namespace {
// Forward over q, k, v given as token-major views with `in_stride` elements between rows.
// `phase` < 0: the whole work list; otherwise the items of that launch phase only.
zl_status fwd_impl(const zl_tasks* t, int32_t phase, const void* q, const void* k, const void* v, int64_t in_stride,
                   float scale, void* o, float* lse, float* o_partial, float* lse_partial, void* stream) {
    const Schedule& s = t->sched;
    const int32_t n_phases = (int32_t)s.fwd_phase_begin.size() - 1;
    if (phase >= n_phases) return ZL_ERR_INVALID_ARG;
    const int32_t item_begin = phase < 0 ? 0 : s.fwd_phase_begin[phase];
    const int32_t item_end = phase < 0 ? (int32_t)s.fwd_items.size() : s.fwd_phase_begin[phase + 1];
    if (item_end == item_begin) return ZL_OK;
    if (t->device < 0) return ZL_ERR_CUDA;
    if (!on_handle_device(t)) return ZL_ERR_INVALID_ARG;
    if (!q || !k || !v || !o || !lse) return ZL_ERR_INVALID_ARG;
    if (s.partial_rows > 0 && (!o_partial || !lse_partial)) return ZL_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(o_partial))
        return ZL_ERR_INVALID_ARG;
    if (!(scale > 0.f) || !std::isfinite(scale)) return ZL_ERR_INVALID_ARG;

    CUtensorMap tq, tk, tv, to, top;
    const int64_t hd = (int64_t)s.n_heads * s.head_dim;
    if (!make_tmap(&tq, q, s.total_q, s.n_heads, s.head_dim, kTileQ, in_stride) ||
        !make_tmap(&tk, k, s.total_kv, s.n_heads, s.head_dim, kTileKV, in_stride) ||
        !make_tmap(&tv, v, s.total_kv, s.n_heads, s.head_dim, kTileKV, in_stride) ||
        !make_tmap(&to, o, s.total_q, s.n_heads, s.head_dim, kTileQ, hd))
        return ZL_ERR_CUDA;
    // partial results leave through the same kind of store; without shards the map is never used
    if (s.partial_rows > 0 ? !make_tmap_f32_acc(&top, o_partial, s.partial_rows, s.n_heads, s.head_dim, kTileQ)
                           : !make_tmap(&top, o, s.total_q, s.n_heads, s.head_dim, kTileQ, hd))
        return ZL_ERR_CUDA;

    FwdParams p{};
    p.tasks = t->d_tasks;
    p.items = t->d_fwd_items + item_begin;
    p.n_items = item_end - item_begin;
    p.n_heads = s.n_heads;
    p.total_q = s.total_q;
    p.partial_rows = (int32_t)s.partial_rows;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    p.o_partial = o_partial;
    p.lse_partial = lse_partial;
    p.status = t->d_status;
    const int grid = std::min<int>(std::max(2, t->n_sms - t->sm_margin), p.n_items);
    {
        LaunchTimer lt(t, ZL_K_FWD, static_cast<cudaStream_t>(stream));
        if (launch_fwd(s.head_dim, tq, tk, tv, to, top, p, grid, static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return ZL_ERR_CUDA;
    }
    g_launches.fetch_add(1);
    return ZL_OK;
}
}  // namespace

extern "C" {

zl_status zl_coalesced_attn_fwd(const zl_tasks* t, const void* q, const void* k, const void* v, float scale,
                                void* o, float* lse, float* o_partial, float* lse_partial, void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    return fwd_impl(t, -1, q, k, v, (int64_t)t->sched.n_heads * t->sched.head_dim, scale, o, lse, o_partial,
                    lse_partial, stream);
}

zl_status zl_coalesced_attn_fwd_phase(const zl_tasks* t, int32_t phase, const void* q, const void* k, const void* v,
                                      float scale, void* o, float* lse, float* o_partial, float* lse_partial,
                                      void* stream) {
    if (!t || phase < 0) return ZL_ERR_INVALID_ARG;
    return fwd_impl(t, phase, q, k, v, (int64_t)t->sched.n_heads * t->sched.head_dim, scale, o, lse, o_partial,
                    lse_partial, stream);
}

zl_status zl_coalesced_attn_fwd_packed(const zl_tasks* t, const void* qkv, float scale, void* o, float* lse,
                                       float* o_partial, float* lse_partial, void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    const Schedule& s = t->sched;
    if (s.total_q != s.total_kv) return ZL_ERR_INVALID_ARG;  // one token row holds its q, k and v
    if (!qkv) return s.fwd_items.empty() ? ZL_OK : ZL_ERR_INVALID_ARG;
    const int64_t hd = (int64_t)s.n_heads * s.head_dim;
    const __nv_bfloat16* base = static_cast<const __nv_bfloat16*>(qkv);
    return fwd_impl(t, -1, base, base + hd, base + 2 * hd, 3 * hd, scale, o, lse, o_partial, lse_partial, stream);
}

zl_status zl_lse_merge(const zl_tasks* t, const float* o_partial, const float* lse_partial, void* o, float* lse,
                       void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    const Schedule& s = t->sched;
    if (s.merge_groups.empty()) return ZL_OK;
    if (t->device < 0) return ZL_ERR_CUDA;
    if (!on_handle_device(t)) return ZL_ERR_INVALID_ARG;
    if (!o_partial || !lse_partial || !o || !lse) return ZL_ERR_INVALID_ARG;
    if (!aligned16(o_partial) || !aligned16(o)) return ZL_ERR_INVALID_ARG;
    MergeParams p{};
    p.groups = t->d_merge_groups;
    p.parts = t->d_merge_parts;
    p.row_prefix = t->d_merge_prefix;
    p.n_groups = (int32_t)s.merge_groups.size();
    p.n_heads = s.n_heads;
    p.total_q = s.total_q;
    p.partial_rows = (int32_t)s.partial_rows;
    p.o_partial = o_partial;
    p.lse_partial = lse_partial;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    int max_parts = 0;
    for (const MergeGroup& mg : s.merge_groups) max_parts = std::max(max_parts, (int)mg.n_parts);
    {
        LaunchTimer lt(t, ZL_K_MERGE, static_cast<cudaStream_t>(stream));
        if (launch_merge(s.head_dim, p, max_parts, t->n_sms, static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return ZL_ERR_CUDA;
    }
    g_launches.fetch_add(1);
    return ZL_OK;
}

}  // extern "C"

namespace {
// Backward over q, k, v views with `in_stride` elements between token rows and dq, dk, dv views
// with `grad_stride` elements between token rows.
// `phase` < 0: everything in one call.  Otherwise the first phase also clears the dQ accumulator and runs the
// preprocess kernel, every phase runs the main kernel over its own kv groups, the last one also converts dQ.
zl_status bwd_impl(const zl_tasks* t, int32_t phase, const void* q, const void* k, const void* v, int64_t in_stride,
                   const void* o, const float* lse, const void* d_o, float scale, void* dq, void* dk, void* dv,
                   int64_t grad_stride, void* workspace, size_t workspace_bytes, void* stream) {
    const Schedule& s = t->sched;
    if (s.tasks.empty()) return ZL_OK;
    const int32_t n_phases = (int32_t)s.bwd_phase_begin.size() - 1;
    if (phase >= n_phases) return ZL_ERR_INVALID_ARG;
    const bool first = phase <= 0, last = phase < 0 || phase == n_phases - 1;
    if (t->device < 0) return ZL_ERR_CUDA;
    if (!on_handle_device(t)) return ZL_ERR_INVALID_ARG;
    if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv || !workspace) return ZL_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv) || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0)
        return ZL_ERR_INVALID_ARG;
    if (!(scale > 0.f) || !std::isfinite(scale)) return ZL_ERR_INVALID_ARG;
    if (workspace_bytes < s.bwd_workspace_bytes) return ZL_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);

    uint8_t* ws = static_cast<uint8_t*>(workspace);
    CUtensorMap tq, tk, tv, tdo, tdq, tdk, tdv;
    if (!make_tmap_f32_acc(&tdq, ws + s.ws_dq_acc_off, s.q_pad_total, s.n_heads, s.head_dim)) return ZL_ERR_CUDA;
    const int64_t hd = (int64_t)s.n_heads * s.head_dim;
    if (!make_tmap(&tq, q, s.total_q, s.n_heads, s.head_dim, kTileQ, in_stride) ||
        !make_tmap(&tk, k, s.total_kv, s.n_heads, s.head_dim, kTileKV, in_stride) ||
        !make_tmap(&tv, v, s.total_kv, s.n_heads, s.head_dim, kTileKV, in_stride) ||
        !make_tmap(&tdo, d_o, s.total_q, s.n_heads, s.head_dim, kTileQ, hd) ||
        !make_tmap(&tdk, dk, s.total_kv, s.n_heads, s.head_dim, kTileKV, grad_stride) ||
        !make_tmap(&tdv, dv, s.total_kv, s.n_heads, s.head_dim, kTileKV, grad_stride))
        return ZL_ERR_CUDA;

    BwdParams p{};
    p.tasks = t->d_tasks;
    const int32_t it0 = phase < 0 ? 0 : s.bwd_phase_begin[phase];
    const int32_t it1 = phase < 0 ? (int32_t)s.bwd_items.size() : s.bwd_phase_begin[phase + 1];
    p.items = t->d_bwd_items + it0;
    p.kv_groups = t->d_kv_groups;
    p.kv_group_tasks = t->d_kv_group_tasks;
    p.q_groups = t->d_q_groups;
    p.n_items = it1 - it0;
    p.n_q_groups = (int32_t)s.q_groups.size();
    p.n_heads = s.n_heads;
    p.total_q = s.total_q;
    p.q_pad_total = (int32_t)s.q_pad_total;
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.o = static_cast<const __nv_bfloat16*>(o);
    p.d_o = static_cast<const __nv_bfloat16*>(d_o);
    p.lse = lse;
    p.dq = static_cast<__nv_bfloat16*>(dq);
    p.dk = static_cast<__nv_bfloat16*>(dk);
    p.dv = static_cast<__nv_bfloat16*>(dv);
    p.grad_row_stride = grad_stride;
    p.dq_acc = reinterpret_cast<float*>(ws + s.ws_dq_acc_off);
    p.aug = ws + s.ws_aug_off;
    p.status = t->d_status;

    if (first) {
        if (cudaMemsetAsync(p.dq_acc, 0, (size_t)s.q_pad_total * s.n_heads * s.head_dim * sizeof(float), cs) != cudaSuccess)
            return ZL_ERR_CUDA;
        LaunchTimer lt(t, ZL_K_BWD_PRE, cs);
        if (launch_bwd_pre(s.head_dim, p, t->n_sms, cs) != cudaSuccess) return ZL_ERR_CUDA;
        g_launches.fetch_add(1);
    }
    const bool pair = s.head_dim == 128 && (t->bwd_kernel == 2 || (t->bwd_kernel == 0 && kDefaultBwdPair));
    if (p.n_items > 0 && pair) {
        CUtensorMap tq64, tdo64, taug, tdq16, tdk32, tdv32;
        if (!make_tmap_f32_acc(&tdq16, ws + s.ws_dq_acc_off, s.q_pad_total, s.n_heads, s.head_dim, 32, 16) ||
            !make_tmap(&tdk32, dk, s.total_kv, s.n_heads, s.head_dim, 32, grad_stride) ||
            !make_tmap(&tdv32, dv, s.total_kv, s.n_heads, s.head_dim, 32, grad_stride) ||
            !make_tmap(&tq64, q, s.total_q, s.n_heads, s.head_dim, 64, in_stride) ||
            !make_tmap(&tdo64, d_o, s.total_q, s.n_heads, s.head_dim, 64, hd) ||
            !make_tmap_aug_rows(&taug, p.aug, (s.q_pad_total / kTileQ) * s.n_heads))
            return ZL_ERR_CUDA;
        BwdParams pp = p;
        const int32_t pi0 = phase < 0 ? 0 : s.bwd_pair_phase_begin[phase];
        const int32_t pi1 = phase < 0 ? (int32_t)s.bwd_pair_items.size() : s.bwd_pair_phase_begin[phase + 1];
        pp.items = t->d_bwd_pair_items + pi0;
        pp.n_items = pi1 - pi0;
        const int n_clusters = std::min<int>(std::max(2, t->n_sms - t->sm_margin) / 2, pp.n_items);
        LaunchTimer lt(t, ZL_K_BWD_MAIN, cs);
        if (launch_bwd_pair(tq, tq64, tk, tv, tdo, tdo64, tdq16, taug, tdk32, tdv32, pp, n_clusters, cs) != cudaSuccess) return ZL_ERR_CUDA;
        g_launches.fetch_add(1);
    } else if (p.n_items > 0) {
        const int grid = std::min<int>(std::max(2, t->n_sms - t->sm_margin), p.n_items);
        LaunchTimer lt(t, ZL_K_BWD_MAIN, cs);
        if (launch_bwd_main(s.head_dim, tq, tk, tv, tdo, tdq, tdk, tdv, p, grid, cs) != cudaSuccess) return ZL_ERR_CUDA;
        g_launches.fetch_add(1);
    }
    if (last) {
        LaunchTimer lt(t, ZL_K_BWD_POST, cs);
        if (launch_bwd_post(s.head_dim, p, t->n_sms, cs) != cudaSuccess) return ZL_ERR_CUDA;
        g_launches.fetch_add(1);
    }
    return ZL_OK;
}
}  // namespace

extern "C" {

zl_status zl_coalesced_attn_bwd(const zl_tasks* t, const void* q, const void* k, const void* v, const void* o,
                                const float* lse, const void* d_o, float scale, void* dq, void* dk, void* dv,
                                void* workspace, size_t workspace_bytes, void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    const int64_t hd = (int64_t)t->sched.n_heads * t->sched.head_dim;
    return bwd_impl(t, -1, q, k, v, hd, o, lse, d_o, scale, dq, dk, dv, hd, workspace, workspace_bytes, stream);
}

zl_status zl_coalesced_attn_bwd_phase(const zl_tasks* t, int32_t phase, const void* q, const void* k, const void* v,
                                      const void* o, const float* lse, const void* d_o, float scale, void* dq, void* dk,
                                      void* dv, void* workspace, size_t workspace_bytes, void* stream) {
    if (!t || phase < 0) return ZL_ERR_INVALID_ARG;
    const int64_t hd = (int64_t)t->sched.n_heads * t->sched.head_dim;
    return bwd_impl(t, phase, q, k, v, hd, o, lse, d_o, scale, dq, dk, dv, hd, workspace, workspace_bytes, stream);
}

zl_status zl_coalesced_attn_bwd_packed(const zl_tasks* t, const void* qkv, const void* o, const float* lse,
                                       const void* d_o, float scale, void* dqkv, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    const Schedule& s = t->sched;
    if (s.total_q != s.total_kv) return ZL_ERR_INVALID_ARG;
    if (!qkv || !dqkv) return s.tasks.empty() ? ZL_OK : ZL_ERR_INVALID_ARG;
    const int64_t hd = (int64_t)s.n_heads * s.head_dim;
    const __nv_bfloat16* in = static_cast<const __nv_bfloat16*>(qkv);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(dqkv);
    return bwd_impl(t, -1, in, in + hd, in + 2 * hd, 3 * hd, o, lse, d_o, scale, out, out + hd, out + 2 * hd, 3 * hd,
                    workspace, workspace_bytes, stream);
}

// ---------------------------------------------------------------------------------------------
// Backward without a caller-provided workspace: the scratch is a fixed array in the library image.
// In host code `g_noalloc_scratch` is only a handle for the symbol, not a device address; the
// address is looked up once per device and cached.
static __device__ __align__(256) unsigned char g_noalloc_scratch[ZL_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (nullptr on failure).
void* noalloc_scratch_for(int device) {
    if (device < 0 || device >= kMaxDevices) return nullptr;
    if (!g_noalloc_ptr[device]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        g_noalloc_ptr[device] = ptr;
    }
    return g_noalloc_ptr[device];
}
}  // namespace

zl_status zl_coalesced_attn_bwd_noalloc(const zl_tasks* t, const void* q, const void* k, const void* v,
                                        const void* o, const float* lse, const void* d_o, float scale, void* dq,
                                        void* dk, void* dv, void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    if (t->sched.tasks.empty()) return ZL_OK;
    if (t->device < 0) return ZL_ERR_CUDA;
    if (t->timing) return ZL_ERR_INVALID_ARG;  // per-kernel timing creates events: not allocation-free
    if (t->sched.bwd_workspace_bytes > (size_t)ZL_NOALLOC_SCRATCH_BYTES) return ZL_ERR_WORKSPACE;
    if (!on_handle_device(t)) return ZL_ERR_INVALID_ARG;
    void* scratch = noalloc_scratch_for(t->device);
    if (!scratch) return ZL_ERR_CUDA;
    return zl_coalesced_attn_bwd(t, q, k, v, o, lse, d_o, scale, dq, dk, dv, scratch, ZL_NOALLOC_SCRATCH_BYTES, stream);
}

namespace {
// Groups a work list by the phase of each item's unit (stable: the order inside a phase stays) and records
// where each phase begins.
void regroup_by_phase(std::vector<WorkItem>* items, const std::vector<int32_t>& unit_phase, int32_t n_phases,
                      std::vector<int32_t>* begin) {
    std::stable_sort(items->begin(), items->end(),
                     [&](const WorkItem& a, const WorkItem& b) { return unit_phase[a.unit] < unit_phase[b.unit]; });
    begin->assign((size_t)n_phases + 1, 0);
    for (const WorkItem& w : *items) ++(*begin)[(size_t)unit_phase[w.unit] + 1];
    for (int32_t i = 0; i < n_phases; ++i) (*begin)[(size_t)i + 1] += (*begin)[i];
}

// Per-task phases from the caller's per-sequence and per-shard arrays (NULL = phase 0); a task that stands for
// several shards (fused chunks) takes the latest of their phases.
zl_status task_phases(const Schedule& s, const int32_t* whole_phase, const int32_t* shard_phase, int32_t n_phases,
                      std::vector<int32_t>* out) {
    if (n_phases < 1 || n_phases > ZL_MAX_PHASES) return ZL_ERR_INVALID_ARG;
    out->assign(s.tasks.size(), 0);
    for (size_t i = 0; i < s.whole_to_task.size(); ++i) {
        const int32_t ph = whole_phase ? whole_phase[i] : 0;
        if (ph < 0 || ph >= n_phases) return ZL_ERR_INVALID_ARG;
        if (s.whole_to_task[i] >= 0) (*out)[s.whole_to_task[i]] = std::max((*out)[s.whole_to_task[i]], ph);
    }
    for (size_t i = 0; i < s.shard_to_task.size(); ++i) {
        const int32_t ph = shard_phase ? shard_phase[i] : 0;
        if (ph < 0 || ph >= n_phases) return ZL_ERR_INVALID_ARG;
        if (s.shard_to_task[i] >= 0) (*out)[s.shard_to_task[i]] = std::max((*out)[s.shard_to_task[i]], ph);
    }
    return ZL_OK;
}

zl_status upload_items(const zl_tasks* t, WorkItem* dst, const std::vector<WorkItem>& items, cudaStream_t cs) {
    if (t->device < 0 || items.empty()) return ZL_OK;
    if (cudaMemcpyAsync(dst, items.data(), items.size() * sizeof(WorkItem), cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaStreamSynchronize(cs) != cudaSuccess)
        return ZL_ERR_CUDA;
    return ZL_OK;
}
}  // namespace

zl_status zl_set_fwd_phases(zl_tasks* t, const int32_t* whole_phase, const int32_t* shard_phase, int32_t n_phases,
                            void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    if (t->device >= 0 && !on_handle_device(t)) return ZL_ERR_INVALID_ARG;
    Schedule& s = t->sched;
    std::vector<int32_t> ph;
    const zl_status st = task_phases(s, whole_phase, shard_phase, n_phases, &ph);
    if (st != ZL_OK) return st;
    s.fwd_task_phase = ph;
    regroup_by_phase(&s.fwd_items, s.fwd_task_phase, n_phases, &s.fwd_phase_begin);
    return upload_items(t, t->d_fwd_items, s.fwd_items, static_cast<cudaStream_t>(stream));
}

zl_status zl_set_bwd_phases(zl_tasks* t, const int32_t* whole_phase, const int32_t* shard_phase, int32_t n_phases,
                            void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    if (t->device >= 0 && !on_handle_device(t)) return ZL_ERR_INVALID_ARG;
    Schedule& s = t->sched;
    std::vector<int32_t> ph;
    const zl_status st = task_phases(s, whole_phase, shard_phase, n_phases, &ph);
    if (st != ZL_OK) return st;
    // a kv group is finished by one work item, so it runs in the latest phase any of its tasks asks for
    s.bwd_group_phase.assign(s.kv_groups.size(), 0);
    for (size_t g = 0; g < s.kv_groups.size(); ++g)
        for (int32_t j = 0; j < s.kv_groups[g].n_tasks; ++j)
            s.bwd_group_phase[g] = std::max(s.bwd_group_phase[g], ph[s.kv_group_tasks[s.kv_groups[g].task_begin + j]]);
    regroup_by_phase(&s.bwd_items, s.bwd_group_phase, n_phases, &s.bwd_phase_begin);
    regroup_by_phase(&s.bwd_pair_items, s.bwd_group_phase, n_phases, &s.bwd_pair_phase_begin);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const zl_status st1 = upload_items(t, t->d_bwd_items, s.bwd_items, cs);
    if (st1 != ZL_OK) return st1;
    return upload_items(t, t->d_bwd_pair_items, s.bwd_pair_items, cs);
}

zl_status zl_phase_info(const zl_tasks* t, int32_t* n_fwd_phases, int32_t* n_bwd_phases, int32_t* fwd_items_per_phase,
                        int32_t* bwd_items_per_phase) {
    if (!t) return ZL_ERR_INVALID_ARG;
    const Schedule& s = t->sched;
    const int32_t nf = (int32_t)s.fwd_phase_begin.size() - 1, nb = (int32_t)s.bwd_phase_begin.size() - 1;
    if (n_fwd_phases) *n_fwd_phases = nf;
    if (n_bwd_phases) *n_bwd_phases = nb;
    if (fwd_items_per_phase)
        for (int32_t i = 0; i < nf; ++i) fwd_items_per_phase[i] = s.fwd_phase_begin[i + 1] - s.fwd_phase_begin[i];
    if (bwd_items_per_phase)
        for (int32_t i = 0; i < nb; ++i) bwd_items_per_phase[i] = s.bwd_phase_begin[i + 1] - s.bwd_phase_begin[i];
    return ZL_OK;
}

zl_status zl_debug_set_fwd_order(zl_tasks* t, int32_t mode, void* stream) {
    if (!t || mode < 0 || mode > 2) return ZL_ERR_INVALID_ARG;
    Schedule& s = t->sched;
    auto placement_order = [](const WorkItem& a, const WorkItem& b) {
        return std::tie(a.unit, a.head, a.row0) < std::tie(b.unit, b.head, b.row0);
    };
    std::stable_sort(s.fwd_items.begin(), s.fwd_items.end(), placement_order);
    if (mode != 1) {
        std::stable_sort(s.fwd_items.begin(), s.fwd_items.end(), [&](const WorkItem& a, const WorkItem& b) {
            const int32_t ka = s.tasks[a.unit].kv_len, kb = s.tasks[b.unit].kv_len;
            if (ka != kb) return mode == 0 ? ka > kb : ka < kb;
            if (a.rows != b.rows) return mode == 0 ? a.rows > b.rows : a.rows < b.rows;
            return false;
        });
    }
    // the list stays grouped by launch phase
    regroup_by_phase(&s.fwd_items, s.fwd_task_phase, (int32_t)s.fwd_phase_begin.size() - 1, &s.fwd_phase_begin);
    return upload_items(t, t->d_fwd_items, s.fwd_items, static_cast<cudaStream_t>(stream));
}

zl_status zl_set_sm_margin(zl_tasks* t, int32_t n_sms) {
    if (!t || n_sms < 0) return ZL_ERR_INVALID_ARG;
    t->sm_margin = n_sms;
    return ZL_OK;
}

zl_status zl_set_bwd_kernel(zl_tasks* t, int32_t kernel) {
    if (!t || kernel < 0 || kernel > 2) return ZL_ERR_INVALID_ARG;
    if (kernel == 2 && t->sched.head_dim != 128) return ZL_ERR_UNSUPPORTED;
    t->bwd_kernel = kernel;
    return ZL_OK;
}

zl_status zl_selftest_bounded_wait(const zl_tasks* t, int32_t limit_us, void* stream) {
    if (!t) return ZL_ERR_INVALID_ARG;
    if (t->device < 0) return ZL_ERR_CUDA;
    if (!on_handle_device(t)) return ZL_ERR_INVALID_ARG;
    const int32_t us = limit_us < 1 ? 1 : (limit_us > 100000 ? 100000 : limit_us);
    if (launch_wait_selftest(t->d_status, (uint64_t)us * 1000ull, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return ZL_ERR_CUDA;
    g_launches.fetch_add(1);
    return ZL_OK;
}

zl_status zl_set_kernel_timing(zl_tasks* t, int32_t enable) {
    if (!t) return ZL_ERR_INVALID_ARG;
    t->timing = enable != 0;
    return ZL_OK;
}

zl_status zl_get_kernel_timing(zl_tasks* t, float* total_ms, int32_t* launches) {
    if (!t || !total_ms || !launches) return ZL_ERR_INVALID_ARG;
    for (int k = 0; k < ZL_K_COUNT; ++k) { total_ms[k] = 0.f; launches[k] = 0; }
    if (t->device < 0) return ZL_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) return ZL_ERR_CUDA;
    for (int k = 0; k < ZL_K_COUNT; ++k) {
        for (int i = 0; i < t->ev_used[k]; ++i) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, t->ev_start[k][i], t->ev_stop[k][i]) != cudaSuccess) return ZL_ERR_CUDA;
            total_ms[k] += ms;
        }
        launches[k] = t->ev_used[k];
        t->ev_used[k] = 0;
    }
    return ZL_OK;
}

zl_status zl_last_device_status(const zl_tasks* t, int32_t* code, int32_t* where) {
    if (!t || !code || !where) return ZL_ERR_INVALID_ARG;
    *code = ZL_OK; *where = 0;
    if (t->device < 0) return ZL_OK;
    int32_t host[2] = {0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) return ZL_ERR_CUDA;
    if (cudaMemcpy(host, t->d_status, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return ZL_ERR_CUDA;
    *code = host[0]; *where = host[1];
    if (host[0] != 0 && cudaMemset(t->d_status, 0, sizeof(host)) != cudaSuccess) return ZL_ERR_CUDA;
    return ZL_OK;
}

}  // extern "C"
