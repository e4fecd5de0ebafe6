/*
 * zellige.h -- C ABI of the coalesced attention engine for NVIDIA B200 (sm_100a).
 *
 * The engine executes, on one GPU, what the paper's Section IV-D ("Coalesced Attention
 * Engine") assigns to one rank: every whole sequence placed on the rank (packed
 * block-diagonally, never attending across sequences) together with the rank's shards of
 * distributed-attention groups, in ONE launch.  A shard task is one query chunk attending
 * to one K/V chunk; it produces a partial output plus a log-sum-exp, and partial results
 * of the same query chunk are combined by a log-sum-exp merge (exact attention under
 * context parallelism, Sections II-B and IV-A).  The K/V chunks that context parallelism
 * would exchange between ranks are plain local inputs here.
 *
 * Conventions
 *   - Two packed token spaces.  Q-space holds Q, O, dO, dQ and LSE (total_q rows);
 *     KV-space holds K, V, dK, dV (total_kv rows).  Whole sequence i owns rows
 *     [cu_seqlens[i], cu_seqlens[i+1]) of BOTH spaces.  Shard chunks are addressed by the
 *     offsets in their descriptor and must lie at or after cu_seqlens[n_whole].
 *   - Tensors are [tokens, n_heads, head_dim], contiguous, bf16, base 16-byte aligned.
 *     LSE is [n_heads, total_q] fp32: natural log of the sum of exp(scale * q.k).
 *   - Attention is bidirectional: no mask, bias or dropout.  head_dim is 64 or 128.
 *   - All tensor arguments are DEVICE pointers unless marked host.  The caller owns every
 *     tensor, the workspace and the stream; the library allocates only the small tables
 *     inside a zl_tasks handle.
 *   - Every function returns a zl_status; nothing throws, aborts or traps.  Kernels bound
 *     all their waits; a wait that expires records ZL_ERR_TIMEOUT in the handle's device
 *     status word (zl_last_device_status) and the kernel returns normally.
 *   - Outputs land at the input token offsets whatever the internal work order
 *     (Section IV-D: outputs keep the rank-local input order).
 *   - A handle may be in flight on one stream at a time.
 *   - A handle belongs to the device that was current when it was built; every compute entry
 *     point returns ZL_ERR_INVALID_ARG when another device is current.
 *   - Every element of Q, K, V and d_o inside [0, total_q) / [0, total_kv) must be finite,
 *     including rows that no task covers: a ragged last tile is fetched as a whole 128-row
 *     tile, the rows beyond the task are masked by selection (their scores, P and dS become
 *     exactly -inf / 0), but their values still enter the tensor-core products, where
 *     0 * Inf or 0 * NaN would poison the valid rows of that tile.  Finite neighbours of any
 *     magnitude cannot leak.
 */
#ifndef ZELLIGE_H_
#define ZELLIGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ZL_OK = 0,
    ZL_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned pointer, bad ordering of cu_seqlens */
    ZL_ERR_OVERLAP = 2,     /* ranges that partially overlap, duplicates, a shard inside the whole region */
    ZL_ERR_UNSUPPORTED = 3, /* head_dim not in {64,128}, or a device that is not sm_100 */
    ZL_ERR_WORKSPACE = 4,   /* workspace smaller than zl_tasks_info.bwd_workspace_bytes */
    ZL_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed */
    ZL_ERR_TIMEOUT = 6      /* a bounded device-side wait expired (reported by zl_last_device_status) */
} zl_status;

/* One shard task: query rows [q_off, q_off+q_len) of Q-space attend to key rows
 * [kv_off, kv_off+kv_len) of KV-space.  seq_id labels the long sequence the chunks belong
 * to; tasks that share a query range must share seq_id.  Units: tokens. */
typedef struct {
    int32_t q_off, q_len, kv_off, kv_len, seq_id;
} zl_shard_desc;

typedef struct zl_tasks zl_tasks; /* opaque, immutable after zl_build_tasks */

typedef struct {
    int32_t n_tasks;        /* whole sequences + shard tasks with q_len > 0 */
    int32_t n_merge_groups; /* distinct shard query ranges */
    int32_t n_kv_groups;    /* distinct key ranges (backward work units) */
    int32_t n_fwd_items;    /* forward work items (task, head, query block) */
    int32_t n_bwd_items;    /* backward work items (kv group, head, key tile) */
    int64_t partial_rows;   /* rows of o_partial / columns of lse_partial (slots are padded) */
    size_t o_partial_bytes;     /* partial_rows * n_heads * head_dim * 4 */
    size_t lse_partial_bytes;   /* n_heads * partial_rows * 4 */
    size_t bwd_workspace_bytes; /* scratch needed by zl_coalesced_attn_bwd */
    int32_t n_fused_ranges; /* shard query ranges lowered to one final task (zl_build_tasks_ex) */
} zl_tasks_info;

/* zl_build_tasks -- lower a placement into the rank-local schedule (Section IV-D: "lowers
 * the placement into a rank-local schedule and coalesces compatible segments").
 *
 *   cu_seqlens  host, n_whole+1 entries, cu[0]=0, non-decreasing; may be NULL if n_whole=0.
 *   shards      host, n_shards descriptors; may be NULL if n_shards=0.
 *   total_q/kv  rows of the two token spaces.
 *   stream      cudaStream_t (as void*) used for the one small table upload.
 *   out         receives the handle; free with zl_free_tasks.
 *
 * Every whole sequence becomes a task whose result is final after the forward launch.
 * Every shard becomes a task that writes a partial result into a slot of o_partial /
 * lse_partial.  Shard tasks with identical (q_off, q_len) form a merge group; tasks with
 * identical (kv_off, kv_len) form a kv group whose dK/dV contributions are summed.  Work
 * lists are ordered longest-first (by key length, then rows in the block; ties by task,
 * head, block) so that a long video cannot straggle the launch.
 *
 * Validation (host only): any two query ranges must be identical or disjoint, likewise
 * key ranges (ZL_ERR_OVERLAP); shard ranges lie inside the totals and at or after
 * cu_seqlens[n_whole]; within a merge group key ranges are pairwise disjoint and seq_id
 * agrees; duplicate (query range, key range) pairs are rejected.  Zero-length whole
 * sequences and shards with q_len = 0 are accepted and ignored; a shard with kv_len = 0
 * contributes an empty partial (O = 0, LSE = -inf). */
zl_status zl_build_tasks(const int32_t* cu_seqlens, int32_t n_whole,
                         const zl_shard_desc* shards, int32_t n_shards,
                         int32_t total_q, int32_t total_kv, int32_t n_heads, int32_t head_dim,
                         void* stream, zl_tasks** out);

/* zl_build_tasks_ex -- zl_build_tasks with options (flags = 0 is zl_build_tasks).
 *
 * ZL_BUILD_FUSE_LOCAL_CHUNKS: a shard query range whose non-empty key chunks are all on this rank
 * and, sorted by offset, tile one contiguous interval of KV-space is lowered to ONE task over
 * that interval instead of one task per chunk.  It is exact attention over the union (the same
 * result the merge produces, Section II-B), final after the forward launch: such a range has no
 * partial slots (zl_tasks_get_partial_slot reports rows_padded = 0 for its shards), is not a
 * merge group, and its backward work units are the tiles of the whole interval.  Fusion is applied
 * to every such range or to none: it is skipped when a fused interval would partially overlap
 * another key range of the placement (e.g. another query range that uses only some of the
 * chunks).  The paper's engine has no counterpart: it receives remote chunks over a ring or an
 * all-gather; this is the case where the all-gather has already made them contiguous. */
#define ZL_BUILD_FUSE_LOCAL_CHUNKS 1u
zl_status zl_build_tasks_ex(const int32_t* cu_seqlens, int32_t n_whole,
                            const zl_shard_desc* shards, int32_t n_shards,
                            int32_t total_q, int32_t total_kv, int32_t n_heads, int32_t head_dim,
                            uint32_t flags, void* stream, zl_tasks** out);

/* zl_build_tasks_heads -- zl_build_tasks_ex for placements whose tasks cover different HEAD RANGES
 * (Section IV-D, second coalescing mode: sequences under Ulysses parallelism hold all their tokens
 * for n_heads / h of the heads, are batched with one QKV-packed all-to-all and run as one
 * block-diagonal attention call; Table II, configuration (1, h, 1)).  Such tasks share one launch
 * and one set of [tokens, n_heads, head_dim] buffers with tasks over all heads.
 *
 *   whole        host, n_whole descriptors: a sequence owning rows [off, off+len) of both token
 *                spaces for heads [head_begin, head_begin+head_count).  Final after the forward
 *                launch.  Unlike cu_seqlens, two whole sequences may own the same rows when their
 *                head ranges are disjoint (two Ulysses sequences packed side by side in the head
 *                dimension).  len = 0 is ignored.
 *   shards       as in zl_build_tasks; shard_heads (host, n_shards entries, or NULL = all heads)
 *                gives each shard's head range.  Shards lie at or after the end of the last whole
 *                sequence.
 * Validation, head by head: among the tasks that cover a head, query ranges are pairwise identical
 * or disjoint and so are key ranges; tasks with an identical query range, or an identical key
 * range, must have the same head range (ZL_ERR_OVERLAP otherwise).  Head ranges must satisfy
 * 0 <= head_begin, 1 <= head_count, head_begin + head_count <= n_heads (ZL_ERR_INVALID_ARG).
 * Merge groups, kv groups and the dQ accumulation units are formed per (range, head range); work
 * items exist only for the heads of their task, and every (row, head) of every output that no
 * task covers is left untouched.  Scratch and partial slots are sized for n_heads heads per row
 * whatever the task's head count.
 * zl_build_tasks_ex(cu_seqlens, ...) equals this call with whole[i] = (cu[i], cu[i+1]-cu[i], 0, n_heads). */
typedef struct { int32_t off, len, head_begin, head_count; } zl_whole_desc;
typedef struct { int32_t head_begin, head_count; } zl_head_range;
zl_status zl_build_tasks_heads(const zl_whole_desc* whole, int32_t n_whole,
                               const zl_shard_desc* shards, const zl_head_range* shard_heads, int32_t n_shards,
                               int32_t total_q, int32_t total_kv, int32_t n_heads, int32_t head_dim,
                               uint32_t flags, void* stream, zl_tasks** out);

zl_status zl_tasks_get_info(const zl_tasks* tasks, zl_tasks_info* info);

/* Slot of shard `shard_idx` (index into the `shards` array given to zl_build_tasks) inside
 * o_partial / lse_partial: rows [row_off, row_off + q_len) hold the task's partial result,
 * rows_padded >= q_len is the slot size.  Shards with q_len = 0 report rows_padded = 0. */
zl_status zl_tasks_get_partial_slot(const zl_tasks* tasks, int32_t shard_idx,
                                    int64_t* row_off, int64_t* rows_padded);

/* Host copies of the work lists, for inspection and tests.  Tasks are numbered in the order: whole
 * sequences with len > 0, then shards with q_len > 0 (the shards of a fused range share one task).
 * Each forward item is 4 int32:
 * (task, head, first query row of the block relative to the task, rows in the block); each
 * backward item is 4 int32: (kv group, head, first key row relative to the group, rows).
 * `items` may be NULL to query the count only. */
zl_status zl_tasks_get_fwd_items(const zl_tasks* tasks, int32_t* items, int32_t capacity, int32_t* count);
zl_status zl_tasks_get_bwd_items(const zl_tasks* tasks, int32_t* items, int32_t capacity, int32_t* count);

void zl_free_tasks(zl_tasks* tasks);

/* Stream behaviour of the compute entry points (zl_coalesced_attn_fwd / _fwd_packed, zl_lse_merge,
 * zl_coalesced_attn_bwd / _bwd_packed): each only enqueues kernels (and, for the backward, one memset)
 * on `stream`; tensor maps are encoded on the host at call time and passed by value.  They do not
 * synchronise, so a whole step can be captured in a CUDA graph and replayed (the captured tensor
 * addresses are baked in); make the first call on a handle's device outside the capture.
 * zl_last_device_status, zl_get_kernel_timing and enabled kernel timing are not capturable. */

/* zl_coalesced_attn_fwd -- one persistent launch over the whole work list (Section IV-D:
 * whole sequences packed into one block-diagonal attention call, shards run beside them).
 *
 *   q            [total_q, H, d] bf16        k, v  [total_kv, H, d] bf16
 *   scale        multiplies q.k before the softmax (1/sqrt(d) in every named workload)
 *   o            [total_q, H, d] bf16; rows of whole sequences are final on return of the
 *                launch, rows of shard query ranges are untouched until zl_lse_merge
 *   lse          [H, total_q] fp32, same rule
 *   o_partial    [partial_rows, H, d] fp32: per shard task softmax(S_t) V_t, i.e.
 *                normalised within the task's own K/V chunk (unnormalised with respect to
 *                the union of chunks); may be NULL when there are no shards
 *   lse_partial  [H, partial_rows] fp32: per shard task log-sum-exp over its chunk
 *
 * Asynchronous on `stream`.  Scores between tokens of different tasks are never formed;
 * masked tail scores are selected to -inf, never multiplied.  Inputs must be finite. */
zl_status zl_coalesced_attn_fwd(const zl_tasks* tasks, const void* q, const void* k, const void* v,
                                float scale, void* o, float* lse,
                                float* o_partial, float* lse_partial, void* stream);

/* zl_coalesced_attn_fwd_packed -- the same launch for QKV-packed input (Section IV-D batches Ulysses
 * sequences through one QKV-packed all-to-all; a fused QKV projection produces the same layout):
 *   qkv  [T, 3, H, d] bf16, row t = q_t | k_t | v_t.  Needs total_q == total_kv == T (query row i
 *        and key row i are the same token); ZL_ERR_INVALID_ARG otherwise.
 * Everything else as zl_coalesced_attn_fwd; results are bit-identical to passing the three
 * tensors separately (the tiles are fetched through strided tensor maps, nothing is repacked). */
zl_status zl_coalesced_attn_fwd_packed(const zl_tasks* tasks, const void* qkv, float scale, void* o, float* lse,
                                       float* o_partial, float* lse_partial, void* stream);

/* zl_lse_merge -- combine the partial results of every merge group (the accumulation step
 * of ring / all-gather context parallelism, Section II-B):
 *     LSE = log sum_t exp(LSE_t),   O = sum_t exp(LSE_t - LSE) * O_t
 * summed in ascending shard order (bit-deterministic).  Writes final bf16 O and fp32 LSE at
 * the group's query rows.  Rows whose parts are all empty get O = 0, LSE = -inf. */
zl_status zl_lse_merge(const zl_tasks* tasks, const float* o_partial, const float* lse_partial,
                       void* o, float* lse, void* stream);

/* zl_coalesced_attn_bwd -- gradients of every task in one call, for dL/dO = d_o and no
 * gradient through LSE.  With P = exp(scale*QK^T - LSE) recomputed from the FINAL
 * (merged) LSE and D_i = sum_c dO_ic O_ic from the FINAL O:
 *     dV = P^T dO,  dS = P o (dO V^T - D),  dQ = scale * dS K,  dK = scale * dS^T Q.
 * dQ is summed over tasks sharing a query range, dK/dV over tasks sharing a key range
 * (on a context-parallel rank that is the contribution of the local queries only).
 *
 *   o, lse       final forward results;  d_o [total_q, H, d] bf16
 *   dq           [total_q, H, d] bf16;   dk, dv [total_kv, H, d] bf16.  Rows covered by at
 *                least one task are overwritten; rows covered by none are left untouched.
 *   workspace    device scratch of at least zl_tasks_info.bwd_workspace_bytes, 256-byte
 *                aligned; contents need not be initialised and are clobbered.
 * Asynchronous on `stream` (three launches: preprocess, main, dQ conversion). */
zl_status zl_coalesced_attn_bwd(const zl_tasks* tasks, const void* q, const void* k, const void* v,
                                const void* o, const float* lse, const void* d_o, float scale,
                                void* dq, void* dk, void* dv,
                                void* workspace, size_t workspace_bytes, void* stream);

/* zl_coalesced_attn_bwd_packed -- the backward for QKV-packed tensors: reads qkv [T, 3, H, d] bf16 and
 * writes dqkv [T, 3, H, d] bf16 (row t = dq_t | dk_t | dv_t); o, lse, d_o, workspace as above.
 * Needs total_q == total_kv.  Gradients equal those of zl_coalesced_attn_bwd element for element
 * (dQ up to the order of the fp32 reduce-adds). */
zl_status zl_coalesced_attn_bwd_packed(const zl_tasks* tasks, const void* qkv, const void* o, const float* lse,
                                       const void* d_o, float scale, void* dqkv,
                                       void* workspace, size_t workspace_bytes, void* stream);

/* Launch phases -- running the tasks of a handle in several launches, in the order their inputs arrive.
 *
 * Section IV-D runs the attention of a context-parallel rank under its collectives: the tasks whose K/V are
 * already local start while the remaining K/V chunks are still on their way (all-gather, or one chunk per
 * ring step), and in the backward the gradients of remote K/V chunks leave for their owners while the local
 * ones are still being computed.  A phase is the unit of that overlap: the caller assigns every whole sequence
 * and every shard a phase number, launches phase p when its inputs are there, and runs the merge once after
 * the last forward phase.
 *
 * zl_set_fwd_phases: `whole_phase` [n_seqs] and `shard_phase` [n_shards] (host arrays; NULL = all zero) give
 * the phase, 0 <= phase < n_phases <= ZL_MAX_PHASES, of every sequence / shard in the order they were passed
 * to zl_build_tasks*.  The forward work list is regrouped by phase (longest-first inside each phase) and
 * uploaded (the call synchronises `stream`).  A shard query range that the builder fused into one task
 * (ZL_BUILD_FUSE_LOCAL_CHUNKS) runs in the latest phase of its shards.  zl_coalesced_attn_fwd still runs the
 * whole list in one launch; zl_coalesced_attn_fwd_phase runs the tasks of one phase: arguments, outputs and
 * errors as zl_coalesced_attn_fwd, plus ZL_ERR_INVALID_ARG for a phase the handle does not have.  K/V rows of
 * tasks of later phases are not used, so they may still be in flight -- but a ragged last tile of a chunk is
 * loaded whole, so the rows that follow a chunk must hold finite values at all times (zero the buffers once;
 * a row that is half old and half new is still finite); O/LSE rows and partial slots of tasks of other phases
 * are not written.  Phases may run in any order and on different streams; zl_lse_merge must
 * follow all of them.  Results are bit-identical to the single launch.
 *
 * zl_set_bwd_phases: the same arrays for the backward.  The unit of the backward is the kv group (all tasks
 * that share a key range: one work item finishes that range's dK and dV), which runs in the latest phase any of
 * its tasks asks for.  zl_coalesced_attn_bwd_phase must be called for phase 0, 1, ..., n_phases-1 in this order
 * on one stream with the same arguments: phase 0 first clears the dQ accumulator and forms D and -LSE/scale
 * for all rows, every phase runs the main kernel over its kv groups, the last phase converts dQ.  After
 * phase p has finished, the dK and dV rows of the kv groups of phases <= p are final (their reduce-scatter may
 * start); dQ is final after the last phase.  dK and dV are bit-identical to zl_coalesced_attn_bwd, dQ up to the
 * order of the fp32 reduce-adds.
 *
 * zl_phase_info reports the number of phases and the work items per phase (arrays of ZL_MAX_PHASES entries,
 * any pointer may be NULL).  A handle starts with one phase per direction. */
#define ZL_MAX_PHASES 64
zl_status zl_set_fwd_phases(zl_tasks* tasks, const int32_t* whole_phase, const int32_t* shard_phase, int32_t n_phases,
                            void* stream);
zl_status zl_set_bwd_phases(zl_tasks* tasks, const int32_t* whole_phase, const int32_t* shard_phase, int32_t n_phases,
                            void* stream);
zl_status zl_coalesced_attn_fwd_phase(const zl_tasks* tasks, int32_t phase, const void* q, const void* k, const void* v,
                                      float scale, void* o, float* lse, float* o_partial, float* lse_partial,
                                      void* stream);
zl_status zl_coalesced_attn_bwd_phase(const zl_tasks* tasks, int32_t phase, const void* q, const void* k, const void* v,
                                      const void* o, const float* lse, const void* d_o, float scale,
                                      void* dq, void* dk, void* dv, void* workspace, size_t workspace_bytes, void* stream);
zl_status zl_phase_info(const zl_tasks* tasks, int32_t* n_fwd_phases, int32_t* n_bwd_phases,
                        int32_t* fwd_items_per_phase /* [ZL_MAX_PHASES] */, int32_t* bwd_items_per_phase /* [ZL_MAX_PHASES] */);

/* zl_coalesced_attn_bwd_noalloc -- the backward for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a convenience of the library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a stream-ordered region
 * owned by another allocator, in a plugin whose host forbids allocations after initialisation, or
 * on a latency-critical path where an allocator call (and the implicit synchronisation it may
 * bring) is not acceptable -- and that therefore has no workspace buffer to hand to
 * zl_coalesced_attn_bwd.  This entry point takes the same inputs and outputs but no workspace:
 * the scratch (fp32 dQ accumulator and the per-tile LSE/D tiles) lives in a fixed device array
 * of ZL_NOALLOC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the
 * library reserves that much memory until the process exits.
 *
 *   - Placements whose zl_tasks_info.bwd_workspace_bytes exceeds ZL_NOALLOC_SCRATCH_BYTES are
 *     rejected with ZL_ERR_WORKSPACE; nothing is launched.
 *   - The call itself performs no cudaMalloc / cudaFree and calls no allocating routine.  The task
 *     handle must have been built beforehand (zl_build_tasks allocates its small tables), and
 *     kernel timing must be off on the handle (ZL_ERR_INVALID_ARG otherwise: timing creates events).
 *   - The first call on each device looks up the device address of the scratch array; make that
 *     first call outside any stream capture.  The first launch of each kernel on a device may also
 *     load its code, so a caller that needs a strictly allocation-free region should have run one
 *     backward (this entry point or zl_coalesced_attn_bwd) on the device before entering it.
 *   - All calls on a device share the one array and it keeps whatever the last call left in it.
 *     The part that must start at zero (the dQ accumulator) is cleared on the stream by every
 *     call.  Two calls that overlap on the GPU (different streams, or different handles at the
 *     same time) race on the array and produce garbage: serialise them.
 * Results equal those of zl_coalesced_attn_bwd (dK, dV bit for bit; dQ up to the order of the
 * fp32 reduce-adds). */
#define ZL_NOALLOC_SCRATCH_BYTES (64u * 1024u * 1024u)
zl_status zl_coalesced_attn_bwd_noalloc(const zl_tasks* tasks, const void* q, const void* k, const void* v,
                                        const void* o, const float* lse, const void* d_o, float scale,
                                        void* dq, void* dk, void* dv, void* stream);

/* Synchronises the handle's device and reads the device status word written by the
 * kernels: code is ZL_OK or ZL_ERR_TIMEOUT, `where` identifies the wait that expired
 * (kernel id * 1000 + site).  Resets the word to ZL_OK. */
zl_status zl_last_device_status(const zl_tasks* tasks, int32_t* code, int32_t* where);

/* Optional per-kernel device timing, for measurement only (no paper counterpart).  While
 * enabled, every launch made through this handle is bracketed by CUDA events on the launch
 * stream (at most 1024 launches per kernel between two reads; further ones are not timed).
 * zl_get_kernel_timing synchronises the device, returns the summed elapsed milliseconds
 * and the number of timed launches per kernel id, and clears the counters. */
typedef enum {
    ZL_K_FWD = 0, ZL_K_MERGE = 1, ZL_K_BWD_PRE = 2, ZL_K_BWD_MAIN = 3, ZL_K_BWD_POST = 4, ZL_K_COUNT = 5
} zl_kernel_id;
zl_status zl_set_kernel_timing(zl_tasks* tasks, int32_t enable);
zl_status zl_get_kernel_timing(zl_tasks* tasks, float* total_ms /* [ZL_K_COUNT] */,
                               int32_t* launches /* [ZL_K_COUNT] */);

/* Measurement / diagnosis aids (no paper counterpart).
 *
 * zl_debug_set_fwd_order re-sorts the handle's forward work list and uploads it: 0 = longest-first
 * (the default built by zl_build_tasks), 1 = placement order (task, head, block), 2 = shortest-first.
 * Results never depend on the order; it exists to measure what longest-first ordering buys.
 *
 * zl_selftest_bounded_wait launches a one-CTA kernel that waits, with the same bounded wait the
 * attention kernels use, on an mbarrier nobody ever arrives on, with a limit of `limit_us`
 * microseconds (clamped to [1, 100000]).  The wait must expire: the kernel then records
 * ZL_ERR_TIMEOUT in the handle's device status word and returns normally, which
 * zl_last_device_status reports.  Nothing hangs and nothing faults. */
zl_status zl_debug_set_fwd_order(zl_tasks* tasks, int32_t mode, void* stream);
/* zl_set_bwd_kernel chooses the main kernel of zl_coalesced_attn_bwd for this handle: 0 = the library's
 * default (pairs at head_dim 128, one CTA otherwise), 1 = one CTA per 128-row key tile, 2 = pairs of CTAs (tcgen05 cta_group::2) that own two
 * neighbouring key tiles, share every B operand and sum dQ over 256 keys before it is reduced
 * (head_dim 128 only: ZL_ERR_UNSUPPORTED otherwise).  Results agree within the gradient tolerance; dK
 * and dV of the two kernels may differ in the last bit (different accumulation order). */
zl_status zl_set_bwd_kernel(zl_tasks* tasks, int32_t kernel);
/* zl_set_sm_margin: the persistent kernels (forward, backward main) of this handle leave `n_sms` of the GPU's SMs
 * without a CTA (at least two SMs are always used), so that kernels of another stream -- the collectives that
 * run beside a launch phase -- find a free SM instead of waiting for the launch to end.  0 (the default) uses
 * every SM.  Results do not depend on it.  (No paper counterpart.) */
zl_status zl_set_sm_margin(zl_tasks* tasks, int32_t n_sms);
zl_status zl_selftest_bounded_wait(const zl_tasks* tasks, int32_t limit_us, void* stream);

const char* zl_status_str(zl_status s);

/* Number of this library's kernel launches enqueued since load (all handles). */
int64_t zl_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ZELLIGE_H_ */
