/*
 * pulseinfer.h - C ABI of the B200 (sm_100a) decode recall path of sparse KV-cache
 * offloading:  score -> top-k select -> miss diff -> gather-scatter recall ->
 * sparse GQA decode attention, one call per step, per layer, for a whole batch.
 *
 * Conventions (all entry points)
 *   - "dev" pointers are device memory, "pinned" pointers are page-locked host
 *     memory that the GPU can address (cudaHostAlloc / cudaHostRegister), "host"
 *     pointers are ordinary host memory.  The caller owns every buffer; the library
 *     allocates only the small scratch held by pi_ctx.  Buffers must stay alive
 *     until the stream has drained.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work and return;
 *     none of the four path calls synchronises the host.
 *   - All per-layer arrays are passed by their per-layer base; `layer` only selects
 *     the retrieval head solo_head[layer].
 *   - Return value: PI_OK or a negative PI_ERR_* code; nothing is launched when an
 *     argument check fails.  Problems only the device can see (an index out of
 *     range, a list longer than its capacity, a bounded wait that ran out, a pool
 *     with too few evictable slots) set a sticky status word read by pi_get_status;
 *     the offending access is skipped, never trapped.
 *   - Shapes use: Hq query heads, Hkv KV heads, G = Hq/Hkv, D = head_dim = 128,
 *     B = block_tokens, K = budget_blocks, C = pool_slots, NB = max_blocks.
 *     frag_bytes = B*D*2*2 (K and V of one KV head of one block; 8 KB at B = 16),
 *     block_bytes = Hkv*frag_bytes.  bf16 everywhere for q, K, V, digests, out.
 *   - Layout of one block, in the host store and in the pool alike:
 *     [Hkv][2 = K,V][B][D] bf16, so one (block, head) fragment is contiguous.
 */
#ifndef PULSEINFER_H
#define PULSEINFER_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PI_OK                   0
#define PI_ERR_INVALID_ARG     (-1)
#define PI_ERR_BAD_ALIGN       (-2)   /* a pointer is not 16-byte aligned            */
#define PI_ERR_UNSUPPORTED_DIM (-3)
#define PI_ERR_POOL_TOO_SMALL  (-4)   /* fewer evictable slots than misses           */
#define PI_ERR_NOT_PINNED      (-5)   /* host KV store is not GPU-addressable        */
#define PI_ERR_CUDA            (-6)   /* a CUDA runtime call failed                  */
#define PI_ERR_TIMEOUT         (-7)   /* a bounded device-side wait ran out          */
#define PI_ERR_INDEX_RANGE     (-8)   /* a block / slot index read from a list is out of range */
#define PI_ERR_CAPACITY        (-9)   /* a count read from device memory exceeds its capacity  */
#define PI_ERR_STATIC_LIMIT   (-10)  /* batch or block count beyond the fixed scratch of pi_score_select_noalloc */

typedef struct pi_ctx pi_ctx;

typedef struct {
    int32_t n_layers;
    int32_t n_q_heads, n_kv_heads, head_dim;  /* head_dim must be 128; Hkv a power of two <= 16 (the attention calls: <= 8); Hq % Hkv == 0; G <= 16 */
    int32_t block_tokens;                     /* 16, 32 or 64                                      */
    int32_t budget_blocks;                    /* K: sink + local + middle blocks per (seq, layer) */
    int32_t n_sink_blocks, n_local_blocks;    /* always-resident, always-selected prefix / suffix */
    int32_t pool_slots;                       /* C per (seq, layer); C >= K                       */
    int32_t max_batch, max_blocks;            /* capacities: batch <= max_batch, NB = max_blocks  */
    int32_t recall_ctas;                      /* CTAs per recall launch, 0 = default (5)           */
    int32_t attn_ctas;                        /* CTAs of the attention kernel, 0 = default (#SMs - 20) */
    int32_t attn_mode;                        /* split of the attention work: 0 = chosen per call, 1 = flat (all KV heads of a block
                                                 per tile, sequences cut across CTAs, partials merged by a second kernel),
                                                 2 = head-major (one (sequence, KV head) per CTA, merged inside the CTA) */
    int32_t wait_limit_us;                    /* bound of every device-side wait of the attention kernel in microseconds,
                                                 0 = default (2 000 000); when it runs out the kernel gives up, returns and
                                                 the status word says PI_ERR_TIMEOUT (stage 4: CTA, first unit, last unit) */
    int32_t test_hold_producer;               /* TEST ONLY, keep 0: when 1 the loads of every CTA's last tile are never
                                                 issued, so that the bounded wait above can be seen to run out */
    const int32_t* solo_head;                 /* host [n_layers]: retrieval KV head per layer (copied) */
} pi_config;

/* One transfer of the recall list: n_units consecutive units of the host store
 * starting at src_unit go to n_units consecutive units of the pool starting at
 * dst_unit.  A unit is `unit_bytes` long (a whole block for the shared selection,
 * one (block, head) fragment for per-head lists); indices are relative to the
 * sequence's base.  units_before = units of the earlier extents of the same list. */
typedef struct {
    int32_t src_unit, dst_unit, n_units, units_before;
} pi_extent;

/* Create / destroy the context (device scratch for scores, split-K partials and
 * completion counters; a pinned status word).  Uses the current CUDA device. */
int pi_create(const pi_config* cfg, pi_ctx** out);
int pi_destroy(pi_ctx* ctx);

/* Step 1+2 of the offloading workflow (Sec. 2.2, sparse selection) with the shared
 * single-head selection of Sec. 4.4.1: score every block of every sequence against
 * the digest of the layer's retrieval head, keep the sink and local blocks, add the
 * K - n_sink - n_local best middle blocks (ties to the lower block index).
 *   q_dev       [batch][Hq][D] bf16           (only the G heads of solo_head[layer] are read)
 *   digest_dev  [batch][NB][2][D] bf16        row 0 = channel-wise min, row 1 = max of the block's keys
 *   ctx_len_dev [batch] int32                 tokens per sequence; n_blocks = ceil(ctx/B) <= NB
 *   sel_blocks_dev [batch][K] int32 (out)     ascending block indices, -1 padded
 *   sel_count_dev  [batch] int32 (out)
 *   scores_dev  [batch][NB] float (out) or NULL: score = sum_d Q+[d]*max[d] + Q-[d]*min[d]
 *               with Q+/- the sums of the positive / negative parts of the group's queries. */
int pi_score_select(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* digest_dev,
                    const int32_t* ctx_len_dev, int32_t* sel_blocks_dev, int32_t* sel_count_dev,
                    float* scores_dev, void* stream);

/* pi_score_select for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this exists for the library's users.)  Some code runs where cudaMalloc is off
 * limits: a plug-in inside a serving engine that hands out all device memory itself, a callback
 * on a latency-critical path where an allocation could stall or fail, a process whose memory
 * pool is already fully committed.  Such a caller cannot call pi_create, which allocates the
 * score buffer and the per-sequence tickets.  This entry point needs no context: it computes the
 * same selection as pi_score_select (same kernel, same results bit for bit) and keeps that
 * scratch in a fixed array inside the library image instead.
 *   Limits: batch <= 64 and max_blocks <= 8192, else PI_ERR_STATIC_LIMIT and nothing runs.  The
 *   array takes 2 MiB + 512 B on every GPU that loads the library, until the process exits.
 *   The call allocates nothing and frees nothing (no cudaMalloc / cudaFree, no library routine
 *   that allocates); it enqueues two small memsets and the kernel on `stream` and returns.
 *   The first call on each device also looks up the array's device address, with that device
 *   current; make that first call outside any stream capture.
 *   All calls on a device share the one array, and it keeps the previous call's contents; the
 *   words that must start at zero are cleared on `stream` before the kernel.  Two calls whose
 *   kernels can overlap on the GPU (different streams, no dependency) race on it: order them.
 *   Model shape and budget come as plain arguments (meaning as in pi_config); solo_head is the
 *   retrieval KV head of this layer.  q, digest, ctx_len, sel_blocks, sel_count: as pi_score_select.
 *   status_dev: NULL, or device int32[8] that receives what pi_get_status would report for this
 *   call ([0] code, [1] stage, [2..4] coordinates; [7] is used internally); cleared on `stream`. */
int pi_score_select_noalloc(int batch, int n_q_heads, int n_kv_heads, int block_tokens,
                            int budget_blocks, int n_sink_blocks, int n_local_blocks, int max_blocks,
                            int solo_head, const void* q_dev, const void* digest_dev,
                            const int32_t* ctx_len_dev, int32_t* sel_blocks_dev, int32_t* sel_count_dev,
                            int32_t* status_dev, void* stream);

/* The two comparison strategies of the paper's selection study (Sec. 4.4.1), for the
 * fragmentation story end to end.  Both read digests of EVERY KV head,
 *   digest_all_dev [batch][NB][Hkv][2][D] bf16 (pi_build_digests_all),
 * and score a KV head with the queries of its own group.
 *   PI_SELECT_AVERAGE   the per-head scores are summed (a sum ranks like the paper's average) and
 *                       one top-k is shared by all heads: sel_blocks_dev [batch][K], sel_count_dev [batch]
 *   PI_SELECT_HEADWISE  every KV head selects for itself: sel_blocks_dev [batch][Hkv][K],
 *                       sel_count_dev [batch][Hkv]; needs max_batch >= batch*Hkv
 * scores_dev: NULL or float [rows][NB], rows = batch or batch*Hkv.  Everything else as pi_score_select.
 * Per-head selections go through pi_diff_misses with batch*Hkv rows (tables, slot arrays and a
 * ctx_len array of that many rows) and through pi_recall_gather_scatter with lists_per_seq = Hkv,
 * unit_bytes = frag_bytes, unit_stride_bytes = block_bytes, list_offset_bytes = frag_bytes: head h
 * of slot s then holds the fragment of whatever block head h selected; attention over such
 * per-head selections is pi_sparse_decode_attn_headwise. */
#define PI_SELECT_AVERAGE  1
#define PI_SELECT_HEADWISE 2
int pi_score_select_strategy(pi_ctx* ctx, int strategy, int layer, int batch, const void* q_dev,
                             const void* digest_all_dev, const int32_t* ctx_len_dev,
                             int32_t* sel_blocks_dev, int32_t* sel_count_dev, float* scores_dev, void* stream);

/* Step 2 of the workflow (Sec. 2.2): B_recall = B_topk \ B_gpu against the
 * device-resident block table, victim choice (least recently selected slot, ties to
 * the lower slot; sink / local / selected blocks are never evicted), table update,
 * and the recall list with adjacent (block, slot) pairs merged into extents.
 *   step             decode step counter, >= 1, written as the stamp of every selected slot
 *   block_table_dev  [batch][NB] int32 (in/out)  slot of each block or -1
 *   slot_block_dev   [batch][C] int32 (in/out)   block held by each slot or -1
 *   slot_stamp_dev   [batch][C] uint32 (in/out)  step the slot was last selected (0 = never)
 *   sel_slots_dev    [batch][K] int32 (out)      pool slot of every selected block, -1 padded
 *   recall_list_dev  [batch][K] pi_extent (out)  units are whole blocks, ascending src_unit
 *   recall_count_dev [batch] int32 (out)         extents per sequence
 * A sequence with too few evictable slots keeps its tables, gets recall count 0 and
 * -1 for its missing blocks in sel_slots, and sets PI_ERR_POOL_TOO_SMALL in the status. */
int pi_diff_misses(pi_ctx* ctx, int layer, int batch, uint32_t step, const int32_t* ctx_len_dev,
                   const int32_t* sel_blocks_dev, const int32_t* sel_count_dev,
                   int32_t* block_table_dev, int32_t* slot_block_dev, uint32_t* slot_stamp_dev,
                   int32_t* sel_slots_dev, pi_extent* recall_list_dev, int32_t* recall_count_dev,
                   void* stream);

/* Steps 1 and 2 of the workflow (Sec. 2.2: sparse selection, then B_recall = B_topk \ B_gpu) in ONE launch:
 * pi_score_select followed by pi_diff_misses with the same arguments and the same results, bit for bit
 * (selection, slots, tables, stamps, recall list).  The CTA that selects for a sequence diffs its selection
 * while it is still in shared memory, and what the diff needs besides the selection is fetched while the
 * digests stream in, so the launch and the global round trips between the two steps disappear.
 * Arguments as in the two calls; scores_dev may be NULL.  The _devstep form reads the step number
 * from device memory like pi_diff_misses_devstep. */
int pi_score_select_diff(pi_ctx* ctx, int layer, int batch, uint32_t step, const void* q_dev, const void* digest_dev,
                         const int32_t* ctx_len_dev, int32_t* sel_blocks_dev, int32_t* sel_count_dev, float* scores_dev,
                         int32_t* block_table_dev, int32_t* slot_block_dev, uint32_t* slot_stamp_dev,
                         int32_t* sel_slots_dev, pi_extent* recall_list_dev, int32_t* recall_count_dev, void* stream);
int pi_score_select_diff_devstep(pi_ctx* ctx, int layer, int batch, const uint32_t* step_dev, const void* q_dev,
                                 const void* digest_dev, const int32_t* ctx_len_dev, int32_t* sel_blocks_dev,
                                 int32_t* sel_count_dev, float* scores_dev, int32_t* block_table_dev,
                                 int32_t* slot_block_dev, uint32_t* slot_stamp_dev, int32_t* sel_slots_dev,
                                 pi_extent* recall_list_dev, int32_t* recall_count_dev, void* stream);

/* pi_diff_misses with the step number read from device memory when the kernel runs (one uint32, > 0), so
 * that a CUDA graph holding the call can be replayed for later steps: the caller advances *step_dev
 * between replays (in the graph or outside).  The paper has no counterpart. */
int pi_diff_misses_devstep(pi_ctx* ctx, int layer, int batch, const uint32_t* step_dev,
                           const int32_t* ctx_len_dev, const int32_t* sel_blocks_dev,
                           const int32_t* sel_count_dev, int32_t* block_table_dev, int32_t* slot_block_dev,
                           uint32_t* slot_stamp_dev, int32_t* sel_slots_dev, pi_extent* recall_list_dev,
                           int32_t* recall_count_dev, void* stream);

/* Step 3 of the workflow (Sec. 2.2; Sec. 4.4.2 gather-scatter transfer): copy every
 * extent of every list from the pinned host store into the HBM pool, byte for byte.
 * The GPU pulls the data itself with wide loads; counts and lists are read from
 * device memory, so no host round trip separates this call from pi_diff_misses.
 *   n_lists, lists_per_seq   list i belongs to sequence i / lists_per_seq (1 for the shared
 *                            selection, Hkv for per-head lists)
 *   host_kv_pinned           sequence s starts at host_kv_pinned + s*host_seq_stride_bytes
 *   pool_dev                 sequence s starts at pool_dev + s*pool_seq_stride_bytes
 *   recall_list_dev          [n_lists][list_capacity] pi_extent; recall_count_dev [n_lists]
 *   unit_bytes               multiple of 4096
 *                            An extent whose units reach beyond the sequence's pool region (C blocks) or,
 *                            in the block-major store, its host region (NB blocks) sets PI_ERR_INDEX_RANGE
 *                            in the status word (stage 3: list, extent, unit); those units are skipped.
 *                            A list whose units add up to more than the pool region holds is skipped as a
 *                            whole with PI_ERR_CAPACITY (stage 3: list, units, capacity).
 *   unit_stride_bytes        distance between consecutive units (0 = unit_bytes: units are contiguous)
 *   list_offset_bytes        list i starts (i % lists_per_seq) * list_offset_bytes into its sequence's
 *                            region, in the host store and in the pool alike (0 for the shared selection) */
int pi_recall_gather_scatter(pi_ctx* ctx, int layer, int n_lists, int lists_per_seq,
                             const void* host_kv_pinned, int64_t host_seq_stride_bytes,
                             void* pool_dev, int64_t pool_seq_stride_bytes,
                             const pi_extent* recall_list_dev, int32_t list_capacity,
                             const int32_t* recall_count_dev, int64_t unit_bytes, int64_t unit_stride_bytes,
                             int64_t list_offset_bytes, void* stream);

/* Attention of the layer over the selected blocks only (Sec. 4.2.1: after the recall
 * completes the offload batch attends over the recalled blocks): for every query
 * head, softmax(q.K^T / sqrt(D)) V over the tokens t < ctx_len of the selected blocks,
 * K/V read from the pool through sel_slots.
 *   pool_dev [batch][C] blocks; sel_slots_dev / sel_blocks_dev [batch][K]; sel_count_dev [batch]
 *   out_dev  [batch][Hq][D] bf16 (out);  lse_dev [batch][Hq] float natural-log-sum-exp (out) or NULL
 * Pool bytes of tokens beyond ctx_len in a selected block must be finite numbers. */
int pi_sparse_decode_attn(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                          const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev,
                          const int32_t* sel_count_dev, const int32_t* ctx_len_dev, void* out_dev,
                          float* lse_dev, void* stream);

/* The same attention split around the recall (Sec. 4.2.1: the recall of the missing blocks and the
 * attention are two stages of a layer; the selected blocks that were already resident do not wait for
 * the first).  The miss diff never evicts a block of the current selection, so
 *   pi_sparse_decode_attn_resident  may run as soon as pi_diff_misses (or pi_score_select_diff) has
 *       finished, beside pi_recall_gather_scatter: it covers the selected blocks whose slot is not a
 *       destination of recall_list_dev and leaves its softmax state in state_dev;
 *   pi_sparse_decode_attn_recalled  runs after both: it covers the blocks the recall brought in,
 *       folds the state in and writes out_dev.
 * Together they compute what pi_sparse_decode_attn computes (same arithmetic per block, the two
 * partial softmax states merged once more; results agree to fp32 rounding, not bit for bit).
 *   recall_list_dev / list_capacity / recall_count_dev: this step's lists of the shared selection as
 *       pi_diff_misses wrote them (one list per sequence, units = blocks, dst_unit = pool slot)
 *   state_dev: device scratch of pi_attn_state_bytes(ctx, batch) bytes, 16-byte aligned, owned by the
 *       caller; written by the first call, read by the second; contents are private to the library
 *   the other arguments: as pi_sparse_decode_attn (no lse output).
 * Ordering is the caller's: _resident after the diff, _recalled after _resident and after the recall.
 * Shapes the split form does not cover (the attention runs in its flat form, or a CTA's blocks exceed
 * the staged metadata): _resident returns PI_OK without launching anything and _recalled computes the
 * whole attention, so the pair can be called unconditionally. */
int pi_sparse_decode_attn_resident(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                                   const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev,
                                   const int32_t* sel_count_dev, const int32_t* ctx_len_dev,
                                   const pi_extent* recall_list_dev, int32_t list_capacity,
                                   const int32_t* recall_count_dev, float* state_dev, void* stream);
int pi_sparse_decode_attn_recalled(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                                   const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev,
                                   const int32_t* sel_count_dev, const int32_t* ctx_len_dev,
                                   const pi_extent* recall_list_dev, int32_t list_capacity,
                                   const int32_t* recall_count_dev, const float* state_dev, void* out_dev,
                                   void* stream);
/* Bytes of state_dev for `batch` sequences (> 0), or a negative PI_ERR_* code. */
int64_t pi_attn_state_bytes(pi_ctx* ctx, int batch);

/* The same attention when every KV head carries its own selection (the headwise strategy of the
 * paper's selection study, Sec. 4.4.1, as produced by pi_score_select_strategy(PI_SELECT_HEADWISE) +
 * pi_diff_misses over batch*Hkv rows + per-head fragment recall): query heads of KV head h attend
 * over the blocks of list (s, h) only, whose K/V fragments sit in the pool at
 * [slot][h] (the pool keeps the [batch][C][Hkv][2][B][D] layout; slots are per head).
 *   sel_slots_dev / sel_blocks_dev [batch][Hkv][K]; sel_count_dev [batch][Hkv]; the rest as above.
 * Heads of one sequence may select different numbers of blocks. */
int pi_sparse_decode_attn_headwise(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                                   const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev,
                                   const int32_t* sel_count_dev, const int32_t* ctx_len_dev, void* out_dev,
                                   float* lse_dev, void* stream);

/* The step before the path: the decode step's new token joins the cache.  (The paper implies it:
 * an offloaded request keeps its full KV in CPU memory and its sink, local and hot middle tokens
 * on the GPU, Sec. 4.2 and Sec. 5 Setup; it does not describe the operation.)  For every sequence
 * the token lands at position p = ctx_len[s] (the length BEFORE the append; the caller adds one
 * afterwards), block b = p / B, row p % B:
 *   - its K and V rows of all KV heads are written into the pool slot of block b and, through the
 *     GPU-addressable pinned pointer, into the host store;
 *   - the digest row of block b takes the retrieval head's new key into its running min / max;
 *   - a block that has just been opened (p % B == 0) is part of the local window and gets a pool
 *     slot first: the least recently selected slot whose block is neither sink nor local under
 *     the new length (ties to the lower slot, free slots first); the evicted block leaves the
 *     table, the new block's rows start zeroed in the pool and in the host store;
 *   - the slot's stamp becomes `step`.
 *   k_new_dev, v_new_dev  [batch][Hkv][D] bf16;  digest_dev [batch][NB][2][D];  other arrays as in
 *   pi_diff_misses.  Device-side problems (block index beyond NB, nothing evictable, a block that
 *   must be resident is not) set the status word with stage 5 and leave the sequence untouched.
 *   Needs n_local_blocks >= 1 (else PI_ERR_INVALID_ARG): the local window is what keeps the block
 *   that is being filled resident between two appends. */
int pi_append_kv(pi_ctx* ctx, int layer, int batch, uint32_t step, const void* k_new_dev,
                 const void* v_new_dev, const int32_t* ctx_len_dev, void* host_kv_pinned,
                 int64_t host_seq_stride_bytes, void* pool_dev, int32_t* block_table_dev,
                 int32_t* slot_block_dev, uint32_t* slot_stamp_dev, void* digest_dev, void* stream);

/* Paged host store (Sec. 4.4.2: the blocks to recall lie scattered across host memory).  Instead
 * of one block-major region per sequence, the store is an arena of pages, one unit each
 * (unit_stride_bytes apart, page g at host_arena_pinned + g * stride), and logical unit u of
 * sequence s is page page_table_dev[s * page_table_seq_stride + u] (int32, device memory).  The
 * extents still name logical units; each 4 KB piece looks its page up, so merged extents need no
 * physical adjacency.  All other arguments as in pi_recall_gather_scatter / pi_append_kv; a page
 * index outside [0, n_pages), or a unit index beyond the sequence's table row (page_table_seq_stride
 * entries, >= 1), sets PI_ERR_INDEX_RANGE in the status word and the unit is skipped.
 * The caller owns the page table and must have assigned the page of a block before the append
 * that opens it. */
int pi_recall_gather_scatter_paged(pi_ctx* ctx, int layer, int n_lists, int lists_per_seq,
                                   const void* host_arena_pinned, const int32_t* page_table_dev,
                                   int64_t page_table_seq_stride, int32_t n_pages, void* pool_dev,
                                   int64_t pool_seq_stride_bytes, const pi_extent* recall_list_dev,
                                   int32_t list_capacity, const int32_t* recall_count_dev, int64_t unit_bytes,
                                   int64_t unit_stride_bytes, int64_t list_offset_bytes, void* stream);
int pi_append_kv_paged(pi_ctx* ctx, int layer, int batch, uint32_t step, const void* k_new_dev,
                       const void* v_new_dev, const int32_t* ctx_len_dev, void* host_arena_pinned,
                       const int32_t* page_table_dev, int64_t page_table_seq_stride, int32_t n_pages,
                       void* pool_dev, int32_t* block_table_dev, int32_t* slot_block_dev,
                       uint32_t* slot_stamp_dev, void* digest_dev, void* stream);

/* pi_append_kv with the step number read from device memory when the kernel runs (see
 * pi_diff_misses_devstep), for appends inside a replayed CUDA graph.  page_table_dev may be NULL
 * (block-major store, host_seq_stride_bytes used) or a page table as in pi_append_kv_paged (then
 * host_kv_pinned is the arena and host_seq_stride_bytes is ignored). */
int pi_append_kv_devstep(pi_ctx* ctx, int layer, int batch, const uint32_t* step_dev, const void* k_new_dev,
                         const void* v_new_dev, const int32_t* ctx_len_dev, void* host_kv_pinned,
                         int64_t host_seq_stride_bytes, const int32_t* page_table_dev,
                         int64_t page_table_seq_stride, int32_t n_pages, void* pool_dev,
                         int32_t* block_table_dev, int32_t* slot_block_dev, uint32_t* slot_stamp_dev,
                         void* digest_dev, void* stream);

/* Helpers around the path (input preparation and measurement; not hot calls).
 * pi_build_digests: channel-wise min / max of the keys of head solo_head[layer] over the
 *   valid tokens of each block; kv may be device memory or pinned host memory laid out
 *   [batch][NB] blocks with the given sequence stride.  Exact: no rounding happens.
 * pi_table_init: slot i of sequence s holds block resident_dev[s][i] (-1 = free);
 *   fills block_table, slot_block and zero stamps.
 * pi_h2d_copy_ms: best time in ms of `reps` cudaMemcpyAsync copies of `bytes` from pinned
 *   host to device memory (the link's reference bandwidth). Synchronises. */
int pi_build_digests(pi_ctx* ctx, int layer, int batch, const void* kv, int64_t kv_seq_stride_bytes,
                     const int32_t* ctx_len_dev, void* digest_dev, void* stream);
/* the same for every KV head: digest_all_dev [batch][NB][Hkv][2][D] */
int pi_build_digests_all(pi_ctx* ctx, int batch, const void* kv, int64_t kv_seq_stride_bytes,
                         const int32_t* ctx_len_dev, void* digest_all_dev, void* stream);
int pi_table_init(pi_ctx* ctx, int batch, const int32_t* resident_dev, int32_t* block_table_dev,
                  int32_t* slot_block_dev, uint32_t* slot_stamp_dev, void* stream);
int pi_h2d_copy_ms(const void* host_pinned, void* dev, int64_t bytes, int reps, float* best_ms);
/* Middle attention mass (Eq. 2 of the paper: MAM_q = sum over the middle positions of the attention
 * weights of query head q), from the log-sum-exps of two attention calls over the same queries: all
 * blocks (lse_all) and the middle blocks only (lse_mid); the mass of a token set is exp(lse_set - lse_all).
 *   lse_mid_dev, lse_all_dev [batch][Hq] float (in);  mam_q_dev [batch][Hq] float (out);
 *   mam_kv_dev [Hkv] float (out): mean over the batch and over each KV head's query heads (Sec. 4.4.1:
 *   the KV head with the highest value is the layer's retrieval head).  Offline profiling helper. */
int pi_middle_attention_mass(pi_ctx* ctx, int batch, const float* lse_mid_dev, const float* lse_all_dev,
                             float* mam_q_dev, float* mam_kv_dev, void* stream);
/* Launches a kernel that does nothing (n_ctas x n_threads): timed between two events it gives the
 * floor under every per-call time of this library on the box at hand (measurement helper). */
int pi_empty_launch(int n_ctas, int n_threads, void* stream);

/* Sticky device status.  out[0] = first PI_ERR_* code seen by a kernel (0 = none),
 * out[1] = stage (1 score/select, 2 diff, 3 recall, 4 attention, 5 append), out[2..4] = sequence
 * or list, position, offending value.  Reads a pinned mirror: call after the stream
 * has been synchronised.  pi_clear_status resets it. */
int pi_get_status(pi_ctx* ctx, int32_t out[8]);
/* Counters accumulated by pi_diff_misses since creation or the last reset: out[0] = sequences
 * diffed, out[1] = selected blocks, out[2] = missing blocks (= blocks recalled), out[3] = extents
 * emitted.  Synchronises the device. */
int pi_get_stats(pi_ctx* ctx, int64_t out[4], int reset);
int pi_clear_status(pi_ctx* ctx);
const char* pi_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PULSEINFER_H */
