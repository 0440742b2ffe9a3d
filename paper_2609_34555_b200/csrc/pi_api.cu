// C-ABI entry points: context life cycle, argument checks, status word.
#include <cstdlib>
#include <cstring>
#include <new>

#include "pi_common.cuh"

namespace {

bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

int check_config(const pi_config* c) {
    if (!c || !c->solo_head) return PI_ERR_INVALID_ARG;
    if (c->head_dim != PI_HEAD_DIM) return PI_ERR_UNSUPPORTED_DIM;
    if (c->block_tokens != 16 && c->block_tokens != 32 && c->block_tokens != 64) return PI_ERR_UNSUPPORTED_DIM;
    if (c->n_kv_heads < 1 || c->n_kv_heads > 16 || !is_pow2(c->n_kv_heads)) return PI_ERR_UNSUPPORTED_DIM;
    if (c->n_q_heads < c->n_kv_heads || c->n_q_heads % c->n_kv_heads) return PI_ERR_UNSUPPORTED_DIM;
    if (c->n_q_heads / c->n_kv_heads > 16) return PI_ERR_UNSUPPORTED_DIM;
    if (c->n_layers < 1 || c->max_batch < 1 || c->max_batch > 4096) return PI_ERR_INVALID_ARG;
    if (c->max_blocks < 1 || c->max_blocks > 16384) return PI_ERR_UNSUPPORTED_DIM;
    if (c->n_sink_blocks < 0 || c->n_local_blocks < 0) return PI_ERR_INVALID_ARG;
    if (c->budget_blocks < 1 || c->budget_blocks < c->n_sink_blocks + c->n_local_blocks) return PI_ERR_INVALID_ARG;
    if (c->budget_blocks > 4096) return PI_ERR_UNSUPPORTED_DIM;
    if (c->pool_slots < c->budget_blocks) return PI_ERR_POOL_TOO_SMALL;
    if (c->pool_slots > 8192) return PI_ERR_UNSUPPORTED_DIM;
    if (c->recall_ctas < 0 || c->attn_ctas < 0 || c->wait_limit_us < 0) return PI_ERR_INVALID_ARG;
    if (c->test_hold_producer != 0 && c->test_hold_producer != 1) return PI_ERR_INVALID_ARG;
    if (c->attn_mode < 0 || c->attn_mode > 2) return PI_ERR_INVALID_ARG;
    for (int l = 0; l < c->n_layers; ++l)
        if (c->solo_head[l] < 0 || c->solo_head[l] >= c->n_kv_heads) return PI_ERR_INVALID_ARG;
    return PI_OK;
}

int check_call(pi_ctx* ctx, int layer, int batch) {
    if (!ctx) return PI_ERR_INVALID_ARG;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return PI_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return PI_ERR_INVALID_ARG;
    return PI_OK;
}

}  // namespace

extern "C" int pi_create(const pi_config* cfg, pi_ctx** out) {
    if (!out) return PI_ERR_INVALID_ARG;
    *out = nullptr;
    int rc = check_config(cfg);
    if (rc != PI_OK) return rc;
    pi_ctx* c = new (std::nothrow) pi_ctx();
    if (!c) return PI_ERR_INVALID_ARG;
    std::memset(c, 0, sizeof(*c));
    c->cfg = *cfg;
    for (int i = 0; i < 2; ++i)
        for (int j = 0; j < 5; ++j) c->sd_resident_clusters[i][j] = -1;
    c->solo_head = static_cast<int32_t*>(std::malloc(sizeof(int32_t) * cfg->n_layers));
    std::memcpy(c->solo_head, cfg->solo_head, sizeof(int32_t) * cfg->n_layers);
    c->cfg.solo_head = c->solo_head;

    cudaError_t e = cudaGetDevice(&c->device);
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, c->device);
    if (e != cudaSuccess) { (void)cudaGetLastError(); pi_destroy(c); return PI_ERR_CUDA; }
    c->n_sms = prop.multiProcessorCount;
    // the persistent attention grid saturates HBM from about 80 SMs on; leaving 20 SMs to the kernels
    // of the other streams (recall CTAs, score/select, diff) costs it nothing and keeps them off its SMs
    c->attn_ctas = cfg->attn_ctas > 0 ? cfg->attn_ctas : (c->n_sms > 40 ? c->n_sms - 20 : c->n_sms);
    // five CTAs per launch (40 warps x 4 KB in flight): two launches running side by side on two
    // streams saturate the host link of a B200 and cover each other's fixed costs; one launch alone
    // still reaches 0.97 of what ten CTAs do, and more requests in flight only queue up
    c->recall_ctas = cfg->recall_ctas > 0 ? cfg->recall_ctas : 5;
    // a wait that lasts this long is a failure: the kernel gives up and reports (default: two seconds)
    c->wait_limit_cycles = static_cast<long long>(cfg->wait_limit_us > 0 ? cfg->wait_limit_us : 2000000) *
                           (prop.clockRate > 0 ? prop.clockRate : 1000000) / 1000;

    const size_t nb = static_cast<size_t>(cfg->max_batch);
    const size_t n_part = static_cast<size_t>(c->attn_ctas) + nb;
    void* host = nullptr;
    bool ok = cudaMalloc(&c->scores, nb * cfg->max_blocks * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&c->sel_counters, nb * sizeof(unsigned int)) == cudaSuccess &&
              cudaMalloc(&c->attn_counters, nb * sizeof(unsigned int)) == cudaSuccess &&
              cudaMalloc(&c->attn_part_o, n_part * cfg->n_q_heads * PI_HEAD_DIM * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&c->attn_part_ml, n_part * cfg->n_q_heads * 2 * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&c->status_flag_dev, sizeof(int)) == cudaSuccess &&
              cudaMalloc(&c->stats_dev, 4 * sizeof(unsigned long long)) == cudaSuccess &&
              cudaHostAlloc(&host, 8 * sizeof(int32_t), cudaHostAllocMapped) == cudaSuccess;
    if (ok) {
        c->status_host = static_cast<volatile int32_t*>(host);
        for (int i = 0; i < 8; ++i) c->status_host[i] = 0;
        void* alias = nullptr;
        ok = cudaHostGetDevicePointer(&alias, host, 0) == cudaSuccess &&
             cudaMemset(c->sel_counters, 0, nb * sizeof(unsigned int)) == cudaSuccess &&
             cudaMemset(c->attn_counters, 0, nb * sizeof(unsigned int)) == cudaSuccess &&
             cudaMemset(c->status_flag_dev, 0, sizeof(int)) == cudaSuccess &&
             cudaMemset(c->stats_dev, 0, 4 * sizeof(unsigned long long)) == cudaSuccess &&
             cudaDeviceSynchronize() == cudaSuccess;
        c->status_host_devptr = static_cast<int32_t*>(alias);
    }
    if (ok) {
        cudaDriverEntryPointQueryResult q;
        ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_tiled_fn, cudaEnableDefault, &q) == cudaSuccess &&
             q == cudaDriverEntryPointSuccess && c->encode_tiled_fn != nullptr;
    }
    if (!ok) { (void)cudaGetLastError(); pi_destroy(c); return PI_ERR_CUDA; }
    *out = c;
    return PI_OK;
}

extern "C" int pi_destroy(pi_ctx* c) {
    if (!c) return PI_ERR_INVALID_ARG;
    cudaFree(c->scores);
    cudaFree(c->sel_counters);
    cudaFree(c->attn_counters);
    cudaFree(c->attn_part_o);
    cudaFree(c->attn_part_ml);
    cudaFree(c->status_flag_dev);
    cudaFree(c->stats_dev);
    if (c->status_host) cudaFreeHost(const_cast<int32_t*>(c->status_host));
    (void)cudaGetLastError();
    std::free(c->solo_head);
    delete c;
    return PI_OK;
}

extern "C" int pi_score_select(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* digest_dev,
                               const int32_t* ctx_len_dev, int32_t* sel_blocks_dev, int32_t* sel_count_dev,
                               float* scores_dev, void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    if (!q_dev || !digest_dev || !ctx_len_dev || !sel_blocks_dev || !sel_count_dev) return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(q_dev) || !pi_aligned16(digest_dev)) return PI_ERR_BAD_ALIGN;
    return pi_launch_select_cluster(ctx, ctx->solo_head[layer], batch, q_dev, digest_dev, ctx_len_dev, sel_blocks_dev,
                                    sel_count_dev, scores_dev, 0, 0, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                                    nullptr, static_cast<cudaStream_t>(stream));
}

static int select_diff_call(pi_ctx* ctx, int layer, int batch, uint32_t step, const uint32_t* step_dev, const void* q_dev,
                            const void* digest_dev, const int32_t* ctx_len_dev, int32_t* sel_blocks_dev,
                            int32_t* sel_count_dev, float* scores_dev, int32_t* block_table_dev, int32_t* slot_block_dev,
                            uint32_t* slot_stamp_dev, int32_t* sel_slots_dev, pi_extent* recall_list_dev,
                            int32_t* recall_count_dev, void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    if (!q_dev || !digest_dev || !ctx_len_dev || !sel_blocks_dev || !sel_count_dev || !block_table_dev ||
        !slot_block_dev || !slot_stamp_dev || !sel_slots_dev || !recall_list_dev || !recall_count_dev ||
        (!step_dev && step == 0))
        return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(q_dev) || !pi_aligned16(digest_dev) || !pi_aligned16(recall_list_dev)) return PI_ERR_BAD_ALIGN;
    return pi_launch_select_cluster(ctx, ctx->solo_head[layer], batch, q_dev, digest_dev, ctx_len_dev, sel_blocks_dev,
                                    sel_count_dev, scores_dev, 1, step, step_dev, block_table_dev, slot_block_dev,
                                    slot_stamp_dev, sel_slots_dev, recall_list_dev, recall_count_dev,
                                    static_cast<cudaStream_t>(stream));
}

extern "C" int pi_score_select_diff(pi_ctx* ctx, int layer, int batch, uint32_t step, const void* q_dev,
                                    const void* digest_dev, const int32_t* ctx_len_dev, int32_t* sel_blocks_dev,
                                    int32_t* sel_count_dev, float* scores_dev, int32_t* block_table_dev,
                                    int32_t* slot_block_dev, uint32_t* slot_stamp_dev, int32_t* sel_slots_dev,
                                    pi_extent* recall_list_dev, int32_t* recall_count_dev, void* stream) {
    return select_diff_call(ctx, layer, batch, step, nullptr, q_dev, digest_dev, ctx_len_dev, sel_blocks_dev, sel_count_dev,
                            scores_dev, block_table_dev, slot_block_dev, slot_stamp_dev, sel_slots_dev, recall_list_dev,
                            recall_count_dev, stream);
}

extern "C" int pi_score_select_diff_devstep(pi_ctx* ctx, int layer, int batch, const uint32_t* step_dev, const void* q_dev,
                                            const void* digest_dev, const int32_t* ctx_len_dev, int32_t* sel_blocks_dev,
                                            int32_t* sel_count_dev, float* scores_dev, int32_t* block_table_dev,
                                            int32_t* slot_block_dev, uint32_t* slot_stamp_dev, int32_t* sel_slots_dev,
                                            pi_extent* recall_list_dev, int32_t* recall_count_dev, void* stream) {
    if (!step_dev) return PI_ERR_INVALID_ARG;
    return select_diff_call(ctx, layer, batch, 0, step_dev, q_dev, digest_dev, ctx_len_dev, sel_blocks_dev, sel_count_dev,
                            scores_dev, block_table_dev, slot_block_dev, slot_stamp_dev, sel_slots_dev, recall_list_dev,
                            recall_count_dev, stream);
}

extern "C" int pi_score_select_strategy(pi_ctx* ctx, int strategy, int layer, int batch, const void* q_dev,
                                       const void* digest_all_dev, const int32_t* ctx_len_dev,
                                       int32_t* sel_blocks_dev, int32_t* sel_count_dev, float* scores_dev,
                                       void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    if (strategy != PI_SELECT_AVERAGE && strategy != PI_SELECT_HEADWISE) return PI_ERR_INVALID_ARG;
    if (!q_dev || !digest_all_dev || !ctx_len_dev || !sel_blocks_dev || !sel_count_dev) return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(q_dev) || !pi_aligned16(digest_all_dev)) return PI_ERR_BAD_ALIGN;
    const int n_virtual = strategy == PI_SELECT_HEADWISE ? batch * ctx->cfg.n_kv_heads : batch;
    if (n_virtual > ctx->cfg.max_batch) return PI_ERR_CAPACITY;      // scratch holds max_batch score rows
    return pi_launch_score_select_strategy(ctx, strategy, batch, q_dev, digest_all_dev, ctx_len_dev, sel_blocks_dev,
                                           sel_count_dev, scores_dev ? scores_dev : ctx->scores, ctx->sel_counters,
                                           static_cast<cudaStream_t>(stream));
}

static int diff_call(pi_ctx* ctx, int layer, int batch, uint32_t step, const uint32_t* step_dev,
                     const int32_t* ctx_len_dev, const int32_t* sel_blocks_dev, const int32_t* sel_count_dev,
                     int32_t* block_table_dev, int32_t* slot_block_dev, uint32_t* slot_stamp_dev,
                     int32_t* sel_slots_dev, pi_extent* recall_list_dev, int32_t* recall_count_dev, void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    if (!ctx_len_dev || !sel_blocks_dev || !sel_count_dev || !block_table_dev || !slot_block_dev ||
        !slot_stamp_dev || !sel_slots_dev || !recall_list_dev || !recall_count_dev || (!step_dev && step == 0))
        return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(recall_list_dev)) return PI_ERR_BAD_ALIGN;
    return pi_launch_diff(ctx, batch, step, step_dev, ctx_len_dev, sel_blocks_dev, sel_count_dev, block_table_dev,
                          slot_block_dev, slot_stamp_dev, sel_slots_dev, recall_list_dev, recall_count_dev,
                          static_cast<cudaStream_t>(stream));
}

extern "C" int pi_diff_misses(pi_ctx* ctx, int layer, int batch, uint32_t step, const int32_t* ctx_len_dev,
                              const int32_t* sel_blocks_dev, const int32_t* sel_count_dev,
                              int32_t* block_table_dev, int32_t* slot_block_dev, uint32_t* slot_stamp_dev,
                              int32_t* sel_slots_dev, pi_extent* recall_list_dev, int32_t* recall_count_dev,
                              void* stream) {
    return diff_call(ctx, layer, batch, step, nullptr, ctx_len_dev, sel_blocks_dev, sel_count_dev, block_table_dev,
                     slot_block_dev, slot_stamp_dev, sel_slots_dev, recall_list_dev, recall_count_dev, stream);
}

extern "C" int pi_diff_misses_devstep(pi_ctx* ctx, int layer, int batch, const uint32_t* step_dev,
                                      const int32_t* ctx_len_dev, const int32_t* sel_blocks_dev,
                                      const int32_t* sel_count_dev, int32_t* block_table_dev,
                                      int32_t* slot_block_dev, uint32_t* slot_stamp_dev, int32_t* sel_slots_dev,
                                      pi_extent* recall_list_dev, int32_t* recall_count_dev, void* stream) {
    if (!step_dev) return PI_ERR_INVALID_ARG;
    return diff_call(ctx, layer, batch, 0, step_dev, ctx_len_dev, sel_blocks_dev, sel_count_dev, block_table_dev,
                     slot_block_dev, slot_stamp_dev, sel_slots_dev, recall_list_dev, recall_count_dev, stream);
}

// Shared by the block-major and the paged entry point (page_table == nullptr: block-major).
static int recall_call(pi_ctx* ctx, int layer, int n_lists, int lists_per_seq, const void* host_kv_pinned,
                       int64_t host_seq_stride_bytes, const int32_t* page_table, int64_t page_stride, int32_t n_pages,
                       void* pool_dev, int64_t pool_seq_stride_bytes, const pi_extent* recall_list_dev,
                       int32_t list_capacity, const int32_t* recall_count_dev, int64_t unit_bytes,
                       int64_t unit_stride_bytes, int64_t list_offset_bytes, void* stream) {
    if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers) return PI_ERR_INVALID_ARG;
    if (n_lists < 1 || lists_per_seq < 1 || n_lists % lists_per_seq || n_lists > 65536) return PI_ERR_INVALID_ARG;
    if (!host_kv_pinned || !pool_dev || !recall_list_dev || !recall_count_dev || list_capacity < 1)
        return PI_ERR_INVALID_ARG;
    if (unit_bytes < 4096 || unit_bytes % 4096 || unit_bytes > (1 << 24)) return PI_ERR_UNSUPPORTED_DIM;
    if (unit_stride_bytes < 0 || (unit_stride_bytes > 0 && unit_stride_bytes < unit_bytes) || unit_stride_bytes % 16 ||
        list_offset_bytes < 0 || list_offset_bytes % 16)
        return PI_ERR_INVALID_ARG;
    if (host_seq_stride_bytes % 16 || pool_seq_stride_bytes % 16 || host_seq_stride_bytes < 0 ||
        pool_seq_stride_bytes < 0)
        return PI_ERR_BAD_ALIGN;
    if (!pi_aligned16(host_kv_pinned) || !pi_aligned16(pool_dev) || !pi_aligned16(recall_list_dev))
        return PI_ERR_BAD_ALIGN;
    // the store must be memory the GPU can address: pinned host (or device) memory
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host_kv_pinned) != cudaSuccess) { (void)cudaGetLastError(); return PI_ERR_NOT_PINNED; }
    const void* src = host_kv_pinned;
    if (attr.type == cudaMemoryTypeHost) {
        if (!attr.devicePointer) return PI_ERR_NOT_PINNED;
        src = attr.devicePointer;
    } else if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) {
        return PI_ERR_NOT_PINNED;
    }
    return pi_launch_recall(ctx, n_lists, lists_per_seq, src, host_seq_stride_bytes, pool_dev,
                            pool_seq_stride_bytes, recall_list_dev, list_capacity, recall_count_dev,
                            unit_bytes, unit_stride_bytes, list_offset_bytes, page_table, page_stride, n_pages,
                            static_cast<cudaStream_t>(stream));
}

extern "C" int pi_recall_gather_scatter(pi_ctx* ctx, int layer, int n_lists, int lists_per_seq,
                                        const void* host_kv_pinned, int64_t host_seq_stride_bytes,
                                        void* pool_dev, int64_t pool_seq_stride_bytes,
                                        const pi_extent* recall_list_dev, int32_t list_capacity,
                                        const int32_t* recall_count_dev, int64_t unit_bytes,
                                        int64_t unit_stride_bytes, int64_t list_offset_bytes, void* stream) {
    return recall_call(ctx, layer, n_lists, lists_per_seq, host_kv_pinned, host_seq_stride_bytes, nullptr, 0, 0,
                       pool_dev, pool_seq_stride_bytes, recall_list_dev, list_capacity, recall_count_dev, unit_bytes,
                       unit_stride_bytes, list_offset_bytes, stream);
}

extern "C" int pi_recall_gather_scatter_paged(pi_ctx* ctx, int layer, int n_lists, int lists_per_seq,
                                              const void* host_arena_pinned, const int32_t* page_table_dev,
                                              int64_t page_table_seq_stride, int32_t n_pages, void* pool_dev,
                                              int64_t pool_seq_stride_bytes, const pi_extent* recall_list_dev,
                                              int32_t list_capacity, const int32_t* recall_count_dev,
                                              int64_t unit_bytes, int64_t unit_stride_bytes,
                                              int64_t list_offset_bytes, void* stream) {
    if (!page_table_dev || page_table_seq_stride < 1 || n_pages < 1) return PI_ERR_INVALID_ARG;
    return recall_call(ctx, layer, n_lists, lists_per_seq, host_arena_pinned, 0, page_table_dev, page_table_seq_stride,
                       n_pages, pool_dev, pool_seq_stride_bytes, recall_list_dev, list_capacity, recall_count_dev,
                       unit_bytes, unit_stride_bytes, list_offset_bytes, stream);
}

static int attn_call(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                     const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev, const int32_t* sel_count_dev,
                     const int32_t* ctx_len_dev, void* out_dev, float* lse_dev, int headwise, void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    if (!q_dev || !pool_dev || !sel_slots_dev || !sel_blocks_dev || !sel_count_dev || !ctx_len_dev || !out_dev)
        return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(q_dev) || !pi_aligned16(out_dev) || (reinterpret_cast<uintptr_t>(pool_dev) & 127u))
        return PI_ERR_BAD_ALIGN;
    return pi_launch_attn(ctx, batch, q_dev, pool_dev, sel_slots_dev, sel_blocks_dev, sel_count_dev,
                          ctx_len_dev, out_dev, lse_dev, headwise, static_cast<cudaStream_t>(stream));
}

extern "C" int pi_sparse_decode_attn(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                                     const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev,
                                     const int32_t* sel_count_dev, const int32_t* ctx_len_dev, void* out_dev,
                                     float* lse_dev, void* stream) {
    return attn_call(ctx, layer, batch, q_dev, pool_dev, sel_slots_dev, sel_blocks_dev, sel_count_dev, ctx_len_dev,
                     out_dev, lse_dev, 0, stream);
}

extern "C" int pi_sparse_decode_attn_headwise(pi_ctx* ctx, int layer, int batch, const void* q_dev,
                                              const void* pool_dev, const int32_t* sel_slots_dev,
                                              const int32_t* sel_blocks_dev, const int32_t* sel_count_dev,
                                              const int32_t* ctx_len_dev, void* out_dev, float* lse_dev,
                                              void* stream) {
    return attn_call(ctx, layer, batch, q_dev, pool_dev, sel_slots_dev, sel_blocks_dev, sel_count_dev, ctx_len_dev,
                     out_dev, lse_dev, 1, stream);
}

// Attention split around the recall.  Where the head-major form with staged metadata does not apply the
// first call does nothing and the second one is the whole attention.
static int attn_phase_call(pi_ctx* ctx, int layer, int batch, int phase, const void* q_dev, const void* pool_dev,
                           const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev, const int32_t* sel_count_dev,
                           const int32_t* ctx_len_dev, const pi_extent* recall_list_dev, int32_t list_capacity,
                           const int32_t* recall_count_dev, float* state_dev, void* out_dev, void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    if (!q_dev || !pool_dev || !sel_slots_dev || !sel_blocks_dev || !sel_count_dev || !ctx_len_dev ||
        !recall_list_dev || !recall_count_dev || list_capacity < 1 || !state_dev || (phase == 2 && !out_dev))
        return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(q_dev) || (out_dev && !pi_aligned16(out_dev)) || !pi_aligned16(state_dev) ||
        !pi_aligned16(recall_list_dev) || (reinterpret_cast<uintptr_t>(pool_dev) & 127u))
        return PI_ERR_BAD_ALIGN;
    if (!pi_attn_phased_fits(ctx, batch)) {
        if (phase == 1) return PI_OK;
        return pi_launch_attn(ctx, batch, q_dev, pool_dev, sel_slots_dev, sel_blocks_dev, sel_count_dev, ctx_len_dev,
                              out_dev, nullptr, 0, static_cast<cudaStream_t>(stream));
    }
    pi_attn_phase ph;
    ph.phase = phase; ph.rlist = recall_list_dev; ph.rcap = list_capacity; ph.rcount = recall_count_dev; ph.state = state_dev;
    return pi_launch_attn_headmajor(ctx, batch, q_dev, pool_dev, sel_slots_dev, sel_blocks_dev, sel_count_dev,
                                    ctx_len_dev, out_dev, nullptr, 0, &ph, static_cast<cudaStream_t>(stream));
}

extern "C" int pi_sparse_decode_attn_resident(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                                              const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev,
                                              const int32_t* sel_count_dev, const int32_t* ctx_len_dev,
                                              const pi_extent* recall_list_dev, int32_t list_capacity,
                                              const int32_t* recall_count_dev, float* state_dev, void* stream) {
    return attn_phase_call(ctx, layer, batch, 1, q_dev, pool_dev, sel_slots_dev, sel_blocks_dev, sel_count_dev,
                           ctx_len_dev, recall_list_dev, list_capacity, recall_count_dev, state_dev, nullptr, stream);
}

extern "C" int pi_sparse_decode_attn_recalled(pi_ctx* ctx, int layer, int batch, const void* q_dev, const void* pool_dev,
                                              const int32_t* sel_slots_dev, const int32_t* sel_blocks_dev,
                                              const int32_t* sel_count_dev, const int32_t* ctx_len_dev,
                                              const pi_extent* recall_list_dev, int32_t list_capacity,
                                              const int32_t* recall_count_dev, const float* state_dev, void* out_dev,
                                              void* stream) {
    return attn_phase_call(ctx, layer, batch, 2, q_dev, pool_dev, sel_slots_dev, sel_blocks_dev, sel_count_dev,
                           ctx_len_dev, recall_list_dev, list_capacity, recall_count_dev, const_cast<float*>(state_dev),
                           out_dev, stream);
}

extern "C" int64_t pi_attn_state_bytes(pi_ctx* ctx, int batch) {
    if (!ctx || batch < 1 || batch > ctx->cfg.max_batch) return PI_ERR_INVALID_ARG;
    return pi_attn_state_floats(ctx, batch) * 4;
}

static int append_call(pi_ctx* ctx, int layer, int batch, uint32_t step, const uint32_t* step_dev, const void* k_new_dev, const void* v_new_dev,
                       const int32_t* ctx_len_dev, void* host_kv_pinned, int64_t host_seq_stride_bytes,
                       const int32_t* page_table, int64_t page_stride, int32_t n_pages, void* pool_dev,
                       int32_t* block_table_dev, int32_t* slot_block_dev, uint32_t* slot_stamp_dev, void* digest_dev,
                       void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    // without a local window nothing keeps the block that is being filled resident: a later token of
    // the same block could find it evicted and be lost from the host store as well
    if (ctx->cfg.n_local_blocks < 1) return PI_ERR_INVALID_ARG;
    if (!k_new_dev || !v_new_dev || !ctx_len_dev || !host_kv_pinned || !pool_dev || !block_table_dev ||
        !slot_block_dev || !slot_stamp_dev || !digest_dev || (!step_dev && step == 0) || host_seq_stride_bytes < 0)
        return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(k_new_dev) || !pi_aligned16(v_new_dev) || !pi_aligned16(host_kv_pinned) ||
        !pi_aligned16(pool_dev) || !pi_aligned16(digest_dev) || host_seq_stride_bytes % 16)
        return PI_ERR_BAD_ALIGN;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host_kv_pinned) != cudaSuccess) { (void)cudaGetLastError(); return PI_ERR_NOT_PINNED; }
    void* dst = host_kv_pinned;
    if (attr.type == cudaMemoryTypeHost) {
        if (!attr.devicePointer) return PI_ERR_NOT_PINNED;
        dst = attr.devicePointer;
    } else if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) {
        return PI_ERR_NOT_PINNED;
    }
    return pi_launch_append(ctx, ctx->solo_head[layer], batch, step, k_new_dev, v_new_dev, ctx_len_dev, dst,
                            host_seq_stride_bytes, pool_dev, block_table_dev, slot_block_dev, slot_stamp_dev,
                            digest_dev, page_table, page_stride, n_pages, step_dev, static_cast<cudaStream_t>(stream));
}

extern "C" int pi_append_kv(pi_ctx* ctx, int layer, int batch, uint32_t step, const void* k_new_dev,
                            const void* v_new_dev, const int32_t* ctx_len_dev, void* host_kv_pinned,
                            int64_t host_seq_stride_bytes, void* pool_dev, int32_t* block_table_dev,
                            int32_t* slot_block_dev, uint32_t* slot_stamp_dev, void* digest_dev, void* stream) {
    return append_call(ctx, layer, batch, step, nullptr, k_new_dev, v_new_dev, ctx_len_dev, host_kv_pinned,
                       host_seq_stride_bytes, nullptr, 0, 0, pool_dev, block_table_dev, slot_block_dev,
                       slot_stamp_dev, digest_dev, stream);
}

extern "C" int pi_append_kv_paged(pi_ctx* ctx, int layer, int batch, uint32_t step, const void* k_new_dev,
                                  const void* v_new_dev, const int32_t* ctx_len_dev, void* host_arena_pinned,
                                  const int32_t* page_table_dev, int64_t page_table_seq_stride, int32_t n_pages,
                                  void* pool_dev, int32_t* block_table_dev, int32_t* slot_block_dev,
                                  uint32_t* slot_stamp_dev, void* digest_dev, void* stream) {
    if (!page_table_dev || page_table_seq_stride < 1 || n_pages < 1) return PI_ERR_INVALID_ARG;
    return append_call(ctx, layer, batch, step, nullptr, k_new_dev, v_new_dev, ctx_len_dev, host_arena_pinned, 0,
                       page_table_dev, page_table_seq_stride, n_pages, pool_dev, block_table_dev, slot_block_dev,
                       slot_stamp_dev, digest_dev, stream);
}

extern "C" int pi_append_kv_devstep(pi_ctx* ctx, int layer, int batch, const uint32_t* step_dev, const void* k_new_dev,
                                    const void* v_new_dev, const int32_t* ctx_len_dev, void* host_kv_pinned,
                                    int64_t host_seq_stride_bytes, const int32_t* page_table_dev,
                                    int64_t page_table_seq_stride, int32_t n_pages, void* pool_dev,
                                    int32_t* block_table_dev, int32_t* slot_block_dev, uint32_t* slot_stamp_dev,
                                    void* digest_dev, void* stream) {
    if (!step_dev) return PI_ERR_INVALID_ARG;
    if (page_table_dev && (page_table_seq_stride < 1 || n_pages < 1)) return PI_ERR_INVALID_ARG;
    return append_call(ctx, layer, batch, 0, step_dev, k_new_dev, v_new_dev, ctx_len_dev, host_kv_pinned,
                       page_table_dev ? 0 : host_seq_stride_bytes, page_table_dev, page_table_seq_stride, n_pages,
                       pool_dev, block_table_dev, slot_block_dev, slot_stamp_dev, digest_dev, stream);
}

extern "C" int pi_build_digests(pi_ctx* ctx, int layer, int batch, const void* kv, int64_t kv_seq_stride_bytes,
                                const int32_t* ctx_len_dev, void* digest_dev, void* stream) {
    int rc = check_call(ctx, layer, batch);
    if (rc != PI_OK) return rc;
    if (!kv || !ctx_len_dev || !digest_dev || kv_seq_stride_bytes < 0) return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(kv) || !pi_aligned16(digest_dev) || kv_seq_stride_bytes % 16) return PI_ERR_BAD_ALIGN;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, kv) != cudaSuccess) { (void)cudaGetLastError(); return PI_ERR_NOT_PINNED; }
    const void* src = kv;
    if (attr.type == cudaMemoryTypeHost) {
        if (!attr.devicePointer) return PI_ERR_NOT_PINNED;
        src = attr.devicePointer;
    } else if (attr.type == cudaMemoryTypeUnregistered) {
        return PI_ERR_NOT_PINNED;
    }
    return pi_launch_build_digests(ctx, ctx->solo_head[layer], batch, src, kv_seq_stride_bytes, ctx_len_dev,
                                   digest_dev, static_cast<cudaStream_t>(stream));
}

extern "C" int pi_build_digests_all(pi_ctx* ctx, int batch, const void* kv, int64_t kv_seq_stride_bytes,
                                    const int32_t* ctx_len_dev, void* digest_all_dev, void* stream) {
    int rc = check_call(ctx, 0, batch);
    if (rc != PI_OK) return rc;
    if (!kv || !ctx_len_dev || !digest_all_dev || kv_seq_stride_bytes < 0) return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(kv) || !pi_aligned16(digest_all_dev) || kv_seq_stride_bytes % 16) return PI_ERR_BAD_ALIGN;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, kv) != cudaSuccess) { (void)cudaGetLastError(); return PI_ERR_NOT_PINNED; }
    const void* src = kv;
    if (attr.type == cudaMemoryTypeHost) {
        if (!attr.devicePointer) return PI_ERR_NOT_PINNED;
        src = attr.devicePointer;
    } else if (attr.type == cudaMemoryTypeUnregistered) {
        return PI_ERR_NOT_PINNED;
    }
    return pi_launch_build_digests_all(ctx, batch, src, kv_seq_stride_bytes, ctx_len_dev, digest_all_dev,
                                       static_cast<cudaStream_t>(stream));
}

extern "C" int pi_table_init(pi_ctx* ctx, int batch, const int32_t* resident_dev, int32_t* block_table_dev,
                             int32_t* slot_block_dev, uint32_t* slot_stamp_dev, void* stream) {
    int rc = check_call(ctx, 0, batch);
    if (rc != PI_OK) return rc;
    if (!resident_dev || !block_table_dev || !slot_block_dev || !slot_stamp_dev) return PI_ERR_INVALID_ARG;
    return pi_launch_table_init(ctx, batch, resident_dev, block_table_dev, slot_block_dev, slot_stamp_dev,
                                static_cast<cudaStream_t>(stream));
}

extern "C" int pi_h2d_copy_ms(const void* host_pinned, void* dev, int64_t bytes, int reps, float* best_ms) {
    if (!host_pinned || !dev || bytes <= 0 || reps < 1 || !best_ms) return PI_ERR_INVALID_ARG;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host_pinned) != cudaSuccess || attr.type != cudaMemoryTypeHost) {
        (void)cudaGetLastError();
        return PI_ERR_NOT_PINNED;
    }
    cudaEvent_t a, b;
    PI_CUDA_TRY(cudaEventCreate(&a));
    PI_CUDA_TRY(cudaEventCreate(&b));
    float best = 1e30f;
    int rc = PI_OK;
    for (int i = 0; i < reps + 1 && rc == PI_OK; ++i) {   // first copy is a warm-up
        float ms = 0.f;
        if (cudaEventRecord(a, 0) != cudaSuccess ||
            cudaMemcpyAsync(dev, host_pinned, static_cast<size_t>(bytes), cudaMemcpyHostToDevice, 0) != cudaSuccess ||
            cudaEventRecord(b, 0) != cudaSuccess || cudaEventSynchronize(b) != cudaSuccess ||
            cudaEventElapsedTime(&ms, a, b) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = PI_ERR_CUDA;
        } else if (i > 0 && ms < best) {
            best = ms;
        }
    }
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    *best_ms = best;
    return rc;
}

extern "C" int pi_get_status(pi_ctx* ctx, int32_t out[8]) {
    if (!ctx || !out) return PI_ERR_INVALID_ARG;
    for (int i = 0; i < 8; ++i) out[i] = ctx->status_host[i];
    return PI_OK;
}

extern "C" int pi_get_stats(pi_ctx* ctx, int64_t out[4], int reset) {
    if (!ctx || !out) return PI_ERR_INVALID_ARG;
    unsigned long long h[4];
    PI_CUDA_TRY(cudaDeviceSynchronize());
    PI_CUDA_TRY(cudaMemcpy(h, ctx->stats_dev, sizeof(h), cudaMemcpyDeviceToHost));
    if (reset) PI_CUDA_TRY(cudaMemset(ctx->stats_dev, 0, sizeof(h)));
    for (int i = 0; i < 4; ++i) out[i] = static_cast<int64_t>(h[i]);
    return PI_OK;
}

extern "C" int pi_clear_status(pi_ctx* ctx) {
    if (!ctx) return PI_ERR_INVALID_ARG;
    PI_CUDA_TRY(cudaDeviceSynchronize());
    PI_CUDA_TRY(cudaMemset(ctx->status_flag_dev, 0, sizeof(int)));
    for (int i = 0; i < 8; ++i) ctx->status_host[i] = 0;
    PI_CUDA_TRY(cudaDeviceSynchronize());
    return PI_OK;
}

extern "C" const char* pi_strerror(int code) {
    switch (code) {
        case PI_OK: return "ok";
        case PI_ERR_INVALID_ARG: return "invalid argument";
        case PI_ERR_BAD_ALIGN: return "pointer or stride not 16-byte aligned";
        case PI_ERR_UNSUPPORTED_DIM: return "unsupported dimension";
        case PI_ERR_POOL_TOO_SMALL: return "pool has too few evictable slots";
        case PI_ERR_NOT_PINNED: return "host store is not GPU-addressable (pin it)";
        case PI_ERR_CUDA: return "CUDA runtime error";
        case PI_ERR_TIMEOUT: return "bounded device wait ran out";
        case PI_ERR_INDEX_RANGE: return "index read from a device list is out of range";
        case PI_ERR_CAPACITY: return "count read from device memory exceeds capacity";
        case PI_ERR_STATIC_LIMIT: return "batch or max_blocks exceeds the fixed scratch of pi_score_select_noalloc (64 x 8192)";
        default: return "unknown error";
    }
}
