// Shared declarations of the CUDA library: context, status word, small device helpers.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>

#include "pulseinfer.h"

#define PI_STAGE_SELECT 1
#define PI_STAGE_DIFF   2
#define PI_STAGE_RECALL 3
#define PI_STAGE_ATTN   4
#define PI_STAGE_APPEND 5

// Programmatic dependent launch.  Every kernel of the path is launched with programmatic stream
// serialization: its grid may be scheduled while the kernel before it in the stream is still
// running, which takes the launch latency off the chain select -> diff -> recall -> attention ->
// merge.  The rule that keeps this safe: a kernel calls pi_grid_dependency_wait() before it reads or
// writes any global memory (the wait returns once the previous kernel has completed and flushed; it
// is a no-op after a plain launch), and lets its own dependents in only AFTER that wait, so at most
// one kernel runs ahead and whatever a kernel reads before its wait was written at least two
// kernels upstream.
#ifdef __CUDACC__
__device__ __forceinline__ void pi_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pi_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// L2 policy for data that is read once per layer-step (digests, pool blocks): its lines are the first to
// go.  A layer-step streams more bytes than L2 holds; without the hint that stream pushes out what every
// launch needs again -- tables, lists, queries and the kernels' own code, whose refetch from HBM costs the
// serial tail of a launch several microseconds.
__device__ __forceinline__ unsigned long long pi_l2_stream_policy() {
    unsigned long long pol;
#ifdef PI_NO_L2_HINTS
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
#else
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
#endif
    return pol;
}

template <typename... KArgs, typename... Args>
inline cudaError_t pi_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 Args&&... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}
#endif

#define PI_HEAD_DIM 128
#define PI_SELECT_BINS 2048

struct pi_ctx {
    pi_config cfg;
    int32_t* solo_head;          // host copy [n_layers]
    int device;
    int n_sms;
    // device scratch
    float* scores;               // [max_batch][max_blocks]
    unsigned int* sel_counters;  // [max_batch], zero between launches
    unsigned int* attn_counters; // [max_batch], zero between launches
    float* attn_part_o;          // [attn_ctas + max_batch][Hq][D]
    float* attn_part_ml;         // [attn_ctas + max_batch][Hq][2]
    int attn_ctas, recall_ctas;
    long long wait_limit_cycles; // bound of the attention kernel's waits, in SM cycles
    unsigned long long* stats_dev; // [4]: sequences diffed, selected blocks, missing blocks, extents
    // status: device flag (first writer wins) + pinned mirror the kernels fill in
    int* status_flag_dev;
    volatile int32_t* status_host;   // pinned, 8 ints
    int32_t* status_host_devptr;     // device alias of status_host
    // cached tensor map of the pool for the attention kernel
    CUtensorMap pool_map;
    const void* pool_map_ptr;
    long long pool_map_slots;
    int pool_map_headwise;       // box of the cached map: all KV heads of a block (0) or one head (1)
    void* encode_tiled_fn;
    // clusters of 2^i CTAs of the selection kernel that are resident at once, [plain | fused][i]; -1 = not asked yet
    int sd_resident_clusters[2][5];
};

struct pi_status_ref {
    int* flag;
    int32_t* mirror;
};

__device__ __forceinline__ void pi_report(pi_status_ref st, int code, int stage, int a, int b, int c) {
    if (atomicCAS(st.flag, 0, code) == 0) {
        volatile int32_t* m = st.mirror;
        m[1] = stage; m[2] = a; m[3] = b; m[4] = c;
        __threadfence_system();
        m[0] = code;
    }
}

static inline pi_status_ref pi_status_of(pi_ctx* c) {
    pi_status_ref r;
    r.flag = c->status_flag_dev;
    r.mirror = c->status_host_devptr;
    return r;
}

#define PI_CUDA_TRY(expr)                                  \
    do {                                                   \
        cudaError_t e__ = (expr);                          \
        if (e__ != cudaSuccess) { (void)cudaGetLastError(); return PI_ERR_CUDA; } \
    } while (0)

static inline bool pi_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__device__ __forceinline__ int pi_ceil_div(int a, int b) { return (a + b - 1) / b; }

// Launchers implemented one per .cu file.
int pi_launch_score_select(pi_ctx*, int h_star, int batch, const void* q, const void* digest,
                           const int32_t* ctx_len, int32_t* sel, int32_t* sel_count, float* scores,
                           unsigned int* counters, cudaStream_t);
// fused != 0: the diff of the selection runs in the same launch (the diff arguments are then required)
int pi_launch_select_cluster(pi_ctx*, int h_star, int batch, const void* q, const void* digest, const int32_t* ctx_len,
                             int32_t* sel, int32_t* sel_count, float* scores, int fused, uint32_t step,
                             const uint32_t* step_dev, int32_t* table, int32_t* slot_block, uint32_t* slot_stamp,
                             int32_t* sel_slots, pi_extent* list, int32_t* count, cudaStream_t);
int pi_launch_score_select_strategy(pi_ctx*, int strategy, int batch, const void* q, const void* digest_all,
                                    const int32_t* ctx_len, int32_t* sel, int32_t* sel_count, float* scores,
                                    unsigned int* counters, cudaStream_t);
int pi_launch_diff(pi_ctx*, int batch, uint32_t step, const uint32_t* step_dev, const int32_t* ctx_len, const int32_t* sel,
                   const int32_t* sel_count, int32_t* table, int32_t* slot_block, uint32_t* slot_stamp,
                   int32_t* sel_slots, pi_extent* list, int32_t* count, cudaStream_t);
int pi_launch_recall(pi_ctx*, int n_lists, int lists_per_seq, const void* host_kv, int64_t host_stride,
                     void* pool, int64_t pool_stride, const pi_extent* list, int32_t cap,
                     const int32_t* count, int64_t unit_bytes, int64_t unit_stride, int64_t list_offset,
                     const int32_t* page_table, int64_t page_stride, int32_t n_pages, cudaStream_t);
int pi_launch_attn(pi_ctx*, int batch, const void* q, const void* pool, const int32_t* sel_slots,
                   const int32_t* sel_blocks, const int32_t* sel_count, const int32_t* ctx_len,
                   void* out, float* lse, int headwise, cudaStream_t);
// head-major form of the attention (one (sequence, KV head) per CTA); `fits` says whether the items fill the grid evenly
bool pi_attn_headmajor_fits(const pi_ctx*, int batch, int* grid_out, int* items_per_cta_out, int* split_out);
// The attention split around the recall: phase 1 covers the selected blocks that were already resident
// (its result is the softmax state in `state`), phase 2 the blocks the step's recall list brings in, merged
// with that state.  phase 0: everything in one call.
struct pi_attn_phase {
    int phase;
    const pi_extent* rlist;
    int rcap;
    const int32_t* rcount;
    float* state;
};
bool pi_attn_phased_fits(const pi_ctx*, int batch);
long long pi_attn_state_floats(const pi_ctx*, int batch);
int pi_launch_attn_headmajor(pi_ctx*, int batch, const void* q, const void* pool, const int32_t* sel_slots,
                             const int32_t* sel_blocks, const int32_t* sel_count, const int32_t* ctx_len,
                             void* out, float* lse, int headwise, const pi_attn_phase* phase, cudaStream_t);
int pi_launch_append(pi_ctx*, int h_star, int batch, uint32_t step, const void* k_new, const void* v_new,
                     const int32_t* ctx_len, void* host_kv, int64_t host_stride, void* pool, int32_t* table,
                     int32_t* slot_block, uint32_t* slot_stamp, void* digest, const int32_t* page_table,
                     int64_t page_stride, int32_t n_pages, const uint32_t* step_dev, cudaStream_t);
int pi_launch_build_digests_all(pi_ctx*, int batch, const void* kv, int64_t stride, const int32_t* ctx_len,
                                void* digest_all, cudaStream_t);
int pi_launch_build_digests(pi_ctx*, int h_star, int batch, const void* kv, int64_t stride,
                            const int32_t* ctx_len, void* digest, cudaStream_t);
int pi_launch_table_init(pi_ctx*, int batch, const int32_t* resident, int32_t* table,
                         int32_t* slot_block, uint32_t* slot_stamp, cudaStream_t);
