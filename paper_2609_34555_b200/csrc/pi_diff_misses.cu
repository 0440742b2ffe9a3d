// Miss diff of the selection against the device-resident block table, victim choice,
// table update and the coalesced recall list.  One CTA per sequence; everything the
// sequence needs (selection, slot keys) sits in shared memory.
//
//   misses     = selected blocks with block_table[b] < 0, ascending
//   candidates = slots whose block is neither selected nor sink/local (free slots count),
//                ordered by (stamp, slot) ascending; the i-th miss takes the i-th candidate
//                (few misses: repeated block-wide arg-min; many: bitonic sort)
//   update     = evicted block leaves the table, the miss enters it, every selected
//                slot gets stamp = step
//   list       = (block -> slot) pairs, runs that are consecutive on both sides merged
#include "pi_common.cuh"

namespace {

constexpr int DIFF_THREADS = 256;
constexpr int DIFF_WARPS = DIFF_THREADS / 32;
constexpr int ARGMIN_MAX_MISSES = 40;            // above this the full sort is cheaper
constexpr int ARGMIN_KEYS_PER_THREAD = 4;        // register-resident keys: pools up to 1024 slots

struct DiffParams {
    const int32_t* ctx_len;
    const int32_t* sel;
    const int32_t* sel_count;
    int32_t* table;
    int32_t* slot_block;
    uint32_t* slot_stamp;
    int32_t* sel_slots;
    pi_extent* list;
    int32_t* count;
    pi_status_ref st;
    unsigned long long* stats;
    uint32_t step;
    const uint32_t* step_dev;      // when set, the step is read from device memory (a captured graph replays with a new step)
    int B, K, C, Cpad, n_sink, n_local, max_blocks;
};

// Ordered compaction step for up to DIFF_THREADS flags: returns this thread's output
// position (valid if flag) and adds the round's total to `base` (uniform across the CTA).
__device__ __forceinline__ int ordered_pos(bool flag, int& base, int* warp_tot) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const unsigned m = __ballot_sync(0xffffffffu, flag);
    __syncthreads();
    if (lane == 0) warp_tot[w] = __popc(m);
    __syncthreads();
    int off = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < DIFF_WARPS; ++i) {
        const int t = warp_tot[i];
        if (i < w) off += t;
        tot += t;
    }
    const int pos = base + off + __popc(m & ((1u << lane) - 1u));
    base += tot;
    return pos;
}

__global__ void __launch_bounds__(DIFF_THREADS)
diff_kernel(DiffParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pi_grid_dependency_wait();
    pi_launch_dependents();
    const uint32_t step = p.step_dev ? *p.step_dev : p.step;
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);       // [Cpad]
    int32_t* s_sel = reinterpret_cast<int32_t*>(keys + p.Cpad);                         // [K]
    int32_t* s_slot = s_sel + p.K;                                                      // [K] slot of sel[j]
    int32_t* s_miss = s_slot + p.K;                                                     // [K] j index of i-th miss
    unsigned char* s_used = reinterpret_cast<unsigned char*>(s_miss + p.K);             // [C] slot holds a selected block
    __shared__ int warp_tot[DIFF_WARPS];
    __shared__ unsigned long long warp_min[2][DIFF_WARPS];
    __shared__ int s_ncand;

    const int seq = blockIdx.x, tid = threadIdx.x;
    int ctx = p.ctx_len[seq];
    if (ctx < 0) ctx = 0;
    const int n_blocks = min((ctx + p.B - 1) / p.B, p.max_blocks);
    int cnt = p.sel_count[seq];
    if (cnt < 0 || cnt > p.K) {
        if (tid == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_DIFF, seq, cnt, p.K);
        cnt = max(0, min(cnt, p.K));
    }
    int32_t* table = p.table + static_cast<size_t>(seq) * p.max_blocks;
    int32_t* slot_block = p.slot_block + static_cast<size_t>(seq) * p.C;
    uint32_t* slot_stamp = p.slot_stamp + static_cast<size_t>(seq) * p.C;
    const int32_t* sel = p.sel + static_cast<size_t>(seq) * p.K;

    for (int s = tid; s < p.C; s += DIFF_THREADS) s_used[s] = 0;
    if (tid == 0) s_ncand = 0;
    __syncthreads();

    // 1. look the selection up; misses compacted in selection (= ascending block) order
    int n_miss = 0;
    for (int j0 = 0; j0 < cnt; j0 += DIFF_THREADS) {
        const int j = j0 + tid;
        bool miss = false;
        if (j < cnt) {
            int b = sel[j];
            int slot = -1;
            if (b < 0 || b >= n_blocks) {
                pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_DIFF, seq, j, b);
                b = -1;
            } else {
                slot = table[b];
                if (slot >= p.C) { pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_DIFF, seq, b, slot); slot = -1; b = -1; }
                else if (slot >= 0) s_used[slot] = 1;
                else miss = true;
            }
            s_sel[j] = b;
            s_slot[j] = slot;
        }
        const int pos = ordered_pos(miss, n_miss, warp_tot);
        if (miss) s_miss[pos] = j;
    }
    __syncthreads();

    // 2. victim candidates keyed by (stamp, slot); everything else sorts to the end
    int my_cand = 0;
    for (int s = tid; s < p.Cpad; s += DIFF_THREADS) {
        unsigned long long key = ~0ull;
        if (s < p.C && n_miss > 0) {
            const int b = slot_block[s];
            const bool pinned = b >= 0 && (b < p.n_sink || b >= n_blocks - p.n_local);
            if (b < 0 || (!s_used[s] && !pinned)) {
                key = (static_cast<unsigned long long>(slot_stamp[s]) << 32) | static_cast<unsigned>(s);
                ++my_cand;
            }
        }
        keys[s] = key;
    }
    if (my_cand) atomicAdd(&s_ncand, my_cand);
    __syncthreads();
    const bool too_small = s_ncand < n_miss;

    if (n_miss > 0 && !too_small) {
        // 3. the n_miss smallest candidate keys, in order, end up in keys[0 .. n_miss).
        if (n_miss <= ARGMIN_MAX_MISSES && p.Cpad <= DIFF_THREADS * ARGMIN_KEYS_PER_THREAD) {
            // few misses (the steady state): n_miss rounds of a block-wide arg-min over keys held
            // in registers, one CTA barrier per round (warp minima are double-buffered).
            const int lane = tid & 31, warp = tid >> 5;
            unsigned long long mine[ARGMIN_KEYS_PER_THREAD];
#pragma unroll
            for (int e = 0; e < ARGMIN_KEYS_PER_THREAD; ++e) {
                const int s_ = tid + e * DIFF_THREADS;
                mine[e] = s_ < p.Cpad ? keys[s_] : ~0ull;
            }
            __syncthreads();                       // keys[] may now be overwritten with the result
            for (int i = 0; i < n_miss; ++i) {
                unsigned long long v = mine[0];
#pragma unroll
                for (int e = 1; e < ARGMIN_KEYS_PER_THREAD; ++e) v = min(v, mine[e]);
#pragma unroll
                for (int o = 16; o; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
                if (lane == 0) warp_min[i & 1][warp] = v;
                __syncthreads();
                unsigned long long g = warp_min[i & 1][0];
#pragma unroll
                for (int w = 1; w < DIFF_WARPS; ++w) g = min(g, warp_min[i & 1][w]);
#pragma unroll
                for (int e = 0; e < ARGMIN_KEYS_PER_THREAD; ++e)
                    if (mine[e] == g) { mine[e] = ~0ull; keys[i] = g; }   // keys are unique (slot in the low word)
            }
            __syncthreads();
        } else {
            // many misses (cold start): bitonic sort of all candidate keys.  Warp w owns elements
            // [32*E*w, 32*E*(w+1)), so exchanges at distance < 32*E stay inside one warp and need
            // only a warp barrier; the few longer ones are fenced by CTA barriers.
            const int E = max(1, p.Cpad / DIFF_THREADS), wspan = 32 * E;
            const int lane = tid & 31, warp = tid >> 5;
            for (int k = 2; k <= p.Cpad; k <<= 1) {
                for (int j = k >> 1; j > 0; j >>= 1) {
                    if (j >= wspan) __syncthreads();
                    for (int e = 0; e < E; ++e) {
                        const int i = (warp * E + e) * 32 + lane, l = i ^ j;
                        if (l > i && l < p.Cpad) {
                            const unsigned long long a = keys[i], b = keys[l];
                            const bool up = (i & k) == 0;
                            if ((a > b) == up) { keys[i] = b; keys[l] = a; }
                        }
                    }
                    if (j >= wspan) __syncthreads(); else __syncwarp();
                }
            }
            __syncthreads();
        }
        // 4. i-th miss takes the i-th candidate
        for (int i = tid; i < n_miss; i += DIFF_THREADS) {
            const int j = s_miss[i];
            const int slot = static_cast<int>(keys[i] & 0xffffffffull);
            const int old = slot_block[slot];
            if (old >= 0 && old < p.max_blocks) table[old] = -1;
            table[s_sel[j]] = slot;
            slot_block[slot] = s_sel[j];
            s_slot[j] = slot;
        }
        __syncthreads();
    } else if (too_small && tid == 0) {
        pi_report(p.st, PI_ERR_POOL_TOO_SMALL, PI_STAGE_DIFF, seq, n_miss, s_ncand);
    }

    // 5. stamps and the slot of every selected block
    int32_t* sel_slots = p.sel_slots + static_cast<size_t>(seq) * p.K;
    for (int j = tid; j < p.K; j += DIFF_THREADS) {
        int slot = -1;
        if (j < cnt) {
            slot = s_slot[j];
            if (slot >= 0 && !too_small) slot_stamp[slot] = step;
        }
        sel_slots[j] = slot;
    }

    // 6. recall list: heads of runs consecutive in block and in slot
    pi_extent* list = p.list + static_cast<size_t>(seq) * p.K;
    int n_ext = 0;
    if (!too_small) {
        for (int i0 = 0; i0 < n_miss; i0 += DIFF_THREADS) {
            const int i = i0 + tid;
            bool head = false;
            if (i < n_miss) {
                const int j = s_miss[i];
                head = true;
                if (i > 0) {
                    const int jp = s_miss[i - 1];
                    head = !(s_sel[jp] + 1 == s_sel[j] && s_slot[jp] + 1 == s_slot[j]);
                }
            }
            const int pos = ordered_pos(head, n_ext, warp_tot);
            if (head) {
                int len = 1;
                while (i + len < n_miss) {
                    const int a = s_miss[i + len - 1], b = s_miss[i + len];
                    if (s_sel[a] + 1 == s_sel[b] && s_slot[a] + 1 == s_slot[b]) ++len; else break;
                }
                pi_extent e;
                e.src_unit = s_sel[s_miss[i]];
                e.dst_unit = s_slot[s_miss[i]];
                e.n_units = len;
                e.units_before = i;
                list[pos] = e;
            }
        }
    }
    if (tid == 0) {
        p.count[seq] = n_ext;
        atomicAdd(p.stats + 0, 1ull);
        atomicAdd(p.stats + 1, static_cast<unsigned long long>(cnt));
        atomicAdd(p.stats + 2, static_cast<unsigned long long>(too_small ? 0 : n_miss));
        atomicAdd(p.stats + 3, static_cast<unsigned long long>(n_ext));
    }
}

}  // namespace

int pi_launch_diff(pi_ctx* c, int batch, uint32_t step, const uint32_t* step_dev, const int32_t* ctx_len, const int32_t* sel,
                   const int32_t* sel_count, int32_t* table, int32_t* slot_block, uint32_t* slot_stamp,
                   int32_t* sel_slots, pi_extent* list, int32_t* count, cudaStream_t stream) {
    DiffParams p;
    p.ctx_len = ctx_len; p.sel = sel; p.sel_count = sel_count;
    p.table = table; p.slot_block = slot_block; p.slot_stamp = slot_stamp;
    p.sel_slots = sel_slots; p.list = list; p.count = count;
    p.st = pi_status_of(c);
    p.stats = c->stats_dev;
    p.step = step;
    p.step_dev = step_dev;
    p.B = c->cfg.block_tokens; p.K = c->cfg.budget_blocks; p.C = c->cfg.pool_slots;
    int cpad = 2;
    while (cpad < p.C) cpad <<= 1;
    p.Cpad = cpad;
    p.n_sink = c->cfg.n_sink_blocks; p.n_local = c->cfg.n_local_blocks; p.max_blocks = c->cfg.max_blocks;
    const size_t smem = static_cast<size_t>(cpad) * 8 + static_cast<size_t>(p.K) * 12 + static_cast<size_t>(p.C);
    if (smem > 40 * 1024)
        PI_CUDA_TRY(cudaFuncSetAttribute(diff_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    PI_CUDA_TRY(pi_launch_pdl(diff_kernel, dim3(batch), dim3(DIFF_THREADS), smem, stream, p));
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
