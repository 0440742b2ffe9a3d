// Digest scoring of the retrieval head + exact top-k block selection (Sec. 2.2 step 1 with the shared
// single-head selection of Sec. 4.4.1) and, in the fused form, the miss diff (step 2) in one launch.
//
// One thread-block cluster per sequence.  Every CTA of the cluster scores an equal share of the
// sequence's blocks (HBM-bound: 512 B of digest per block, 16 independent 16-byte loads per lane
// in flight) and writes the order-preserving keys of its fp32 scores straight into the shared
// memory of the cluster's first CTA (distributed shared memory; the scores never make a round
// trip through global memory and no ticket or fence is needed).  After one cluster barrier that CTA
// holds all keys of the sequence and selects; in the fused form it goes on to diff the selection,
// which is still in its shared memory, against the block table.  What the diff needs besides the
// selection (the sequence's slot arrays and its table row) is fetched with asynchronous copies
// while the scoring loads are in flight, so that no global round trip is left between the steps.
// The cluster's other CTAs, idle once their keys are delivered, meanwhile work out the order in
// which the pool's slots would be evicted (least recently selected first) and hand it to the first
// CTA through its shared memory and an mbarrier: the victims of the diff are then the first
// evictable slots of that order instead of a second top-k by the one CTA that is already the
// launch's critical path.
#include "pi_common.cuh"
#include "pi_block_select.cuh"
#include "pi_diff_core.cuh"
#include "pi_score_core.cuh"

namespace {

using pi_score::BLOCKS_PER_WARP;
using pi_score::padded;

// 256 threads and two CTAs per SM: clusters of 8 CTAs then find room in any group of 4 SMs, so 16 and more
// of them are resident at once (with one 512-thread CTA per SM only 15 clusters of 8 fit a B200, and a 16th
// sequence would wait for a whole cluster to finish)
#ifndef SD_THREADS_OVERRIDE
#define SD_THREADS_OVERRIDE 256
#endif
constexpr int SD_THREADS = SD_THREADS_OVERRIDE;
constexpr bool SD_TWO_SETS = SD_THREADS <= 256;            // two register sets of loads per lane (else one)
constexpr int SD_WARPS = SD_THREADS / 32;
constexpr int SD_CHUNK = SD_WARPS * BLOCKS_PER_WARP;      // 64 blocks (32 KB of digests); a CTA loads two chunks a round
// chunks a sequence must have before it gets a cluster of 16 CTAs (below four chunks per CTA the extra CTAs
// gain nothing: measured at 32 chunks)
#ifndef SD_CL16_MIN_CHUNKS
#define SD_CL16_MIN_CHUNKS 64
#endif
constexpr int SD_MAX_CLUSTER = 16;                        // 16 is beyond the portable cluster size: taken only where the device holds enough of them
constexpr size_t SD_SMEM_LIMIT = 200 * 1024;              // dynamic shared memory the kernel may ask for

struct SDParams {
    const __nv_bfloat16* q;
    const uint4* digest;
    const int32_t* ctx_len;
    int32_t* sel;
    int32_t* sel_count;
    float* scores;                 // may be null: the scores then never leave the chip
    pi_status_ref st;
    int h_star, Hq, G, B, K, n_sink, n_local, max_blocks;
    int cpc;                       // chunks of SD_CHUNK blocks per CTA
    // the diff of the fused form
    int32_t* table;
    int32_t* slot_block;
    uint32_t* slot_stamp;
    int32_t* sel_slots;
    pi_extent* list;
    int32_t* count;
    unsigned long long* stats;
    const uint32_t* step_dev;
    uint32_t step;
    int C, Cpad, table_in_smem;
    unsigned key_bytes;            // bytes of the key region at the start of the dynamic shared memory
    // eviction order prepared by the cluster's second CTA while the first one selects (fused form, clusters of 2+)
    int lru_help;
    unsigned order_off;            // byte offset of the order array (uint16 [C]) in the first CTA's dynamic shared memory
    long long wait_cycles;
};

__device__ __forceinline__ unsigned cluster_ctarank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ unsigned cluster_nctarank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// shared-memory address of the same variable in the cluster's CTA `rank`
__device__ __forceinline__ uint32_t map_shared_rank(const void* p, unsigned rank) {
    uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(p)), r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_shared_cluster(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void st_shared_cluster_u16(uint32_t addr, unsigned short v) {
    asm volatile("st.shared::cluster.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem))), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem))), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

template <bool FUSED>
__global__ void __launch_bounds__(SD_THREADS, 2)
score_select_cluster_kernel(SDParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ pi_select::Scratch<SD_WARPS> sc;
    __shared__ int warp_tot[2 * SD_WARPS];
    __shared__ int s_ncand;
    __shared__ uint32_t s_mm[2 * SD_MAX_CLUSTER * SD_WARPS];       // first CTA: every scoring warp's smallest and largest middle key
    __shared__ __align__(8) unsigned long long s_lru_bar;          // first CTA: the second CTA arrives here when the eviction order is written

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned rank = cluster_ctarank(), CL = cluster_nctarank();
    const int seq = blockIdx.x / CL;
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw);
    // every CTA of the cluster has started once all have arrived here: from then on the first CTA's
    // shared memory may be written from outside
    cluster_arrive_relaxed();
    pi_grid_dependency_wait();
    pi_launch_dependents();

    pi_diff::Smem m;
    int32_t* s_table = nullptr;
    if (FUSED) {
        m = pi_diff::carve(smem_raw + p.key_bytes, p.K, p.C);
        s_table = reinterpret_cast<int32_t*>(smem_raw + p.key_bytes + pi_diff::smem_lists_bytes(p.K, p.C));
    }
    // ---------------- scoring: this CTA's share of the sequence, two chunks (16 loads per lane) a round
    const int blk_lo = static_cast<int>(rank) * p.cpc * SD_CHUNK;
    const uint4* dg = p.digest + static_cast<size_t>(seq) * p.max_blocks * 32;        // 32 uint4 per block
    const uint32_t keys_remote = map_shared_rank(keys, 0);
    float w[8];
    int n_blocks = 0, m_lo = 0, m_hi = 0;
    uint32_t kmin = 0xffffffffu, kmax = 0u;            // extremes of this lane's keys of middle blocks
    // Two register sets of 8 loads per lane, refilled in turn: while one chunk is reduced, the loads of the
    // next are already in flight (8 to 16 independent 16-byte loads per lane at any time).  Digest rows up
    // to max_blocks are allocated, so they are read whatever the sequence's length and masked afterwards.
    uint4 va[BLOCKS_PER_WARP], vb[BLOCKS_PER_WARP];
    const unsigned long long stream_policy = pi_l2_stream_policy();
    auto issue = [&](uint4 (&v)[BLOCKS_PER_WARP], int c) {
        const int b0 = blk_lo + c * SD_CHUNK + warp * BLOCKS_PER_WARP;
#pragma unroll
        for (int i = 0; i < BLOCKS_PER_WARP; ++i) {
            v[i] = make_uint4(0, 0, 0, 0);
            if (c < p.cpc && b0 + i < p.max_blocks) v[i] = pi_score::ld_stream16(dg + static_cast<size_t>(b0 + i) * 32 + lane, stream_policy);
        }
    };
    auto finish = [&](uint4 (&v)[BLOCKS_PER_WARP], int c) {
        float s[BLOCKS_PER_WARP];
#pragma unroll
        for (int i = 0; i < BLOCKS_PER_WARP; ++i) s[i] = pi_score::dot8(v[i], w);
        pi_score::reduce8(s, lane);
        const int b = blk_lo + c * SD_CHUNK + warp * BLOCKS_PER_WARP + (lane >> 2);
        if ((lane & 3) == 0 && b < p.max_blocks) {
            const uint32_t key = pi_score::float_key(s[0]);
            st_shared_cluster(keys_remote + static_cast<uint32_t>(padded(b)) * 4u, key);
            if (b >= m_lo && b < m_hi) { kmin = min(kmin, key); kmax = max(kmax, key); }
            if (p.scores && b < n_blocks) p.scores[static_cast<size_t>(seq) * p.max_blocks + b] = s[0];
        }
    };
    issue(va, 0);
    if (SD_TWO_SETS) issue(vb, 1);
    // The first loads of the digests are in flight; what else the launch needs is set up behind them.
    if (rank == 0) {
        pi_select::clear<SD_THREADS>(sc);
        // The rows this CTA writes at the very end are touched now: the address translation of a page an SM has
        // not used yet takes a microsecond or two, and at the end of the launch nothing would hide it.
        if (tid < 8) {
            const void* row = nullptr;
            switch (tid) {
                case 0: row = p.sel + static_cast<size_t>(seq) * p.K; break;
                case 1: row = p.sel_count + seq; break;
                case 2: row = FUSED ? static_cast<const void*>(p.sel_slots + static_cast<size_t>(seq) * p.K) : nullptr; break;
                case 3: row = FUSED ? static_cast<const void*>(p.list + static_cast<size_t>(seq) * p.K) : nullptr; break;
                case 4: row = FUSED ? static_cast<const void*>(p.count + seq) : nullptr; break;
                case 5: row = FUSED ? static_cast<const void*>(p.stats) : nullptr; break;
                case 6: row = p.scores ? static_cast<const void*>(p.scores + static_cast<size_t>(seq) * p.max_blocks) : nullptr; break;
                default: row = FUSED ? static_cast<const void*>(p.step_dev) : nullptr; break;
            }
            if (row) asm volatile("prefetch.global.L2 [%0];" ::"l"(row));
        }
        if (FUSED) {
            // what the diff needs besides the selection, fetched while the digests stream in
            const int32_t* sb = p.slot_block + static_cast<size_t>(seq) * p.C;
            const uint32_t* stp = p.slot_stamp + static_cast<size_t>(seq) * p.C;
            for (int s = tid; s < p.C; s += SD_THREADS) {
                cp_async4(m.sb + s, sb + s);
                cp_async4(m.stp + s, stp + s);
                m.used[s] = 0;
            }
            if (p.table_in_smem) {
                const int32_t* row = p.table + static_cast<size_t>(seq) * p.max_blocks;
                if (((reinterpret_cast<uintptr_t>(row) | reinterpret_cast<uintptr_t>(s_table)) & 15) == 0 && (p.max_blocks & 3) == 0) {
                    for (int b = tid * 4; b < p.max_blocks; b += SD_THREADS * 4) cp_async16(s_table + b, row + b);
                } else {
                    for (int b = tid; b < p.max_blocks; b += SD_THREADS) cp_async4(s_table + b, row + b);
                }
            }
            if (tid == 0) s_ncand = 0;
            if (tid == 0 && p.lru_help) {
                asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(&s_lru_bar))), "r"(CL - 1u));
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            }
        }
    } else if (FUSED && p.lru_help) {
        // the stamps of all slots, for the eviction order the other CTAs work out after their share of the scoring
        // (their own dynamic shared memory is free: the keys go to the first CTA)
        uint32_t* st = reinterpret_cast<uint32_t*>(smem_raw + static_cast<size_t>((p.C + 1) & ~1) * 8);
        const uint32_t* stp = p.slot_stamp + static_cast<size_t>(seq) * p.C;
        for (int s = tid; s < p.C; s += SD_THREADS) cp_async4(st + s, stp + s);
    }
    {
        pi_score::load_q_weights(p.q + (static_cast<size_t>(seq) * p.Hq + static_cast<size_t>(p.h_star) * p.G) * PI_HEAD_DIM,
                                 p.G, lane, w);
        int ctx = p.ctx_len[seq];
        if (ctx < 0) ctx = 0;
        n_blocks = (ctx + p.B - 1) / p.B;
        if (n_blocks > p.max_blocks) {
            if (tid == 0 && rank == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_SELECT, seq, n_blocks, p.max_blocks);
            n_blocks = p.max_blocks;
        }
        m_lo = min(p.n_sink, n_blocks);
        m_hi = max(n_blocks - p.n_local, m_lo);
    }
    cluster_wait_acquire();                            // completes the start-up barrier: all CTAs are running
    if (SD_TWO_SETS) {
        for (int c = 0; c < p.cpc; c += 2) {
            finish(va, c);
            issue(va, c + 2);
            if (c + 1 < p.cpc) finish(vb, c + 1);
            issue(vb, c + 3);
        }
    } else {
        for (int c = 0; c < p.cpc; ++c) {
            finish(va, c);
            issue(va, c + 1);
        }
    }
    // the extremes travel with the keys: the selecting CTA then needs no pass of its own to find them
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) {
        const uint32_t mm_remote = map_shared_rank(s_mm, 0) + (rank * SD_WARPS + warp) * 8u;
        st_shared_cluster(mm_remote, kmin);
        st_shared_cluster(mm_remote + 4u, kmax);
    }
    if (FUSED && (rank == 0 || p.lru_help)) cp_async_wait_all();
    // all keys of the sequence are in the first CTA's shared memory once every CTA has arrived
    cluster_arrive_release();
    cluster_wait_acquire();
    if (FUSED && rank != 0 && p.lru_help) {
        // ---------------- eviction order for the first CTA's diff, worked out while that CTA selects: position of
        // slot s = number of slots before it in (stamp, slot) order, by counting.  The CL - 1 other CTAs take every
        // (CL - 1)-th slot each; four lanes share the comparisons of one slot.  The positions go straight into the
        // first CTA's shared memory, then every CTA arrives once on its mbarrier.
        __syncthreads();                                   // every thread's share of the stamps has landed
        const int Cq = (p.C + 1) & ~1;
        unsigned long long* k64 = reinterpret_cast<unsigned long long*>(smem_raw);
        const uint32_t* st = reinterpret_cast<const uint32_t*>(smem_raw + static_cast<size_t>(Cq) * 8);
        for (int u = tid; u < Cq; u += SD_THREADS)
            k64[u] = u < p.C ? ((static_cast<unsigned long long>(st[u]) << 32) | static_cast<unsigned>(u)) : ~0ull;
        __syncthreads();
        const uint32_t order_remote = map_shared_rank(smem_raw + p.order_off, 0);
        const int parts = static_cast<int>(CL) - 1, part = static_cast<int>(rank) - 1;
        const int n_mine = (p.C - part + parts - 1) / parts;                  // slots part, part + parts, ...
        const int qd = tid & 3, pairs = Cq >> 1;
        for (int i0 = 0; i0 < n_mine; i0 += SD_THREADS / 4) {
            const int i = i0 + (tid >> 2);
            const int s = part + i * parts;
            const unsigned long long mine = i < n_mine ? k64[s] : 0ull;
            int before = 0;
#pragma unroll 4
            for (int u2 = qd; u2 < pairs; u2 += 4) {
                const ulonglong2 v = reinterpret_cast<const ulonglong2*>(k64)[u2];
                before += (v.x < mine ? 1 : 0) + (v.y < mine ? 1 : 0);
            }
            before += __shfl_xor_sync(0xffffffffu, before, 1);
            before += __shfl_xor_sync(0xffffffffu, before, 2);
            if (qd == 0 && i < n_mine)
                st_shared_cluster_u16(order_remote + 2u * static_cast<uint32_t>(before), static_cast<unsigned short>(s));
        }
        __syncthreads();
        if (tid == 0) {
            const uint32_t bar_remote = map_shared_rank(&s_lru_bar, 0);
            asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_remote) : "memory");
        }
        return;
    }
    if (rank != 0) return;

    // ---------------- selection: sink and local blocks always, the k_mid best middle blocks, ties to the lower index
    const int k_mid = p.K - p.n_sink - p.n_local;
    const unsigned k = static_cast<unsigned>(max(0, min(k_mid, m_hi - m_lo)));
    {
        uint32_t a = 0xffffffffu, b = 0u;
        for (int i = lane; i < static_cast<int>(CL) * SD_WARPS; i += 32) { a = min(a, s_mm[2 * i]); b = max(b, s_mm[2 * i + 1]); }
        kmin = __reduce_min_sync(0xffffffffu, a);
        kmax = __reduce_max_sync(0xffffffffu, b);
    }
    int32_t* out = p.sel + static_cast<size_t>(seq) * p.K;
    unsigned n_sel = pi_select::block_topk_emit<SD_THREADS, true, false, true>(keys, n_blocks, m_lo, m_hi, k, sc, true, kmin, kmax,
                                                                              [&](unsigned pos, int i, uint32_t) {
        if (pos < static_cast<unsigned>(p.K)) {
            out[pos] = i;
            if (FUSED) m.sel[pos] = i;
        }
    });
    n_sel = min(n_sel, static_cast<unsigned>(p.K));
    for (int i = n_sel + tid; i < p.K; i += SD_THREADS) out[i] = -1;
    if (tid == 0) p.sel_count[seq] = static_cast<int32_t>(n_sel);
    if (!FUSED) return;

    // ---------------- diff of the selection that is still in shared memory
    // (every warp has passed the barrier inside the emission, so nobody reads the histogram any more)
    pi_select::clear<SD_THREADS>(sc);
    pi_diff::SeqArgs a;
    a.step = p.step_dev ? *p.step_dev : p.step;
    a.n_blocks = n_blocks;
    a.cnt = static_cast<int>(n_sel);
    a.seq = seq; a.K = p.K; a.C = p.C; a.Cpad = p.Cpad; a.n_sink = p.n_sink; a.n_local = p.n_local; a.max_blocks = p.max_blocks;
    a.table = p.table + static_cast<size_t>(seq) * p.max_blocks;
    a.slot_block = p.slot_block + static_cast<size_t>(seq) * p.C;
    a.slot_stamp = p.slot_stamp + static_cast<size_t>(seq) * p.C;
    a.sel_slots = p.sel_slots + static_cast<size_t>(seq) * p.K;
    a.list = p.list + static_cast<size_t>(seq) * p.K;
    a.count = p.count + seq;
    a.stats = p.stats; a.st = p.st;
    m.keys = keys;                                     // the score keys are dead: their region holds the victim keys now
    m.table_s = p.table_in_smem ? s_table : nullptr;
    m.warp_tot = warp_tot;
    m.n_cand = &s_ncand;
    if (p.lru_help && CL >= 2) {
        m.lru_order = reinterpret_cast<const unsigned short*>(smem_raw + p.order_off);
        m.lru_bar = static_cast<uint32_t>(__cvta_generic_to_shared(&s_lru_bar));
        m.lru_wait = p.wait_cycles;
    }
    __syncthreads();
    pi_diff::diff_sequence<SD_THREADS>(a, m, sc);
    if (p.lru_help && CL >= 2 && tid == 0) {
        // The second CTA writes the eviction order into this CTA's shared memory whether or not the diff needed it
        // (no misses, or too many for the ranked path): this CTA stays until that CTA has arrived.
        const long long t0 = clock64();
        uint32_t done = 0;
        while (!done && clock64() - t0 <= p.wait_cycles)
            asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                         : "=r"(done) : "r"(m.lru_bar), "r"(0u) : "memory");
        if (!done) pi_report(p.st, PI_ERR_TIMEOUT, PI_STAGE_DIFF, seq, 0, 0);
    }
}

// Clusters of `cluster` CTAs of this kernel that the device holds at once (0 if the query fails).
template <class Kernel>
int resident_clusters(Kernel kern, int cluster, size_t smem) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(cluster);
    lc.blockDim = dim3(SD_THREADS);
    lc.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &lc) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

}  // namespace

int pi_launch_select_cluster(pi_ctx* c, int h_star, int batch, const void* q, const void* digest, const int32_t* ctx_len,
                             int32_t* sel, int32_t* sel_count, float* scores, int fused, uint32_t step,
                             const uint32_t* step_dev, int32_t* table, int32_t* slot_block, uint32_t* slot_stamp,
                             int32_t* sel_slots, pi_extent* list, int32_t* count, cudaStream_t stream) {
    const pi_config& cfg = c->cfg;
    SDParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.digest = static_cast<const uint4*>(digest);
    p.ctx_len = ctx_len;
    p.sel = sel; p.sel_count = sel_count; p.scores = scores;
    p.st = pi_status_of(c);
    p.h_star = h_star;
    p.Hq = cfg.n_q_heads; p.G = cfg.n_q_heads / cfg.n_kv_heads; p.B = cfg.block_tokens; p.K = cfg.budget_blocks;
    p.n_sink = cfg.n_sink_blocks; p.n_local = cfg.n_local_blocks; p.max_blocks = cfg.max_blocks;
    p.table = table; p.slot_block = slot_block; p.slot_stamp = slot_stamp; p.sel_slots = sel_slots;
    p.list = list; p.count = count; p.stats = c->stats_dev; p.step = step; p.step_dev = step_dev;
    p.C = cfg.pool_slots;
    int cpad = 2;
    while (cpad < p.C) cpad <<= 1;
    p.Cpad = cpad;

    // shared memory: the key region (score keys; in the fused form later the victim keys), then the diff's lists,
    // then a copy of the table row when it still fits
    size_t key_bytes = ((static_cast<size_t>(cfg.max_blocks) + cfg.max_blocks / 32 + 1) * 4 + 15) & ~size_t(15);
    size_t smem = key_bytes;
    p.table_in_smem = 0;
    if (fused) {
        const size_t dk = pi_diff::smem_keys_bytes(p.C, p.Cpad);
        if (dk > key_bytes) key_bytes = dk;
        smem = key_bytes + pi_diff::smem_lists_bytes(p.K, p.C);
        const size_t row = static_cast<size_t>(cfg.max_blocks) * 4;
        if (smem + row <= SD_SMEM_LIMIT) { p.table_in_smem = 1; smem += row; }
    }
    p.key_bytes = static_cast<unsigned>(key_bytes);
    // room for the eviction order (uint16 per slot) the second CTA of a cluster hands to the first
    p.lru_help = 0; p.order_off = 0; p.wait_cycles = c->wait_limit_cycles;
    const bool order_room = fused && p.C <= 1024 && smem + 2 * static_cast<size_t>(p.C) + 16 <= SD_SMEM_LIMIT;
    if (order_room) {
        p.order_off = static_cast<unsigned>((smem + 15) & ~size_t(15));
        smem = p.order_off + 2 * static_cast<size_t>(p.C);
    }
    auto kern = fused ? score_select_cluster_kernel<true> : score_select_cluster_kernel<false>;
    if (smem > 36 * 1024)
        PI_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    // Cluster size: the largest power of two <= 16 that leaves no CTA without blocks and lets the clusters of all
    // sequences be resident at once (a cluster that has to wait for another one to finish doubles the
    // latency of the call); what the device holds is asked once per shape and kept.
    const int n_chunks = (cfg.max_blocks + SD_CHUNK - 1) / SD_CHUNK;
    int* resident = c->sd_resident_clusters[fused ? 1 : 0];
    int cluster = 1;
    for (int log2c = 4; log2c >= 1; --log2c) {
        const int cl = 1 << log2c;
        if (cl > n_chunks) continue;                               // more CTAs than chunks
        // a cluster of 16 only for long sequences: below four chunks per CTA the extra CTAs of a sequence gain nothing
        if (cl == 16 && n_chunks < SD_CL16_MIN_CHUNKS) continue;
        if (resident[log2c] < 0) {
            if (cl == 16 && cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
                (void)cudaGetLastError();
                resident[log2c] = 0;
            } else {
                resident[log2c] = resident_clusters(kern, cl, smem);
            }
        }
        if (batch <= resident[log2c]) { cluster = cl; break; }
    }
    p.cpc = (n_chunks + cluster - 1) / cluster;
    p.lru_help = (order_room && cluster >= 2) ? 1 : 0;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(batch * cluster);
    lc.blockDim = dim3(SD_THREADS);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // one CTA per SM where there is room: two streaming CTAs on one SM share its path to L2
    attr[1].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
    attr[1].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicySpread;
    lc.attrs = attr;
    lc.numAttrs = 2;
    PI_CUDA_TRY(cudaLaunchKernelEx(&lc, kern, p));
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
