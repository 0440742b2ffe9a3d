// Sparse GQA decode attention, head-major form: one work item is one (sequence, KV head); a persistent
// CTA takes items c, c + grid, ... and streams the item's selected blocks through a ring of shared-memory
// stages.  A stage holds eight 16-token tiles of that one head (K and V rows: 8 KB each, fetched by two
// tiled TMA loads with 128-byte swizzle), one tile per consumer warp; every warp keeps its own online-
// softmax state for the head's G query heads, and at the end of the item the eight states are merged
// through shared memory in a fixed tree and the result is written out.
//
// Compared with the flat split over all KV heads (pi_attn.cu) nothing leaves the CTA: no fp32 partials in
// global memory and no second kernel, which is where the flat form loses its time at decode shapes
// (tail + merge + second launch).  CTAs working on the heads of one sequence read neighbouring 8 KB
// fragments of the same blocks at about the same time.  The form needs (sequences x KV heads) to fill the
// grid evenly; the launcher falls back to the flat split when it does not.  With fewer items than half the
// grid, an item is shared by a cluster of 2 or 4 CTAs that take its stages in turn; the first CTA of the
// cluster reads the others' final states out of their shared memory (distributed shared memory, plain
// loads) and writes the result.  The same kernel serves per-head selections (the headwise strategy of
// Sec. 4.4.1): item (s, h) then walks list (s, h).
//
// Split around the recall (PHASE 1 and 2): the blocks of a selection that were resident before the step do
// not depend on the recall (the diff never evicts a selected block), so their share of the attention can run
// while the missing blocks are still on their way.  PHASE 1 walks the selected blocks whose slot is not a
// destination of the step's recall list and leaves the merged softmax state of every item in global memory;
// PHASE 2 walks the others (a handful per sequence), folds that state in and writes the result.  Both build
// the set of slots being filled from the recall list itself (a bitmap per item in shared memory) and compact
// their units in selection order, so the split is a function of the lists alone.
#include "pi_common.cuh"
#include "pi_attn_core.cuh"

using namespace pi_attn;

namespace {

constexpr int HM_WARPS = 8;                        // consumer warps = tiles per stage
constexpr int HM_STAGE_BYTES = HM_WARPS * 8192;    // 64 KB
constexpr int HM_HALF_BYTES = HM_WARPS * 4096;
constexpr int HM_META_UNITS = 1024;                // units per CTA whose metadata is staged in shared memory

__device__ __forceinline__ void named_barrier_consumers() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ unsigned cluster_ctarank() { unsigned r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ unsigned cluster_nctarank() { unsigned r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_shared_cluster_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t map_shared_rank(uint32_t addr, unsigned rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

template <int NT, int PHASE>
__global__ void __launch_bounds__(288, 1)
attn_headmajor_kernel(const __grid_constant__ CUtensorMap pool_map, AttnParams p, int n_items, int items_per_cta) {
    extern __shared__ unsigned char smem_dyn[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t ring = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* after_ring = smem_dyn + (ring - smem_u32(smem_dyn)) + static_cast<size_t>(p.stages) * HM_STAGE_BYTES;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(after_ring);      // full[8], empty[8]
    int* s_nvalid = reinterpret_cast<int*>(bars + 2 * ATTN_MAX_STAGES);                // [8 stages][8 tiles]
    int* s_abort = s_nvalid + ATTN_MAX_STAGES * 8;
    int2* s_meta = reinterpret_cast<int2*>(s_abort + 2);                               // [HM_META_UNITS] {slot row, token offset | nvalid << 8}
    int* s_units = reinterpret_cast<int*>(s_meta + HM_META_UNITS);                     // [items_per_cta + 1] units before each of my items
    float* s_merge = reinterpret_cast<float*>(s_units + ((items_per_cta + 2 + 3) & ~3)); // [4][NT * 36][32]
    unsigned* s_fresh = reinterpret_cast<unsigned*>(s_merge + 4 * NT * 36 * 32);         // PHASE: [items_per_cta][ceil(C / 32)] slots being filled
    const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + ATTN_MAX_STAGES);
    const int SUB = p.B >> 4;
    if (tid == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&pool_map) : "memory");
    pi_grid_dependency_wait();
    pi_launch_dependents();

    // ---- my items and their unit counts (a cluster of S CTAs shares its items: CTA `rank` takes every S-th stage)
    const int S = static_cast<int>(cluster_nctarank()), rank = static_cast<int>(cluster_ctarank());
    const int first_item = blockIdx.x / S, stride = gridDim.x / S;
    int n_mine = 0;
    for (int it = first_item; it < n_items; it += stride) ++n_mine;
    auto list_of = [&](int item) -> int { return p.headwise ? item : item / p.Hkv; };
    // ---- metadata of my units: global row of the slot, token offset, valid tokens.  Staged by all threads in ONE
    // round of independent loads (list entries up to K are read whatever the list's length: the tail holds -1),
    // so that the producer never waits on a dependent global load.  Unit r of my k-th item sits at k * upi + r.
    const int upi = p.K * SUB;                             // units an item can have
    auto unit_meta = [&](int k, int r) -> int2 {
        const int item = first_item + k * stride, seq = item / p.Hkv;
        const size_t list = static_cast<size_t>(list_of(item));
        const int j = r / SUB, sub = r - j * SUB;
        int slot = p.sel_slots[list * p.K + j];
        const int blk = p.sel_blocks[list * p.K + j];
        const int ctx = p.ctx_len[seq], cnt = p.sel_count[list];
        const bool listed = cnt >= 0 && cnt <= p.K && j < cnt && blk >= 0;
        bool bad = false;
        if (slot < 0 || slot >= p.C) {
            if (listed) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_ATTN, seq, j, slot);
            slot = 0; bad = true;
        }
        const int nvalid = (!listed || bad) ? 0 : max(0, min(16, ctx - (blk * p.B + sub * 16)));
        return make_int2(seq * p.C + slot, (sub * 16) | (nvalid << 8));
    };
    if (PHASE == 0) {
        for (int i = tid; i < n_mine * upi && i < HM_META_UNITS; i += blockDim.x) {
            const int k = i / upi;
            s_meta[i] = unit_meta(k, i - k * upi);
        }
    } else {
        // slots the step's recall fills, per item; then the kept units of every item, compacted in selection order
        // (the launcher has checked that all of a CTA's units fit the staged metadata)
        const int words = (p.C + 31) >> 5;
        for (int i = tid; i < n_mine * words; i += blockDim.x) s_fresh[i] = 0u;
        __syncthreads();
        for (int k = 0; k < n_mine; ++k) {
            const int seq = (first_item + k * stride) / p.Hkv;
            int n = p.rcount[seq];
            if (n < 0 || n > p.rcap) n = 0;                 // (the recall kernel reports such a count)
            for (int e = tid; e < n; e += blockDim.x) {
                const pi_extent x = p.rlist[static_cast<size_t>(seq) * p.rcap + e];
                // (an extent that leaves the pool is the recall kernel's to report; here it is clipped, which also
                // bounds the loop whatever the list holds)
                if (x.dst_unit < 0 || x.dst_unit >= p.C) continue;
                const int nu = min(x.n_units, p.C - x.dst_unit);
                for (int u = 0; u < nu; ++u) {
                    const int slot = x.dst_unit + u;
                    atomicOr(&s_fresh[k * words + (slot >> 5)], 1u << (slot & 31));
                }
            }
        }
        __syncthreads();
        for (int k = warp; k < n_mine; k += HM_WARPS + 1) {
            const int item = first_item + k * stride, seq = item / p.Hkv;
            int cnt = p.sel_count[seq];
            if (cnt < 0 || cnt > p.K) cnt = 0;              // reported below
            const int ctx = p.ctx_len[seq];
            int kept = 0;
            for (int base = 0; base < cnt; base += 32) {
                const int j = base + lane;
                bool keep = false;
                int slot = 0, blk = -1;
                if (j < cnt) {
                    slot = p.sel_slots[static_cast<size_t>(seq) * p.K + j];
                    blk = p.sel_blocks[static_cast<size_t>(seq) * p.K + j];
                    if (slot < 0 || slot >= p.C) {
                        if (blk >= 0 && PHASE == 1) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_ATTN, seq, j, slot);
                    } else if (blk >= 0) {
                        const bool fresh = (s_fresh[k * words + (slot >> 5)] >> (slot & 31)) & 1u;
                        keep = fresh == (PHASE == 2);
                    }
                }
                const unsigned b = __ballot_sync(0xffffffffu, keep);
                if (keep) {
                    const int pos = kept + __popc(b & ((1u << lane) - 1u));
                    for (int sub = 0; sub < SUB; ++sub) {
                        const int nvalid = max(0, min(16, ctx - (blk * p.B + sub * 16)));
                        s_meta[k * upi + pos * SUB + sub] = make_int2(seq * p.C + slot, (sub * 16) | (nvalid << 8));
                    }
                }
                kept += __popc(b);
            }
            if (lane == 0) s_units[k + 1] = kept * SUB;       // turned into a running sum below
        }
        __syncthreads();
    }
    if (tid == 0) {
        int run = 0;
        for (int k = 0; k < n_mine; ++k) {
            const int item = first_item + k * stride;
            int n = p.sel_count[list_of(item)];
            if (n < 0 || n > p.K) { if (PHASE != 2) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_ATTN, item / p.Hkv, n, p.K); n = 0; }
            const int units = PHASE == 0 ? n * SUB : s_units[k + 1];
            s_units[k] = run;
            run += units;
        }
        s_units[n_mine] = run;
        *s_abort = 0;
        for (int i = 0; i < p.stages; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, HM_WARPS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int total_units = s_units[n_mine];

    if (warp == HM_WARPS) {
        // =============================== producer warp: a stage = up to 8 tiles of one item.  Lane 0 waits for the
        // stage to be free and announces the bytes; lanes 0..15 then issue one TMA load each (tile lane / 2, half
        // lane % 2 of the head dimension), so that a stage's sixteen loads go out together.
        int sidx = 0;
        bool alive = true;
        const int w = lane >> 1, half = lane & 1;
        const unsigned long long stream_policy = pi_l2_stream_policy();
        for (int k = 0; k < n_mine && alive; ++k) {
            const int item = first_item + k * stride, h = item % p.Hkv;
            const int n_u = s_units[k + 1] - s_units[k];
            for (int g = rank * HM_WARPS; g < n_u; g += HM_WARPS * S, ++sidx) {
                const int st = sidx % p.stages, round = sidx / p.stages;
                int ok = 1;
                if (lane == 0) {
                    if (round > 0 && !mbar_wait(bar_empty + 8 * st, (round - 1) & 1, s_abort, p.wait_cycles)) ok = 0;
                    if (p.hold_last && k == n_mine - 1 && g + HM_WARPS * S >= n_u) ok = 0;   // (test only)
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { alive = false; break; }
                const int n_here = min(HM_WARPS, n_u - g);
                const uint32_t dst = ring + st * HM_STAGE_BYTES;
                int2 md = make_int2(0, 0);
                if (lane < 16 && w < n_here) md = (k * upi + g + w) < HM_META_UNITS ? s_meta[k * upi + g + w] : unit_meta(k, g + w);
                if (lane < 16 && half == 0) s_nvalid[st * 8 + w] = w < n_here ? (md.y >> 8) : 0;
                __syncwarp();                               // the valid-token counts are written before the arrive, which publishes them
                if (lane == 0) mbar_expect_tx(bar_full + 8 * st, static_cast<uint32_t>(n_here) * 8192u);
                __syncwarp();
                if (lane < 16 && w < n_here)
                    tma_load_4d(dst + half * HM_HALF_BYTES + w * 4096, &pool_map, bar_full + 8 * st, half * 64, md.y & 0xff, 2 * h, md.x, stream_policy);
            }
        }
        __syncwarp();
        if (S > 1) { cluster_sync_all(); cluster_sync_all(); }   // the two barriers of the cross-CTA merge below
        return;
    }

    // =============================== consumers: warp w owns tile w of every stage
    const int row = lane >> 2, colp = (lane & 3) * 2;
    const int r8 = lane & 7, mi = lane >> 3;
    const int tK = r8 + 8 * (mi & 1), cK = mi >> 1;         // K as A operand (rows = tokens)
    const int tV = r8 + 8 * (mi >> 1), cV = mi & 1;         // V^T as A operand via .trans
    const uint32_t offK = (2 * warp) * 2048 + tK * 128, offV = (2 * warp + 1) * 2048 + tV * 128;
    bool alive = true, aborted = false;
    int sidx = 0;
    float o[NT][8][4], m[NT][2], l[NT][2];
    // a region of the merge area holds one warp's state as [value][lane] (conflict-free)
    auto region = [&](int r) -> float* { return s_merge + static_cast<size_t>(r) * (NT * 36 * 32) + lane; };
    auto put = [&](float* reg) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int c = 0; c < 4; ++c) reg[((nt * 36) + i * 4 + c) * 32] = o[nt][i][c];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                reg[((nt * 36) + 32 + e) * 32] = m[nt][e];
                reg[((nt * 36) + 34 + e) * 32] = l[nt][e];
            }
        }
    };
    auto take = [&](auto load) {                            // load(i): value i of the other state
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float m2 = load((nt * 36) + 32 + e), l2 = load((nt * 36) + 34 + e);
                const float mn = fmaxf(m[nt][e], m2);
                const float a1 = m[nt][e] == -INFINITY ? 0.f : exp2f(m[nt][e] - mn);
                const float a2 = m2 == -INFINITY ? 0.f : exp2f(m2 - mn);
                m[nt][e] = mn;
                l[nt][e] = l[nt][e] * a1 + l2 * a2;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    o[nt][i][e] = o[nt][i][e] * a1 + load((nt * 36) + i * 4 + e) * a2;
                    o[nt][i][e + 2] = o[nt][i][e + 2] * a1 + load((nt * 36) + i * 4 + e + 2) * a2;
                }
            }
    };
    auto finish = [&](int seq, int h) {                     // sums of the weights over the tile rows, then the result
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float v = l[nt][e];
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                l[nt][e] = v;
            }
        attn_write_out<NT>(p, seq, h, row, colp, o, m, l);
    };
    // what an item ends with: the result (PHASE 0), its state left for the second call (PHASE 1), or the first
    // call's state folded in before the result (PHASE 2).  Called by warp 0 of the CTA that holds the item's state.
    auto conclude = [&](int item) {
        if (PHASE == 1) {
            put(p.state + static_cast<size_t>(item) * (NT * 36 * 32) + lane);
            return;
        }
        if (PHASE == 2) {
            const float* g = p.state + static_cast<size_t>(item) * (NT * 36 * 32) + lane;
            take([&](int i) { return g[i * 32]; });
        }
        finish(item / p.Hkv, item % p.Hkv);
    };
    int last_item = 0;
    for (int k = 0; k < n_mine; ++k) {
        const int item = first_item + k * stride, seq = item / p.Hkv, h = item % p.Hkv;
        const int n_u = s_units[k + 1] - s_units[k];
        last_item = item;
        uint32_t bq[NT][8][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int g = nt * 8 + row;
            const __nv_bfloat16* qg = p.q + (static_cast<size_t>(seq) * p.Hq + static_cast<size_t>(h) * p.G + g) * PI_HEAD_DIM + colp;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                bq[nt][j][0] = g < p.G ? *reinterpret_cast<const uint32_t*>(qg + 16 * j) : 0u;
                bq[nt][j][1] = g < p.G ? *reinterpret_cast<const uint32_t*>(qg + 16 * j + 8) : 0u;
            }
            m[nt][0] = m[nt][1] = -INFINITY;
            l[nt][0] = l[nt][1] = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) o[nt][i][0] = o[nt][i][1] = o[nt][i][2] = o[nt][i][3] = 0.f;
        }
        for (int g = rank * HM_WARPS; g < n_u && alive; g += HM_WARPS * S, ++sidx) {
            const int st = sidx % p.stages;
            if (!mbar_wait(bar_full + 8 * st, (sidx / p.stages) & 1, s_abort, p.wait_cycles)) { alive = false; break; }
            const int nvalid = s_nvalid[st * 8 + warp];
            if (g + warp < n_u)
                attn_tile<NT>(ring + st * HM_STAGE_BYTES, HM_HALF_BYTES, offK, offV, r8, cK, cV, row, nvalid, p.scale_log2, bq, o, m, l);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * st);
        }
        // `alive` may differ between warps for a moment (each learns of the abort at its own wait); the shared flag
        // decides, so that all eight warps take the same path through the barriers below
        named_barrier_consumers();
        if (*s_abort) { aborted = true; break; }

        // ---- the eight states are merged in a fixed tree through shared memory: 4..7 into 0..3, 2..3 into 0..1, 1 into 0
        if (warp >= 4) put(region(warp - 4));
        named_barrier_consumers();
        if (warp < 4) { const float* r = region(warp); take([&](int i) { return r[i * 32]; }); }
        named_barrier_consumers();
        if (warp == 2 || warp == 3) put(region(warp - 2));
        named_barrier_consumers();
        if (warp < 2) { const float* r = region(warp); take([&](int i) { return r[i * 32]; }); }
        named_barrier_consumers();
        if (warp == 1) put(region(0));
        named_barrier_consumers();
        if (warp == 0) {
            const float* r = region(0);
            take([&](int i) { return r[i * 32]; });
            if (S == 1) conclude(item);
        }
    }
    if (S > 1) {
        // ---- an item shared by a cluster (one item per CTA in this form): the first CTA folds the others' states in,
        // in rank order, reading them out of their shared memory
        named_barrier_consumers();                          // warp 0 has read region 0 for the last time
        if (warp == 0 && rank != 0 && !aborted) put(region(0));
        cluster_sync_all();
        if (warp == 0 && rank == 0 && !aborted) {
            const uint32_t mine = smem_u32(region(0));
            for (int r = 1; r < S; ++r) {
                const uint32_t theirs = map_shared_rank(mine, static_cast<unsigned>(r));
                take([&](int i) { return ld_shared_cluster_f32(theirs + static_cast<uint32_t>(i) * 128u); });
            }
            conclude(last_item);
        }
        cluster_sync_all();                                 // nobody leaves while its state may still be read
    }
    if (*s_abort && lane == 0 && warp == 0) pi_report(p.st, PI_ERR_TIMEOUT, PI_STAGE_ATTN, blockIdx.x, 0, total_units);
}

}  // namespace

// Whether the head-major form fills the attention grid well enough, and its launch shape: CTAs per item
// (cluster size 1, 2 or 4), grid, items per CTA.
bool pi_attn_headmajor_fits(const pi_ctx* c, int batch, int* grid_out, int* items_per_cta_out, int* split_out) {
    const int items = batch * c->cfg.n_kv_heads, ctas = c->attn_ctas;
    int split = 1;
    while (split < 4 && items * split * 2 <= ctas) split *= 2;    // fewer items than half the grid: 2 or 4 CTAs share one
    if (c->cfg.n_q_heads / c->cfg.n_kv_heads > 8) split = 1;     // (the wide states of G > 8 stay inside one CTA)
    const int grid = items * split <= ctas ? items * split : ctas;
    const int rounds = split > 1 ? 1 : (items + grid - 1) / grid;
    if (grid_out) *grid_out = grid;
    if (items_per_cta_out) *items_per_cta_out = rounds;
    if (split_out) *split_out = split;
    // at least three fifths of the attention grid busy (the memory system is saturated from there on), and no
    // more than a tenth of the last round idle
    return grid * 5 >= ctas * 3 && static_cast<long long>(items) * split * 10 >= static_cast<long long>(rounds) * grid * 9;
}

static size_t hm_smem_bytes(const pi_config& cfg, int per_cta, int NT, int stages, bool phased) {
    return 1024 + static_cast<size_t>(stages) * HM_STAGE_BYTES + 2 * ATTN_MAX_STAGES * 8 +
           (ATTN_MAX_STAGES * 8 + 2) * 4 + HM_META_UNITS * 8 + ((static_cast<size_t>(per_cta) + 2 + 3) & ~size_t(3)) * 4 +
           static_cast<size_t>(4) * NT * 36 * 32 * 4 + 16 +
           (phased ? static_cast<size_t>(per_cta) * ((cfg.pool_slots + 31) / 32) * 4 : 0);
}

// The split around the recall needs the head-major form with every unit of a CTA in the staged metadata.
bool pi_attn_phased_fits(const pi_ctx* c, int batch) {
    int grid = 1, per_cta = 1, split = 1;
    const bool fits = pi_attn_headmajor_fits(c, batch, &grid, &per_cta, &split);
    if (c->cfg.attn_mode == 1 || (c->cfg.attn_mode == 0 && !fits)) return false;
    if (c->cfg.n_kv_heads > 8) return false;
    const long long units = static_cast<long long>(per_cta) * c->cfg.budget_blocks * (c->cfg.block_tokens / 16);
    const int NT = c->cfg.n_q_heads / c->cfg.n_kv_heads <= 8 ? 1 : 2;
    return units <= HM_META_UNITS && hm_smem_bytes(c->cfg, per_cta, NT, NT == 1 ? 3 : 2, true) <= 227 * 1024;
}
long long pi_attn_state_floats(const pi_ctx* c, int batch) {
    const int NT = c->cfg.n_q_heads / c->cfg.n_kv_heads <= 8 ? 1 : 2;
    return static_cast<long long>(batch) * c->cfg.n_kv_heads * NT * 36 * 32;
}

int pi_launch_attn_headmajor(pi_ctx* c, int batch, const void* q, const void* pool, const int32_t* sel_slots,
                             const int32_t* sel_blocks, const int32_t* sel_count, const int32_t* ctx_len, void* out,
                             float* lse, int headwise, const pi_attn_phase* phase, cudaStream_t stream) {
    const pi_config& cfg = c->cfg;
    const long long n_slots = static_cast<long long>(batch) * cfg.pool_slots;
    // the tensor map with a box of one head's K and V rows (shared with the headwise form of the flat kernel)
    if (c->pool_map_ptr != pool || c->pool_map_slots != n_slots || c->pool_map_headwise != 1) {
        typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        const cuuint64_t B = cfg.block_tokens, hk = 2ull * cfg.n_kv_heads;
        cuuint64_t gdim[4] = {PI_HEAD_DIM, B, hk, static_cast<cuuint64_t>(n_slots)};
        cuuint64_t gstride[3] = {PI_HEAD_DIM * 2ull, B * PI_HEAD_DIM * 2ull, hk * B * PI_HEAD_DIM * 2ull};
        cuuint32_t box[4] = {64, 16, 2u, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = reinterpret_cast<encode_fn>(c->encode_tiled_fn)(
            &c->pool_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { c->pool_map_ptr = nullptr; return PI_ERR_CUDA; }
        c->pool_map_ptr = pool;
        c->pool_map_slots = n_slots;
        c->pool_map_headwise = 1;
    }
    AttnParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.sel_slots = sel_slots; p.sel_blocks = sel_blocks; p.sel_count = sel_count; p.ctx_len = ctx_len;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.part_o = nullptr; p.part_ml = nullptr; p.counters = nullptr;
    p.st = pi_status_of(c);
    p.batch = batch; p.Hq = cfg.n_q_heads; p.Hkv = cfg.n_kv_heads; p.G = cfg.n_q_heads / cfg.n_kv_heads;
    p.B = cfg.block_tokens; p.K = cfg.budget_blocks; p.C = cfg.pool_slots;
    p.headwise = headwise ? 1 : 0;
    p.hold_last = cfg.test_hold_producer;
    p.wait_cycles = c->wait_limit_cycles;
    p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(PI_HEAD_DIM));
    const int ph = phase ? phase->phase : 0;
    p.rlist = phase ? phase->rlist : nullptr;
    p.rcount = phase ? phase->rcount : nullptr;
    p.rcap = phase ? phase->rcap : 0;
    p.state = phase ? phase->state : nullptr;
    const int NT = p.G <= 8 ? 1 : 2;
    p.stages = NT == 1 ? 3 : 2;                      // the wider merge regions of G > 8 take the room of a stage
    int grid = 1, per_cta = 1, split = 1;
    (void)pi_attn_headmajor_fits(c, batch, &grid, &per_cta, &split);
    const size_t smem = hm_smem_bytes(cfg, per_cta, NT, p.stages, ph != 0);
    const int n_items = batch * cfg.n_kv_heads;
    auto launch = [&](auto kernel) -> int {
        PI_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(grid);
        lc.blockDim = dim3(288);
        lc.dynamicSmemBytes = smem;
        lc.stream = stream;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = split;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        lc.attrs = attr;
        lc.numAttrs = split > 1 ? 2 : 1;
        PI_CUDA_TRY(cudaLaunchKernelEx(&lc, kernel, c->pool_map, p, n_items, per_cta));
        return PI_OK;
    };
    int rc;
    if (ph == 0) rc = NT == 1 ? launch(attn_headmajor_kernel<1, 0>) : launch(attn_headmajor_kernel<2, 0>);
    else if (ph == 1) rc = NT == 1 ? launch(attn_headmajor_kernel<1, 1>) : launch(attn_headmajor_kernel<2, 1>);
    else rc = NT == 1 ? launch(attn_headmajor_kernel<1, 2>) : launch(attn_headmajor_kernel<2, 2>);
    if (rc != PI_OK) return rc;
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
