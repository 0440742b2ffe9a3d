// Miss diff of one sequence's selection against its block table, by one whole CTA (Sec. 2.2 step 2:
// B_recall = B_topk \ B_gpu), with the victim choice, the table update and the coalesced recall list.
// Shared by the stand-alone diff kernel and by the kernel that scores, selects and diffs in one launch.
//
//   misses     = selected blocks with block_table[b] < 0, ascending
//   candidates = slots whose block is neither selected nor sink/local (free slots count), ordered by
//                (stamp, slot) ascending; the i-th miss takes the i-th candidate.  Up to RANK_MAX_MISSES
//                misses: the victims are the top-n_miss of the inverted stamps (the same block-wide
//                top-k routine that selects the blocks; ties to the lower slot), then ranked among
//                themselves by pairwise comparison.  More misses (a cold pool with a wide budget):
//                bitonic sort of all candidate keys.
//   update     = evicted block leaves the table, the miss enters it, every selected slot gets stamp = step
//   list       = (block -> slot) pairs, runs that are consecutive on both sides merged
#pragma once

#include "pi_block_select.cuh"
#include "pi_common.cuh"

namespace pi_diff {

using pi_score::padded;

constexpr int RANK_MAX_MISSES = 512;

struct SeqArgs {
    int32_t* table;                 // this sequence's rows in global memory
    int32_t* slot_block;
    uint32_t* slot_stamp;
    int32_t* sel_slots;
    pi_extent* list;
    int32_t* count;
    unsigned long long* stats;
    pi_status_ref st;
    int seq, n_blocks, cnt, K, C, Cpad, n_sink, n_local, max_blocks;
    uint32_t step;
};

// Shared-memory views.  `keys` is a union: uint32 [padded(C)] for the ranking path, 64-bit [Cpad] for
// the sort path.  `table_s` (may be null) is a copy of the sequence's table row.
struct Smem {
    uint32_t* keys;
    int32_t *sel, *slot, *miss;     // [K]: selected block, its slot, position in `sel` of the i-th miss
    int32_t* vslot;                 // [min(K, RANK_MAX_MISSES)] victims in slot order
    uint32_t* vkey;                 // [min(K, RANK_MAX_MISSES)]
    int32_t* vict;                  // [min(K, RANK_MAX_MISSES)] victims in eviction order
    int32_t* sb;                    // [C] copy of slot_block
    uint32_t* stp;                  // [C] copy of slot_stamp
    unsigned char* used;            // [C] slot holds a selected block
    const int32_t* table_s;
    int* warp_tot;                  // [2][NT / 32]
    int* n_cand;
    // Optional (cluster form): all C slots in eviction order, (stamp, slot) ascending, written into this CTA's
    // shared memory by another CTA of the cluster, which arrives on the mbarrier `lru_bar` when it is done.
    const unsigned short* lru_order;
    uint32_t lru_bar;               // shared-memory address of that mbarrier (phase 0)
    long long lru_wait;             // bound of the wait in cycles
};

// Bytes of the arrays above (without the key union), and of the union.
__host__ __device__ inline size_t smem_lists_bytes(int K, int C) {
    const size_t kv = static_cast<size_t>(K < RANK_MAX_MISSES ? K : RANK_MAX_MISSES);
    const size_t words = (3 * static_cast<size_t>(K) + 3 * kv + 2 * static_cast<size_t>(C)) * 4;
    return ((words + 15) & ~size_t(15)) + ((static_cast<size_t>(C) + 15) & ~size_t(15));
}
__host__ __device__ inline size_t smem_keys_bytes(int C, int Cpad) {
    const size_t a = (static_cast<size_t>(C) + C / 32 + 1) * 4, b = static_cast<size_t>(Cpad) * 8;
    return ((a > b ? a : b) + 15) & ~size_t(15);
}

// Carves the list arrays out of `base` (16-byte aligned); `keys` and `table_s` are set by the caller.
__device__ __forceinline__ Smem carve(unsigned char* base, int K, int C) {
    Smem m;
    const int kv = K < RANK_MAX_MISSES ? K : RANK_MAX_MISSES;
    m.sel = reinterpret_cast<int32_t*>(base);
    m.slot = m.sel + K;
    m.miss = m.slot + K;
    m.vslot = m.miss + K;
    m.vkey = reinterpret_cast<uint32_t*>(m.vslot + kv);
    m.vict = reinterpret_cast<int32_t*>(m.vkey + kv);
    m.sb = m.vict + kv;
    m.stp = reinterpret_cast<uint32_t*>(m.sb + C);
    m.used = reinterpret_cast<unsigned char*>(m.stp + C);
    m.keys = nullptr; m.table_s = nullptr; m.warp_tot = nullptr; m.n_cand = nullptr;
    m.lru_order = nullptr; m.lru_bar = 0; m.lru_wait = 0;
    return m;
}

// Preconditions, followed by a CTA barrier: m.sel[0, cnt) holds the selection, m.sb / m.stp the
// slot arrays, m.used and *m.n_cand are zero, the select scratch is cleared.
template <int NT>
__device__ __forceinline__ void diff_sequence(const SeqArgs& a, const Smem& m, pi_select::Scratch<NT / 32>& sc) {
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // 1. look the selection up; misses compacted in selection (= ascending block) order
    int n_miss = 0;
    for (int j0 = 0, it = 0; j0 < a.cnt; j0 += NT, ++it) {
        const int j = j0 + tid;
        bool miss = false;
        if (j < a.cnt) {
            const int b = m.sel[j];
            int slot = -1;
            if (b < 0 || b >= a.n_blocks) {
                pi_report(a.st, PI_ERR_INDEX_RANGE, PI_STAGE_DIFF, a.seq, j, b);
                m.sel[j] = -1;
            } else {
                slot = m.table_s ? m.table_s[b] : a.table[b];
                if (slot >= a.C) { pi_report(a.st, PI_ERR_INDEX_RANGE, PI_STAGE_DIFF, a.seq, b, slot); slot = -1; m.sel[j] = -1; }
                else if (slot >= 0) m.used[slot] = 1;
                else miss = true;
            }
            m.slot[j] = slot;
        }
        // ordered position of this round's misses (warp totals double-buffered: one barrier per round)
        const unsigned bal = __ballot_sync(0xffffffffu, miss);
        int* wt = m.warp_tot + (it & 1) * NW;
        if (lane == 0) wt[warp] = __popc(bal);
        __syncthreads();
        int off = 0, tot = 0;
#pragma unroll
        for (int i = 0; i < NW; ++i) {
            const int t = wt[i];
            if (i < warp) off += t;
            tot += t;
        }
        if (miss) m.miss[n_miss + off + __popc(bal & ((1u << lane) - 1u))] = j;
        n_miss += tot;
    }
    __syncthreads();

    // 2'. The slots in eviction order came from another CTA of the cluster: the victims are the first n_miss of
    //     them that may be evicted (not holding a block of this selection, not holding a sink or local block).
    bool use_order = m.lru_order != nullptr && n_miss > 0 && n_miss <= RANK_MAX_MISSES;
    bool too_small = false;
    int n_cand = 0;
    if (use_order) {
        bool ok = false;
        {
            uint32_t done = 0;
            const long long t0 = clock64();
            for (;;) {
                asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                             : "=r"(done) : "r"(m.lru_bar), "r"(0u) : "memory");
                if (done || clock64() - t0 > m.lru_wait) break;
            }
            ok = done != 0;
        }
        use_order = __syncthreads_and(ok) != 0;             // (a wait that ran out: the victims are found the other way)
    }
    if (use_order) {
        int found = 0;
        for (int base = 0, it = 0; base < a.C && found < n_miss; base += NT, ++it) {
            const int r = base + tid;
            bool cand = false;
            int s = 0;
            if (r < a.C) {
                s = m.lru_order[r];
                const int b = m.sb[s];
                const bool pinned = b >= 0 && (b < a.n_sink || b >= a.n_blocks - a.n_local);
                cand = b < 0 || (!m.used[s] && !pinned);
            }
            const unsigned bal = __ballot_sync(0xffffffffu, cand);
            int* wt = m.warp_tot + (it & 1) * NW;
            if (lane == 0) wt[warp] = __popc(bal);
            __syncthreads();
            int off = 0, tot = 0;
#pragma unroll
            for (int i = 0; i < NW; ++i) {
                const int t = wt[i];
                if (i < warp) off += t;
                tot += t;
            }
            const int pos = found + off + __popc(bal & ((1u << lane) - 1u));
            if (cand && pos < n_miss) m.vict[pos] = s;
            found += tot;
        }
        n_cand = found;                                     // all candidates when there are too few of them
        too_small = found < n_miss;
        __syncthreads();
    }

    // 2. victim candidates.  Ranking path: key = inverted stamp (older = larger), 0 for a slot that may not
    //    be evicted.  Sort path: (stamp, slot) in 64 bits, everything else sorts to the end.
    const bool rank_path = n_miss <= RANK_MAX_MISSES;
    unsigned long long* keys64 = reinterpret_cast<unsigned long long*>(m.keys);
    uint32_t kmin = 0xffffffffu, kmax = 0u;             // extremes of the candidates' ranking keys, found on the way
    if (n_miss > 0 && !use_order) {
        int my_cand = 0;
#pragma unroll 1
        for (int s = tid; s < (rank_path ? a.C : a.Cpad); s += NT) {
            bool cand = false;
            uint32_t stamp = 0;
            if (s < a.C) {
                const int b = m.sb[s];
                const bool pinned = b >= 0 && (b < a.n_sink || b >= a.n_blocks - a.n_local);
                cand = b < 0 || (!m.used[s] && !pinned);
                stamp = m.stp[s];
            }
            if (rank_path) {
                const uint32_t key = cand ? max(~stamp, 1u) : 0u;
                m.keys[padded(s)] = key;
                if (cand) { kmin = min(kmin, key); kmax = max(kmax, key); }
            } else {
                keys64[s] = cand ? ((static_cast<unsigned long long>(stamp) << 32) | static_cast<unsigned>(s)) : ~0ull;
            }
            my_cand += cand ? 1 : 0;
        }
        my_cand = __reduce_add_sync(0xffffffffu, my_cand);
        kmin = __reduce_min_sync(0xffffffffu, kmin);
        kmax = __reduce_max_sync(0xffffffffu, kmax);
        if (lane == 0) {
            if (my_cand) atomicAdd(m.n_cand, my_cand);
            sc.red_lo[warp] = kmin; sc.red_hi[warp] = kmax;
        }
    }
    if (!use_order) {
        __syncthreads();
        n_cand = *m.n_cand;
        too_small = n_cand < n_miss;
    }
    if (n_miss > 0 && !use_order) {
        kmin = __reduce_min_sync(0xffffffffu, lane < NW ? sc.red_lo[lane] : 0xffffffffu);
        kmax = __reduce_max_sync(0xffffffffu, lane < NW ? sc.red_hi[lane] : 0u);
    }

    if (n_miss > 0 && !too_small) {
        if (use_order) {
            // (the victims are in m.vict already)
        } else if (rank_path) {
            // 3a. the n_miss oldest candidates (ties to the lower slot), gathered in slot order, then
            //     ranked by (stamp ascending, slot ascending) against each other
            // (stamps repeat a lot: lanes that hit the same histogram bin add once; the slots that may not be
            // evicted carry key 0, below the candidates' smallest key, and so never enter the search)
            pi_select::block_topk_emit<NT, false, true, false>(m.keys, a.C, 0, a.C, static_cast<unsigned>(n_miss), sc, true, kmin, kmax,
                                                               [&](unsigned pos, int s, uint32_t key) {
                if (pos < static_cast<unsigned>(n_miss)) { m.vslot[pos] = s; m.vkey[pos] = key; }
            });
            __syncthreads();
            for (int v = tid; v < n_miss; v += NT) {
                const uint32_t kv = m.vkey[v];
                int rank = 0;
                for (int u = 0; u < n_miss; ++u) {
                    const uint32_t ku = m.vkey[u];
                    rank += (ku > kv || (ku == kv && u < v)) ? 1 : 0;
                }
                m.vict[rank] = m.vslot[v];
            }
            __syncthreads();
        } else {
            // 3b. bitonic sort of all candidate keys.  Warp w owns elements [32*E*w, 32*E*(w+1)), so exchanges
            //     at distance < 32*E stay inside one warp and need only a warp barrier
            const int E = max(1, a.Cpad / NT), wspan = 32 * E;
            for (int k = 2; k <= a.Cpad; k <<= 1) {
                for (int j = k >> 1; j > 0; j >>= 1) {
                    if (j >= wspan) __syncthreads();
                    for (int e = 0; e < E; ++e) {
                        const int i = (warp * E + e) * 32 + lane, l = i ^ j;
                        if (l > i && l < a.Cpad) {
                            const unsigned long long x = keys64[i], y = keys64[l];
                            const bool up = (i & k) == 0;
                            if ((x > y) == up) { keys64[i] = y; keys64[l] = x; }
                        }
                    }
                    if (j >= wspan) __syncthreads(); else __syncwarp();
                }
            }
            __syncthreads();
        }
        // 4. i-th miss takes the i-th victim
        for (int i = tid; i < n_miss; i += NT) {
            const int j = m.miss[i];
            const int slot = rank_path ? m.vict[i] : static_cast<int>(keys64[i] & 0xffffffffull);
            const int old = m.sb[slot];
            if (old >= 0 && old < a.max_blocks) a.table[old] = -1;
            a.table[m.sel[j]] = slot;
            a.slot_block[slot] = m.sel[j];
            m.slot[j] = slot;
        }
        __syncthreads();
    } else if (too_small && tid == 0) {
        pi_report(a.st, PI_ERR_POOL_TOO_SMALL, PI_STAGE_DIFF, a.seq, n_miss, n_cand);
    }

    // 5. stamps and the slot of every selected block
    for (int j = tid; j < a.K; j += NT) {
        int slot = -1;
        if (j < a.cnt) {
            slot = m.slot[j];
            if (slot >= 0 && !too_small) a.slot_stamp[slot] = a.step;
        }
        a.sel_slots[j] = slot;
    }

    // 6. recall list: heads of runs consecutive in block and in slot
    int n_ext = 0;
    if (!too_small) {
        for (int i0 = 0, it = 0; i0 < n_miss; i0 += NT, ++it) {
            const int i = i0 + tid;
            bool head = false;
            if (i < n_miss) {
                const int j = m.miss[i];
                head = true;
                if (i > 0) {
                    const int jp = m.miss[i - 1];
                    head = !(m.sel[jp] + 1 == m.sel[j] && m.slot[jp] + 1 == m.slot[j]);
                }
            }
            const unsigned bal = __ballot_sync(0xffffffffu, head);
            int* wt = m.warp_tot + (it & 1) * NW;
            if (lane == 0) wt[warp] = __popc(bal);
            __syncthreads();
            int off = 0, tot = 0;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const int t = wt[w];
                if (w < warp) off += t;
                tot += t;
            }
            if (head) {
                int len = 1;
                while (i + len < n_miss) {
                    const int x = m.miss[i + len - 1], y = m.miss[i + len];
                    if (m.sel[x] + 1 == m.sel[y] && m.slot[x] + 1 == m.slot[y]) ++len; else break;
                }
                pi_extent e;
                e.src_unit = m.sel[m.miss[i]];
                e.dst_unit = m.slot[m.miss[i]];
                e.n_units = len;
                e.units_before = i;
                a.list[n_ext + off + __popc(bal & ((1u << lane) - 1u))] = e;
            }
            n_ext += tot;
        }
    }
    if (tid == 0) {
        *a.count = n_ext;
        atomicAdd(a.stats + 0, 1ull);
        atomicAdd(a.stats + 1, static_cast<unsigned long long>(a.cnt));
        atomicAdd(a.stats + 2, static_cast<unsigned long long>(too_small ? 0 : n_miss));
        atomicAdd(a.stats + 3, static_cast<unsigned long long>(n_ext));
    }
}

}  // namespace pi_diff
