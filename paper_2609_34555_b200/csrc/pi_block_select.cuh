// Exact top-k of 32-bit keys held in shared memory, by one whole CTA: the k largest keys win,
// equal keys go to the lower index.  Used twice on the path: for the block scores (the
// order-preserving images of the fp32 scores, Sec. 2.2 step 1 / Sec. 4.4.1) and for the choice
// of the slots to evict (keys = inverted last-selected stamps, ties to the lower slot).
//
// The search narrows a key interval [lo, hi] with one histogram pass over the 11 most significant
// bits in which the remaining keys still differ; every warp then walks the histogram down from
// the top by itself (64 coarse counters, then the 32 bins under one of them), so finding the
// bucket of the k-th key costs no further CTA barrier; a bucket of at most 32 keys is ranked
// directly by every warp.  Typical cost: three CTA barriers.  The result is a pair of thresholds:
// keys above `hi` are winners, and so are the first `need` keys (by index) inside [lo, hi].
// A second routine emits the winners in ascending index order.
#pragma once

#include "pi_common.cuh"
#include "pi_score_core.cuh"

namespace pi_select {

using pi_score::padded;

constexpr int BINS = 2048;
constexpr int COARSE = BINS / 32;                 // one coarse counter per 32 bins
constexpr int RESOLVE_MAX = 32;                   // bucket sizes a warp ranks directly

template <int NW>
struct Scratch {
    unsigned hist[BINS + BINS / 32 + 1];          // padded like the key arrays
    unsigned coarse[COARSE];
    uint32_t red_lo[NW], red_hi[NW];
    unsigned warp_tot[NW];
    uint32_t cand_key[RESOLVE_MAX];
    int cand_idx[RESOLVE_MAX];
    unsigned ncand;
};

struct Result {
    uint32_t lo, hi;
    unsigned need;
};

// Zeroes the counters.  A CTA barrier must separate this from the next call of block_select.
template <int NT>
__device__ __forceinline__ void clear(Scratch<NT / 32>& sc) {
    for (int i = threadIdx.x; i < BINS + BINS / 32 + 1; i += NT) sc.hist[i] = 0;
    if (threadIdx.x < COARSE) sc.coarse[threadIdx.x] = 0;
    if (threadIdx.x == 0) sc.ncand = 0;
}

__device__ __forceinline__ unsigned warp_inclusive_scan(unsigned v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Thresholds of the k largest keys among keys[padded(i)], i in [m_lo, m_hi).  All NT threads
// call; the scratch must have been cleared (and the keys written) before the last CTA barrier.
// The result is the same in every thread.
template <int NT>
__device__ __forceinline__ Result block_select(const uint32_t* keys, int m_lo, int m_hi, unsigned k, Scratch<NT / 32>& sc) {
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_mid = m_hi - m_lo;
    Result r;
    if (k == 0 || n_mid <= 0) {                       // nothing from the range
        r.lo = 0xffffffffu; r.hi = 0xffffffffu; r.need = 0;
        return r;
    }
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    for (int i = m_lo + tid; i < m_hi; i += NT) {
        const uint32_t key = keys[padded(i)];
        kmin = min(kmin, key); kmax = max(kmax, key);
    }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) { sc.red_lo[warp] = kmin; sc.red_hi[warp] = kmax; }
    __syncthreads();
    kmin = __reduce_min_sync(0xffffffffu, lane < NW ? sc.red_lo[lane] : 0xffffffffu);
    kmax = __reduce_max_sync(0xffffffffu, lane < NW ? sc.red_hi[lane] : 0u);
    if (k >= static_cast<unsigned>(n_mid)) {          // everything: [lo, hi] spans all keys
        r.lo = kmin; r.hi = kmax; r.need = static_cast<unsigned>(n_mid);
        return r;
    }

    uint32_t lo = kmin, hi = kmax;
    unsigned need = k;
    for (int pass = 0; pass < 4; ++pass) {
        const uint32_t range = hi - lo;
        if (range == 0) break;                        // every key left is equal: ties by index
        const int bits = 32 - __clz(range);
        const int shift = bits > 11 ? bits - 11 : 0;
        if (pass > 0) {                               // every warp has finished reading the last histogram
            __syncthreads();
            clear<NT>(sc);
            __syncthreads();
        }
        for (int i = m_lo + tid; i < m_hi; i += NT) {
            const uint32_t key = keys[padded(i)];
            if (key >= lo && key <= hi) {
                const unsigned bin = (key - lo) >> shift;
                atomicAdd(&sc.hist[padded(bin)], 1u);
                atomicAdd(&sc.coarse[bin >> 5], 1u);
            }
        }
        __syncthreads();
        // walk down from the top bin: first the coarse counters (lane i of the first round holds
        // coarse[63 - i], of the second coarse[31 - i]), then the 32 bins under the one found
        const unsigned c1 = sc.coarse[COARSE - 1 - lane], c2 = sc.coarse[COARSE - 33 - lane];
        const unsigned s1 = warp_inclusive_scan(c1, lane);
        const unsigned s2 = warp_inclusive_scan(c2, lane) + __shfl_sync(0xffffffffu, s1, 31);
        const unsigned m1 = __ballot_sync(0xffffffffu, s1 >= need), m2 = __ballot_sync(0xffffffffu, s2 >= need);
        int pos;
        unsigned above;
        if (m1) {
            const int l = __ffs(m1) - 1;
            pos = l; above = __shfl_sync(0xffffffffu, s1 - c1, l);
        } else {
            const int l = m2 ? __ffs(m2) - 1 : 31;
            pos = 32 + l; above = __shfl_sync(0xffffffffu, s2 - c2, l);
        }
        const int cbin = COARSE - 1 - pos;
        const unsigned f = sc.hist[padded(cbin * 32 + 31 - lane)];
        const unsigned sf = warp_inclusive_scan(f, lane) + above;
        const unsigned m3 = __ballot_sync(0xffffffffu, sf >= need);
        const int l3 = m3 ? __ffs(m3) - 1 : 31;
        const int bin = cbin * 32 + 31 - l3;
        const unsigned acc = __shfl_sync(0xffffffffu, sf - f, l3), cnt = __shfl_sync(0xffffffffu, f, l3);
        const uint32_t nlo = lo + (static_cast<uint32_t>(bin) << shift);
        const uint32_t span = shift ? ((1u << shift) - 1u) : 0u;
        hi = (hi - nlo < span) ? hi : nlo + span;
        lo = nlo;
        need -= acc;
        if (shift == 0 || cnt == need) break;
        if (cnt <= RESOLVE_MAX) {
            // few keys left in the bucket: gather them, then every warp ranks them by
            // (key descending, index ascending) by itself
            for (int i = m_lo + tid; i < m_hi; i += NT) {
                const uint32_t key = keys[padded(i)];
                if (key >= lo && key <= hi) {
                    const unsigned p = atomicAdd(&sc.ncand, 1u);
                    if (p < RESOLVE_MAX) { sc.cand_key[p] = key; sc.cand_idx[p] = i; }
                }
            }
            __syncthreads();
            const bool have = lane < static_cast<int>(cnt);
            const uint32_t mk = have ? sc.cand_key[lane] : 0u;
            const int mi = have ? sc.cand_idx[lane] : 0x7fffffff;
            unsigned rank = 0;
            for (unsigned j = 0; j < cnt; ++j) {
                const uint32_t ok = __shfl_sync(0xffffffffu, mk, j);
                const int oi = __shfl_sync(0xffffffffu, mi, j);
                rank += (ok > mk || (ok == mk && oi < mi)) ? 1u : 0u;
            }
            // the need-th best candidate fixes the threshold key; ties at it go by index
            const unsigned is_tau = __ballot_sync(0xffffffffu, have && rank == need - 1);
            const uint32_t tau = __shfl_sync(0xffffffffu, mk, is_tau ? __ffs(is_tau) - 1 : 0);
            need = __popc(__ballot_sync(0xffffffffu, have && mk == tau && rank < need));
            lo = tau; hi = tau;
            break;
        }
    }
    r.lo = lo; r.hi = hi; r.need = need;
    return r;
}

// Emits the winners in ascending index order: emit(position, index) for every index i in [0, n)
// that is outside [m_lo, m_hi) (when OUTSIDE_TAKEN: the always-selected sink and local blocks) or
// whose key wins under `r`.  Every thread owns a run of consecutive indices; one CTA barrier.
// Returns the number of winners (the same in every thread).
template <int NT, bool OUTSIDE_TAKEN, class Emit>
__device__ __forceinline__ unsigned block_emit_ordered(const uint32_t* keys, int n, int m_lo, int m_hi, Result r,
                                                       Scratch<NT / 32>& sc, Emit emit) {
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ipt = (n + NT - 1) / NT;
    const int i0 = min(tid * ipt, n), i1 = min(i0 + ipt, n);
    unsigned c_sure = 0, c_eq = 0;
    for (int i = i0; i < i1; ++i) {
        if (i < m_lo || i >= m_hi) { c_sure += OUTSIDE_TAKEN ? 1u : 0u; continue; }
        const uint32_t key = keys[padded(i)];
        if (key > r.hi) ++c_sure;
        else if (key >= r.lo) ++c_eq;
    }
    // block-wide exclusive scan of both counts at once (each stays below 2^16)
    const unsigned packed = c_sure | (c_eq << 16);
    const unsigned inc = warp_inclusive_scan(packed, lane);
    if (lane == 31) sc.warp_tot[warp] = inc;
    __syncthreads();
    const unsigned ws = warp_inclusive_scan(lane < NW ? sc.warp_tot[lane] : 0u, lane);
    const unsigned total = __shfl_sync(0xffffffffu, ws, NW - 1);
    const unsigned base = __shfl_sync(0xffffffffu, ws, warp > 0 ? warp - 1 : 0);
    const unsigned before = (warp > 0 ? base : 0u) + inc - packed;
    unsigned sure_b = before & 0xffffu, eq_b = before >> 16;
    for (int i = i0; i < i1; ++i) {
        bool take;
        const unsigned pos = sure_b + min(eq_b, r.need);
        if (i < m_lo || i >= m_hi) { take = OUTSIDE_TAKEN; sure_b += OUTSIDE_TAKEN ? 1u : 0u; }
        else {
            const uint32_t key = keys[padded(i)];
            if (key > r.hi) { take = true; ++sure_b; }
            else if (key >= r.lo) { take = eq_b < r.need; ++eq_b; }
            else take = false;
        }
        if (take) emit(pos, i);
    }
    return (total & 0xffffu) + min(total >> 16, r.need);
}

}  // namespace pi_select
