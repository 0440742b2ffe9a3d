// Exact top-k of 32-bit keys held in shared memory, by one whole CTA: the k largest keys win,
// equal keys go to the lower index, and the winners come out in ascending index order.  Used twice
// on the path: for the block scores (the order-preserving images of the fp32 scores, Sec. 2.2
// step 1 / Sec. 4.4.1) and for the choice of the slots to evict (keys = inverted last-selected
// stamps, ties to the lower slot).
//
// One histogram pass of 1024 bins narrows the search to the bucket of the k-th key (for score keys the
// pass bins the score VALUES linearly between the extremes, which spreads a bell-shaped distribution
// evenly; else it bins the 10 most significant bits in which the keys still differ); every warp then
// walks the histogram down from the top by itself, so no CTA barrier is spent on finding the bucket.
// If the bucket holds at most 32 keys (the usual case) they are gathered while the sure winners are
// counted, ranked by every warp on its own, and the winners are emitted: two CTA barriers in all.
// Crowded buckets (many equal keys) take further passes over the key bits and end in thresholds:
// keys above `hi` win, and so do the first `need` keys (by index) inside [lo, hi].
//
// The code runs once per launch in a single CTA per sequence with two warps per scheduler: it is bound
// by the latency of each warp's dependent instruction chain (a rolled loop iteration of one shared-memory
// load and an add costs about 55 cycles), so the loops over the keys are unrolled by four for a few
// independent loads in flight, and the passes over the keys are as few as the algorithm allows.
#pragma once

#include "pi_common.cuh"
#include "pi_score_core.cuh"

namespace pi_select {

using pi_score::padded;

constexpr int BINS = 1024;                        // at most 10 bits a pass; a lane of the walking warp sums up to 32 bins
constexpr int LINEAR_BINS = 512;                  // bins of the value-space pass (a handful of keys in the k-th bucket)
constexpr int RESOLVE_MAX = 32;                   // bucket sizes a warp ranks directly

template <int NW>
struct Scratch {
    unsigned hist[BINS + BINS / 32 + 1];          // padded like the key arrays
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

// Zeroes the counters.  A CTA barrier must separate this from the next selection.
template <int NT>
__device__ __forceinline__ void clear(Scratch<NT / 32>& sc) {
#pragma unroll 1
    for (int i = threadIdx.x; i < BINS + BINS / 32 + 1; i += NT) sc.hist[i] = 0;
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

// the fp32 value whose order-preserving image is `key` (inverse of pi_score::float_key)
__device__ __forceinline__ float key_float(uint32_t key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// How one pass maps a key of [lo, hi] to its bin: linearly in the score value, or by key bits.
struct Binning {
    uint32_t lo, hi;
    int shift, nbins;                             // bins in use: the walk skips the rest
    float fmin, scale;
    bool linear;
    __device__ __forceinline__ void set(uint32_t lo_, uint32_t hi_, bool linear_) {
        lo = lo_; hi = hi_; linear = linear_;
        const int bits = 32 - __clz(hi - lo);
        shift = bits > 10 ? bits - 10 : 0;
        nbins = linear ? LINEAR_BINS : static_cast<int>((hi - lo) >> shift) + 1;
        fmin = key_float(lo);
        scale = static_cast<float>(LINEAR_BINS) / (key_float(hi) - fmin);
    }
    // bin of a key, 0xffffffff if the key is outside [lo, hi]
    __device__ __forceinline__ unsigned bin(uint32_t key) const {
        if (key < lo || key > hi) return 0xffffffffu;
        if (linear) return min(static_cast<unsigned>(LINEAR_BINS - 1), static_cast<unsigned>((key_float(key) - fmin) * scale));
        return (key - lo) >> shift;
    }
};

// A thread's share of the keys: the consecutive indices [i0, i1) of the padded shared array.
struct Share {
    int i0, i1;
};
template <int NT>
__device__ __forceinline__ Share share_of(int n) {
    const int ipt = (n + NT - 1) / NT;
    Share s;
    s.i0 = min(static_cast<int>(threadIdx.x) * ipt, n);
    s.i1 = min(s.i0 + ipt, n);
    return s;
}

// Block-wide minimum and maximum of the keys of [m_lo, m_hi) that fall into bin `only` of `bn`
// (only == 0xfffffffe: every key of the range).  One CTA barrier.
template <int NT>
__device__ __forceinline__ void block_min_max(const uint32_t* keys, int m_lo, int m_hi, Scratch<NT / 32>& sc, const Binning& bn,
                                              unsigned only, uint32_t& kmin, uint32_t& kmax) {
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t a = 0xffffffffu, b = 0u;
#pragma unroll 1
    for (int i = m_lo + threadIdx.x; i < m_hi; i += NT) {
        const uint32_t key = keys[padded(i)];
        if (only == 0xfffffffeu || bn.bin(key) == only) { a = min(a, key); b = max(b, key); }
    }
    a = __reduce_min_sync(0xffffffffu, a);
    b = __reduce_max_sync(0xffffffffu, b);
    if (lane == 0) { sc.red_lo[warp] = a; sc.red_hi[warp] = b; }
    __syncthreads();
    kmin = __reduce_min_sync(0xffffffffu, lane < NW ? sc.red_lo[lane] : 0xffffffffu);
    kmax = __reduce_max_sync(0xffffffffu, lane < NW ? sc.red_hi[lane] : 0u);
}

// One histogram pass over the keys of [m_lo, m_hi) and, after a CTA barrier, the walk down from the top
// bin that every warp does by itself.  Returns the bin of the need-th largest
// key; `above` = keys in higher bins, `cnt` = keys in that bin.  AGGREGATE: lanes of a warp that hit
// the same bin add once (for keys with many duplicates).
template <int NT, bool AGGREGATE>
__device__ __forceinline__ unsigned histogram_walk(const uint32_t* keys, int m_lo, int m_hi, Scratch<NT / 32>& sc, const Binning& bn,
                                                   unsigned need, unsigned& above, unsigned& cnt) {
    const int lane = threadIdx.x & 31;
#pragma unroll 4
    for (int i0 = m_lo; i0 < m_hi; i0 += NT) {
        const int i = i0 + threadIdx.x;
        const unsigned bin = i < m_hi ? bn.bin(keys[padded(i)]) : 0xffffffffu;
        if (AGGREGATE) {
            const unsigned peers = __match_any_sync(0xffffffffu, bin);
            if (bin != 0xffffffffu && lane == __ffs(peers) - 1) atomicAdd(&sc.hist[padded(bin)], static_cast<unsigned>(__popc(peers)));
        } else if (bin != 0xffffffffu) {
            atomicAdd(&sc.hist[padded(bin)], 1u);
        }
    }
    __syncthreads();
    // the walk: lane l sums the bpl bins below top - l * bpl, a scan finds the lane whose group holds the
    // need-th key, a second scan over that group's bins finds the bin
    const int bpl = (bn.nbins + 31) >> 5, top = bn.nbins - 1 - lane * bpl;
    unsigned part = 0;
#pragma unroll 4
    for (int j = 0; j < bpl; ++j)
        if (top - j >= 0) part += sc.hist[padded(top - j)];
    const unsigned s1 = warp_inclusive_scan(part, lane);
    const unsigned m1 = __ballot_sync(0xffffffffu, s1 >= need);
    const int l1 = m1 ? __ffs(m1) - 1 : 31;
    const unsigned over = __shfl_sync(0xffffffffu, s1 - part, l1);
    const int gtop = bn.nbins - 1 - l1 * bpl;           // top bin of the group found
    const unsigned f = (lane < bpl && gtop - lane >= 0) ? sc.hist[padded(gtop - lane)] : 0u;
    const unsigned sf = warp_inclusive_scan(f, lane) + over;
    const unsigned m3 = __ballot_sync(0xffffffffu, sf >= need);
    const int l3 = m3 ? __ffs(m3) - 1 : 31;
    above = __shfl_sync(0xffffffffu, sf - f, l3);
    cnt = __shfl_sync(0xffffffffu, f, l3);
    return static_cast<unsigned>(max(gtop - l3, 0));
}

// Candidates of the scratch ranked by every warp on its own by (key descending, index ascending):
// lane c holds candidate c.  Returns the mask of the `need` best; mi = this lane's candidate index.
template <int NW>
__device__ __forceinline__ unsigned rank_candidates(const Scratch<NW>& sc, unsigned cnt, unsigned need, uint32_t& mk, int& mi) {
    const int lane = threadIdx.x & 31;
    const bool have = lane < static_cast<int>(cnt);
    mk = have ? sc.cand_key[lane] : 0u;
    mi = have ? sc.cand_idx[lane] : 0x7fffffff;
    unsigned rank = 0;
#pragma unroll 1
    for (unsigned j = 0; j < cnt; ++j) {
        const uint32_t ok = __shfl_sync(0xffffffffu, mk, j);
        const int oi = __shfl_sync(0xffffffffu, mi, j);
        rank += (ok > mk || (ok == mk && oi < mi)) ? 1u : 0u;
    }
    return __ballot_sync(0xffffffffu, have && rank < need);
}

// Emits, in ascending index order, the indices outside [m_lo, m_hi) (when OUTSIDE_TAKEN: the always-
// selected sink and local blocks) and the winners under the thresholds `r`: emit(position, index, key).
// Every thread owns a run of consecutive indices; one CTA barrier.  Returns the number emitted.
template <int NT, bool OUTSIDE_TAKEN, class Emit>
__device__ __forceinline__ unsigned block_emit_ordered(const uint32_t* keys, int n, int m_lo, int m_hi, Result r,
                                                       Scratch<NT / 32>& sc, Emit emit) {
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const Share sh = share_of<NT>(n);
    unsigned c_sure = 0, c_eq = 0;
#pragma unroll 4
    for (int i = sh.i0; i < sh.i1; ++i) {
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
#pragma unroll 4
    for (int i = sh.i0; i < sh.i1; ++i) {
        bool take;
        uint32_t key = 0;
        const unsigned pos = sure_b + min(eq_b, r.need);
        if (i < m_lo || i >= m_hi) { take = OUTSIDE_TAKEN; sure_b += OUTSIDE_TAKEN ? 1u : 0u; }
        else {
            key = keys[padded(i)];
            if (key > r.hi) { take = true; ++sure_b; }
            else if (key >= r.lo) { take = eq_b < r.need; ++eq_b; }
            else take = false;
        }
        if (take) emit(pos, i, key);
    }
    return (total & 0xffffu) + min(total >> 16, r.need);
}

// The whole selection: emit(position, index, key) for the always-taken indices outside [m_lo, m_hi)
// (when OUTSIDE_TAKEN) and for the k largest keys of [m_lo, m_hi), in ascending index order; returns
// their number.  All NT threads call; the scratch must have been cleared (and the keys written) before
// the last CTA barrier.  The result is the same in every thread.
//   FLOAT_KEYS  the keys are images of fp32 scores (first pass bins the values linearly)
//   AGGREGATE   warp-aggregated histogram updates
//   have_mm     kmin / kmax already hold the extremes of the keys that take part (else one more barrier
//               finds them).  Keys below kmin never win: the diff hides the slots that may not be evicted
//               that way.
template <int NT, bool FLOAT_KEYS, bool AGGREGATE, bool OUTSIDE_TAKEN, class Emit>
__device__ __forceinline__ unsigned block_topk_emit(const uint32_t* keys, int n, int m_lo, int m_hi, unsigned k, Scratch<NT / 32>& sc,
                                                    bool have_mm, uint32_t kmin, uint32_t kmax, Emit emit) {
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_mid = m_hi - m_lo;
    Binning bn;
    Result r;
    if (k == 0 || n_mid <= 0) {                       // nothing from the range
        r.lo = 0xffffffffu; r.hi = 0xffffffffu; r.need = 0;
        return block_emit_ordered<NT, OUTSIDE_TAKEN>(keys, n, m_lo, m_hi, r, sc, emit);
    }
    if (!have_mm) block_min_max<NT>(keys, m_lo, m_hi, sc, bn, 0xfffffffeu, kmin, kmax);
    r.lo = kmin; r.hi = kmax; r.need = min(k, static_cast<unsigned>(n_mid));
    if (k >= static_cast<unsigned>(n_mid) || kmax == kmin)   // everything, or all keys equal: ties by index
        return block_emit_ordered<NT, OUTSIDE_TAKEN>(keys, n, m_lo, m_hi, r, sc, emit);

    bn.set(kmin, kmax, FLOAT_KEYS);
    unsigned above, cnt;
    const unsigned t = histogram_walk<NT, AGGREGATE>(keys, m_lo, m_hi, sc, bn, k, above, cnt);
    unsigned need = k - above;                        // winners still to come from bucket t

    const Share sh = share_of<NT>(n);
    const bool wide = (n + NT - 1) / NT > 64;         // more keys per thread than the winner masks below hold
    if (cnt > RESOLVE_MAX || wide || (!bn.linear && (bn.shift == 0 || cnt == need))) {
        // Thresholds instead of a gathered bucket: one key value per bin, a bucket that wins as a whole,
        // or a crowded bucket (many equal or nearly equal keys) that further passes over the key bits narrow.
        uint32_t lo, hi;
        if (bn.linear) {
            block_min_max<NT>(keys, m_lo, m_hi, sc, bn, t, lo, hi);
        } else {
            lo = bn.lo + (t << bn.shift);
            const uint32_t span = bn.shift ? ((1u << bn.shift) - 1u) : 0u;
            hi = (bn.hi - lo < span) ? bn.hi : lo + span;
        }
#pragma unroll 1
        for (int pass = 0; pass < 5 && cnt != need && hi != lo; ++pass) {
            __syncthreads();                          // every warp has finished reading the last histogram
            clear<NT>(sc);
            __syncthreads();
            bn.set(lo, hi, false);
            const unsigned tb = histogram_walk<NT, AGGREGATE>(keys, m_lo, m_hi, sc, bn, need, above, cnt);
            need -= above;
            lo = bn.lo + (tb << bn.shift);
            const uint32_t span = bn.shift ? ((1u << bn.shift) - 1u) : 0u;
            hi = (bn.hi - lo < span) ? bn.hi : lo + span;
        }
        r.lo = lo; r.hi = hi; r.need = need;
        return block_emit_ordered<NT, OUTSIDE_TAKEN>(keys, n, m_lo, m_hi, r, sc, emit);
    }

    // ---- the bucket's keys are gathered while the sure winners (higher bins) are counted; every thread
    // remembers which of its keys are sure winners and which sit in the bucket (bit j = its j-th key), so
    // that the emission below touches the winners only
    unsigned long long sure_mask = 0ull, bucket_mask = 0ull;
    unsigned c_sure = 0;
#pragma unroll 4
    for (int i = sh.i0; i < sh.i1; ++i) {
        const unsigned long long bit = 1ull << (i - sh.i0);
        if (i < m_lo || i >= m_hi) {
            if (OUTSIDE_TAKEN) { sure_mask |= bit; ++c_sure; }
            continue;
        }
        const uint32_t key = keys[padded(i)];
        const unsigned b = bn.bin(key);
        if (b == t) {
            const unsigned p = atomicAdd(&sc.ncand, 1u);
            if (p < RESOLVE_MAX) { sc.cand_key[p] = key; sc.cand_idx[p] = i; }
            bucket_mask |= bit;
        } else if (b != 0xffffffffu && b > t) {
            sure_mask |= bit;
            ++c_sure;
        }
    }
    const unsigned inc = warp_inclusive_scan(c_sure, lane);
    if (lane == 31) sc.warp_tot[warp] = inc;
    __syncthreads();
    uint32_t mk;
    int mi;
    const unsigned winmask = rank_candidates(sc, cnt, need, mk, mi);
    // winners before this thread's first index: sure ones (scan) and bucket ones (their indices are known)
    const unsigned ws = warp_inclusive_scan(lane < NW ? sc.warp_tot[lane] : 0u, lane);
    const unsigned total_sure = __shfl_sync(0xffffffffu, ws, NW - 1);
    const unsigned wbase = __shfl_sync(0xffffffffu, ws, warp > 0 ? warp - 1 : 0);
    unsigned pos = (warp > 0 ? wbase : 0u) + inc - c_sure;
#pragma unroll 1
    for (unsigned j = 0; j < cnt; ++j) {
        const int oi = __shfl_sync(0xffffffffu, mi, j);
        pos += (((winmask >> j) & 1u) && oi < sh.i0) ? 1u : 0u;
    }
    // my bucket keys whose candidate made it join my sure winners
    while (bucket_mask) {
        const int j = __ffsll(static_cast<long long>(bucket_mask)) - 1;
        bucket_mask &= bucket_mask - 1;
        for (unsigned c = 0; c < cnt; ++c)
            if (sc.cand_idx[c] == sh.i0 + j && ((winmask >> c) & 1u)) sure_mask |= 1ull << j;
    }
    while (sure_mask) {
        const int j = __ffsll(static_cast<long long>(sure_mask)) - 1;
        sure_mask &= sure_mask - 1;
        const int i = sh.i0 + j;
        emit(pos, i, (i < m_lo || i >= m_hi) ? 0u : keys[padded(i)]);
        ++pos;
    }
    return total_sure + static_cast<unsigned>(__popc(winmask));
}

}  // namespace pi_select
