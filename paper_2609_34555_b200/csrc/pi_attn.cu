// Sparse GQA decode attention over the selected pool slots.
//
// Work is one flat list of "units": (sequence, selected block, 16-token sub-tile),
// each unit being the K and V rows of those 16 tokens for ALL kv heads (Hkv * 8 KB).
// A persistent grid splits the list evenly (split-K across CTAs, ranges may cross
// sequence boundaries); a CTA is one TMA producer warp plus one consumer warp per kv
// head.  The producer streams units through a ring of shared-memory stages with
// tiled TMA loads (128-byte swizzle, every CTA fetches its own tiles); consumer warp h computes, for its
// G query heads,  S^T = K q^T  (tokens on M, heads on N, bf16 mma, fp32 accumulate),
// an online softmax over tokens, and  O^T += V^T P.  A (CTA, sequence) segment that
// does not cover its whole sequence writes an fp32 partial (m, l, O); a small second
// kernel, launched with programmatic stream serialization so that its start-up overlaps
// this kernel's tail, merges the partials.  No CTA waits for another.
//
// The arithmetic intensity is G flop per byte: HBM-bound by a wide margin, so the
// design goal is bytes in flight (ring of Hkv*8 KB stages), not tensor throughput.
#include "pi_common.cuh"
#include "pi_attn_core.cuh"

namespace {

using namespace pi_attn;

constexpr int ATTN_META_UNITS = 1024;              // units per CTA whose metadata is staged in shared memory
constexpr int ATTN_SMEM_BUDGET = 196 * 1024;       // ring bytes
constexpr int MERGE_BATCH = 12;                    // partial outputs a lane of the merge kernel has in flight

// CTA that owns unit u when U units are split over P CTAs as [U*c/P, U*(c+1)/P).
__device__ __forceinline__ int cta_of_unit(long long u, long long U, long long P) {
    long long c = (u * P) / U;
    while ((U * (c + 1)) / P <= u) ++c;
    while ((U * c) / P > u) --c;
    return static_cast<int>(c);
}

__device__ __forceinline__ int seq_of_unit(const int* pref, int batch, int u) {
    int lo = 0, hi = batch;                          // last s with pref[s] <= u
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pref[mid] <= u) lo = mid; else hi = mid;
    }
    return lo;
}

// Second kernel of the attention call: merges the split-K partials of every sequence that
// was cut across CTAs.  Grid (Hkv, batch), one warp per query head, lane = 4 channels.  It is
// launched with programmatic stream serialization: its CTAs may start while the main kernel
// still runs, work out which partials belong to their sequence (same split arithmetic as the
// main kernel), and only then wait for the main grid to complete and flush.
__global__ void __launch_bounds__(512)
attn_merge_kernel(AttnParams p, int main_ctas) {
    __shared__ int s_red[3][16];
    const int seq = blockIdx.y, h = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int SUB = p.B >> 4;
    // units before this sequence, of this sequence, and in total
    int before = 0, mine = 0, total = 0;
    for (int s = threadIdx.x; s < p.batch; s += blockDim.x) {
        int n = blocks_of_seq(p, s) * SUB;
        total += n;
        if (s < seq) before += n;
        if (s == seq) mine = n;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        mine += __shfl_xor_sync(0xffffffffu, mine, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if (lane == 0) { s_red[0][warp] = before; s_red[1][warp] = mine; s_red[2][warp] = total; }
    __syncthreads();
    before = mine = total = 0;
    for (int w = 0; w < n_warps; ++w) { before += s_red[0][w]; mine += s_red[1][w]; total += s_red[2][w]; }
    const long long U = total, P = min(static_cast<long long>(main_ctas), max(U, 1ll));
    int c_first = 0, n_seg = 0;
    if (mine > 0) {
        c_first = cta_of_unit(before, U, P);
        n_seg = cta_of_unit(before + mine - 1, U, P) - c_first + 1;
    }
    // Every CTA executes the wait, also the ones with nothing to merge: a dependent grid that retired
    // without waiting would let the stream move on while the main grid is still writing.
    pi_grid_dependency_wait();                                // main grid complete, its stores visible
    if (mine == 0) return;                                    // nothing selected: the main kernel wrote zeros
    if (n_seg == 1) return;                                   // one CTA covered the sequence and wrote the result

    const size_t slot0 = static_cast<size_t>(c_first) + seq;
    for (int g = warp; g < p.G; g += n_warps) {
        const size_t head = static_cast<size_t>(h) * p.G + g;
        // lane i holds (m, l) of segment i (+32, +64, ...).  The first MERGE_BATCH partial outputs are
        // requested in the same breath (they do not depend on the weights), so a sequence cut into
        // up to that many segments costs one round trip to L2.
        float2 ml0 = make_float2(-INFINITY, 0.f);
        float M = -INFINITY;
        for (int sg = lane; sg < n_seg; sg += 32) {
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + ((slot0 + sg) * p.Hq + head) * 2));
            if (sg < 32) ml0 = ml;
            M = fmaxf(M, ml.x);
        }
        float4 v[MERGE_BATCH];
        auto fetch = [&](int first, int end) {       // segments [first, first + MERGE_BATCH) below `end`
#pragma unroll
            for (int kk = 0; kk < MERGE_BATCH; ++kk) {
                v[kk] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (first + kk < end)
                    v[kk] = __ldcg(reinterpret_cast<const float4*>(p.part_o + ((slot0 + first + kk) * p.Hq + head) * PI_HEAD_DIM) + lane);
            }
        };
        fetch(0, min(32, n_seg));
#pragma unroll
        for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float L = 0.f;
        for (int s0 = 0; s0 < n_seg; s0 += 32) {
            const int sg = s0 + lane;
            float w = 0.f;
            if (sg < n_seg) {
                const float2 ml = s0 == 0 ? ml0
                    : __ldcg(reinterpret_cast<const float2*>(p.part_ml + ((slot0 + sg) * p.Hq + head) * 2));
                w = ml.x == -INFINITY ? 0.f : exp2f(ml.x - M);
                L += w * ml.y;
            }
            const int cnt = min(32, n_seg - s0);
            for (int k = 0; k < cnt; k += MERGE_BATCH) {
                if (s0 + k > 0) fetch(s0 + k, s0 + cnt);
#pragma unroll
                for (int kk = 0; kk < MERGE_BATCH; ++kk) {
                    const float wk = __shfl_sync(0xffffffffu, w, (k + kk) & 31);
                    acc.x += wk * v[kk].x; acc.y += wk * v[kk].y; acc.z += wk * v[kk].z; acc.w += wk * v[kk].w;
                }
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
        const float inv = L > 0.f ? 1.f / L : 0.f;
        const size_t gh = static_cast<size_t>(seq) * p.Hq + head;
        __nv_bfloat162 lo2 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
        __nv_bfloat162 hi2 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo2);
        pk.y = *reinterpret_cast<uint32_t*>(&hi2);
        *reinterpret_cast<uint2*>(p.out + gh * PI_HEAD_DIM + lane * 4) = pk;
        if (p.lse && lane == 0) p.lse[gh] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
    }
}

// HW = false: one selection per sequence, a stage is one TMA box pair covering all KV heads of a block.
// HW = true: every KV head has its own selection (the headwise strategy of Sec. 4.4.1): a stage holds,
// for each head, the (K, V) fragment of that head's own j-th selected block, fetched with a box of two
// rows of the head dimension (pool_map then has box {64, 16, 2, 1}); consumer warp h sees the same stage
// layout either way.
template <int NT, bool HW>
__global__ void __launch_bounds__(288, 1)
attn_kernel(const __grid_constant__ CUtensorMap pool_map, AttnParams p) {
    extern __shared__ unsigned char smem_dyn[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int stage_bytes = p.Hkv * 8192, half_bytes = p.Hkv * 4096;
    const uint32_t ring = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* after_ring = smem_dyn + (ring - smem_u32(smem_dyn)) + static_cast<size_t>(p.stages) * stage_bytes;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(after_ring);      // full[8], empty[8], seg
    int* s_nvalid = reinterpret_cast<int*>(bars + 2 * ATTN_MAX_STAGES + 1);            // [8 stages][8 heads]
    int* s_abort = s_nvalid + ATTN_MAX_STAGES * 8;
    int* s_last = s_abort + 1;
    int2* s_meta = reinterpret_cast<int2*>(s_last + 1);                                // [ATTN_META_UNITS] {slot row, sub*16 | nvalid<<8}
    int* s_pref = reinterpret_cast<int*>(s_meta + ATTN_META_UNITS);                    // [batch + 1]
    const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + ATTN_MAX_STAGES);
    const int SUB = p.B >> 4;
    if (tid == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&pool_map) : "memory");
    pi_grid_dependency_wait();
    // the merge kernel that follows in the stream may be scheduled from now on; it waits for this
    // grid to finish before it reads anything this grid writes
    pi_launch_dependents();

    // ---- unit prefix over sequences (every CTA computes the same table)
    for (int s = tid; s < p.batch; s += blockDim.x) {
        if (blockIdx.x == 0) {
            const int lists = HW ? p.Hkv : 1;
            for (int i = 0; i < lists; ++i) {
                const int n = p.sel_count[s * lists + i];
                if (n < 0 || n > p.K) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_ATTN, s, n, p.K);
            }
        }
        s_pref[s + 1] = blocks_of_seq(p, s) * SUB;
    }
    if (tid == 0) {
        s_pref[0] = 0;
        *s_abort = 0;
        for (int i = 0; i < p.stages; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, p.Hkv);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {                                   // inclusive scan in place, 32 entries a time
        int run = 0;
        for (int s0 = 0; s0 < p.batch; s0 += 32) {
            const int s = s0 + lane;
            int v = s < p.batch ? s_pref[s + 1] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v += t;
            }
            if (s < p.batch) s_pref[s + 1] = run + v;
            run += __shfl_sync(0xffffffffu, v, 31);
        }
    }
    __syncthreads();

    // never more CTAs than units: then every CTA in [0, P) owns at least one unit, which the
    // segment count of a sequence (last owner - first owner + 1) relies on
    const long long U = s_pref[p.batch], P = min(static_cast<long long>(gridDim.x), max(U, 1ll));
    // sequences with nothing selected: defined output, written by CTA 0
    if (blockIdx.x == 0) {
        for (int s = 0; s < p.batch; ++s) {
            if (s_pref[s + 1] != s_pref[s]) continue;
            for (int i = tid; i < p.Hq * PI_HEAD_DIM; i += blockDim.x)
                p.out[static_cast<size_t>(s) * p.Hq * PI_HEAD_DIM + i] = __float2bfloat16(0.f);
            if (p.lse)
                for (int i = tid; i < p.Hq; i += blockDim.x) p.lse[static_cast<size_t>(s) * p.Hq + i] = -INFINITY;
        }
    }
    if (U == 0 || blockIdx.x >= P) return;
    const int u0 = static_cast<int>((U * blockIdx.x) / P), u1 = static_cast<int>((U * (blockIdx.x + 1)) / P);
    if (u0 >= u1) return;

    // ---- metadata of this CTA's units: global row of the slot, token offset, valid tokens.
    // Staged up front by all threads so the producer never waits on a dependent global load.
    // hh: the KV head whose list is read (ignored when all heads share one selection)
    auto unit_meta = [&](int u, int seq, int hh) -> int2 {
        const int r = u - s_pref[seq], j = r / SUB, sub = r - j * SUB;
        const size_t list = HW ? static_cast<size_t>(seq) * p.Hkv + hh : static_cast<size_t>(seq);
        int jj = j;
        bool empty = false;
        if (HW) {                                    // a head with a shorter list: an empty tile of its first block
            const int cnt = p.sel_count[list];
            if (cnt < 0 || cnt > p.K || j >= cnt) { empty = true; jj = 0; }
        }
        int slot = p.sel_slots[list * p.K + jj];
        const int blk = p.sel_blocks[list * p.K + jj];
        if (slot < 0 || slot >= p.C) {
            if (!empty) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_ATTN, seq, j, slot);
            slot = 0;
            empty = HW ? true : empty;
        }
        const int nvalid = (blk < 0 || empty) ? 0 : max(0, min(16, p.ctx_len[seq] - (blk * p.B + sub * 16)));
        return make_int2(seq * p.C + slot, (sub * 16) | (nvalid << 8));
    };
    const int meta_per_unit = HW ? p.Hkv : 1;
    const int meta_units = ATTN_META_UNITS / meta_per_unit;
    for (int i = tid; i < (u1 - u0) * meta_per_unit && i < meta_units * meta_per_unit; i += blockDim.x) {
        const int ui = i / meta_per_unit, hh = i - ui * meta_per_unit;
        s_meta[i] = unit_meta(u0 + ui, seq_of_unit(s_pref, p.batch, u0 + ui), hh);
    }
    __syncthreads();

    if (warp == p.Hkv) {
        // =============================== producer: one lane issues all TMA loads
        if (lane == 0) {
            const unsigned long long stream_policy = pi_l2_stream_policy();
            int seq = seq_of_unit(s_pref, p.batch, u0);
            for (int u = u0, it = 0; u < u1; ++u, ++it) {
                while (u >= s_pref[seq + 1]) ++seq;
                const int st = it % p.stages, round = it / p.stages;
                if (round > 0 && !mbar_wait(bar_empty + 8 * st, (round - 1) & 1, s_abort, p.wait_cycles)) break;
                if (p.hold_last && u == u1 - 1) break;           // (test only) the consumers' wait for this unit runs out
                const uint32_t dst = ring + st * stage_bytes;
                // valid-token counts are written before the arrive below, which publishes them
                if (HW) {
                    int rows[8], offs[8];
                    for (int hh = 0; hh < p.Hkv; ++hh) {
                        const int2 md = it < meta_units ? s_meta[it * p.Hkv + hh] : unit_meta(u, seq, hh);
                        s_nvalid[st * 8 + hh] = md.y >> 8;
                        rows[hh] = md.x; offs[hh] = md.y & 0xff;
                    }
                    mbar_expect_tx(bar_full + 8 * st, stage_bytes);
                    for (int hh = 0; hh < p.Hkv; ++hh) {
                        tma_load_4d(dst + hh * 4096, &pool_map, bar_full + 8 * st, 0, offs[hh], 2 * hh, rows[hh], stream_policy);
                        tma_load_4d(dst + half_bytes + hh * 4096, &pool_map, bar_full + 8 * st, 64, offs[hh], 2 * hh, rows[hh], stream_policy);
                    }
                } else {
                    const int2 md = it < meta_units ? s_meta[it] : unit_meta(u, seq, 0);
                    s_nvalid[st * 8] = md.y >> 8;
                    mbar_expect_tx(bar_full + 8 * st, stage_bytes);
                    tma_load_4d(dst, &pool_map, bar_full + 8 * st, 0, md.y & 0xff, 0, md.x, stream_policy);
                    tma_load_4d(dst + half_bytes, &pool_map, bar_full + 8 * st, 64, md.y & 0xff, 0, md.x, stream_policy);
                }
            }
        }
        return;
    }
    if (warp > p.Hkv) return;

    // =============================== consumers: warp h owns kv head h
    const int h = warp;
    const int row = lane >> 2, colp = (lane & 3) * 2;
    int seq = seq_of_unit(s_pref, p.batch, u0);
    // per-lane ldmatrix offsets inside a stage (swizzled 128-byte rows)
    const int r8 = lane & 7, mi = lane >> 3;
    const int tK = r8 + 8 * (mi & 1), cK = mi >> 1;         // K as A operand (rows = tokens)
    const int tV = r8 + 8 * (mi >> 1), cV = mi & 1;         // V^T as A operand via .trans
    const uint32_t offK = (2 * h) * 2048 + tK * 128, offV = (2 * h + 1) * 2048 + tV * 128;
    bool alive = true;

    // One iteration per (CTA, sequence) segment: the running softmax state lives only inside it.
    for (int u = u0, it = 0; u < u1 && alive;) {
        while (u >= s_pref[seq + 1]) ++seq;
        const int seg_end = min(u1, s_pref[seq + 1]);
        uint32_t bq[NT][8][2];
        float o[NT][8][4], m[NT][2], l[NT][2];
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
      for (; u < seg_end; ++u, ++it) {
        const int st = it % p.stages;
        if (!mbar_wait(bar_full + 8 * st, (it / p.stages) & 1, s_abort, p.wait_cycles)) { alive = false; break; }
        const int nvalid = s_nvalid[st * 8 + (HW ? h : 0)];
        const uint32_t base = ring + st * stage_bytes;

        attn_tile<NT>(base, half_bytes, offK, offV, r8, cK, cV, row, nvalid, p.scale_log2, bq, o, m, l);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * st);
      }
        if (!alive) break;

        // ---- end of this CTA's segment of the sequence
        {
            const int c_first = cta_of_unit(s_pref[seq], U, P), c_last = cta_of_unit(s_pref[seq + 1] - 1, U, P);
            const int n_seg = c_last - c_first + 1;
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
            if (n_seg == 1) {
                attn_write_out<NT>(p, seq, h, row, colp, o, m, l);
            } else {
                const size_t pslot = static_cast<size_t>(blockIdx.x) + seq;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int g = nt * 8 + colp + e;
                        if (g >= p.G) continue;
                        const size_t gh = pslot * p.Hq + static_cast<size_t>(h) * p.G + g;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            p.part_o[gh * PI_HEAD_DIM + 16 * i + row] = o[nt][i][e];
                            p.part_o[gh * PI_HEAD_DIM + 16 * i + row + 8] = o[nt][i][e + 2];
                        }
                        if (row == 0) { p.part_ml[gh * 2] = m[nt][e]; p.part_ml[gh * 2 + 1] = l[nt][e]; }
                    }
            }
        }
    }
    if (*s_abort && lane == 0 && warp == 0) pi_report(p.st, PI_ERR_TIMEOUT, PI_STAGE_ATTN, blockIdx.x, u0, u1);
}

}  // namespace

int pi_launch_attn(pi_ctx* c, int batch, const void* q, const void* pool, const int32_t* sel_slots,
                   const int32_t* sel_blocks, const int32_t* sel_count, const int32_t* ctx_len, void* out,
                   float* lse, int headwise, cudaStream_t stream) {
    const pi_config& cfg = c->cfg;
    if (cfg.n_kv_heads > 8) return PI_ERR_UNSUPPORTED_DIM;
    // the head-major form keeps everything inside the CTA (no partials, no merge kernel); it is taken when
    // (sequences x KV heads) fills the grid evenly, or when the configuration asks for it
    if (cfg.attn_mode == 2 || (cfg.attn_mode == 0 && pi_attn_headmajor_fits(c, batch, nullptr, nullptr, nullptr)))
        return pi_launch_attn_headmajor(c, batch, q, pool, sel_slots, sel_blocks, sel_count, ctx_len, out, lse, headwise, nullptr, stream);
    const long long n_slots = static_cast<long long>(batch) * cfg.pool_slots;
    // the map is rebuilt when the pool, its size or the box (all heads / one head per load) changes
    if (c->pool_map_ptr != pool || c->pool_map_slots != n_slots || c->pool_map_headwise != headwise) {
        typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        const cuuint64_t B = cfg.block_tokens, hk = 2ull * cfg.n_kv_heads;
        cuuint64_t gdim[4] = {PI_HEAD_DIM, B, hk, static_cast<cuuint64_t>(n_slots)};
        cuuint64_t gstride[3] = {PI_HEAD_DIM * 2ull, B * PI_HEAD_DIM * 2ull, hk * B * PI_HEAD_DIM * 2ull};
        cuuint32_t box[4] = {64, 16, headwise ? 2u : static_cast<cuuint32_t>(hk), 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = reinterpret_cast<encode_fn>(c->encode_tiled_fn)(
            &c->pool_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { c->pool_map_ptr = nullptr; return PI_ERR_CUDA; }
        c->pool_map_ptr = pool;
        c->pool_map_slots = n_slots;
        c->pool_map_headwise = headwise;
    }
    AttnParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.sel_slots = sel_slots; p.sel_blocks = sel_blocks; p.sel_count = sel_count; p.ctx_len = ctx_len;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.part_o = c->attn_part_o; p.part_ml = c->attn_part_ml; p.counters = c->attn_counters;
    p.st = pi_status_of(c);
    p.batch = batch; p.Hq = cfg.n_q_heads; p.Hkv = cfg.n_kv_heads; p.G = cfg.n_q_heads / cfg.n_kv_heads;
    p.B = cfg.block_tokens; p.K = cfg.budget_blocks; p.C = cfg.pool_slots;
    p.headwise = headwise ? 1 : 0;
    p.hold_last = cfg.test_hold_producer;
    p.wait_cycles = c->wait_limit_cycles;
    const int stage_bytes = cfg.n_kv_heads * 8192;
    int stages = ATTN_SMEM_BUDGET / stage_bytes;
    if (stages > ATTN_MAX_STAGES) stages = ATTN_MAX_STAGES;
    p.stages = stages;
    p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(PI_HEAD_DIM));
    const size_t smem = 1024 + static_cast<size_t>(stages) * stage_bytes + (2 * ATTN_MAX_STAGES + 1) * 8 +
                        (ATTN_MAX_STAGES * 8 + 2) * 4 + ATTN_META_UNITS * 8 + (static_cast<size_t>(batch) + 1) * 4 + 16;
    const int threads = (cfg.n_kv_heads + 1) * 32;
    auto launch = [&](auto kernel) -> int {
        PI_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        PI_CUDA_TRY(pi_launch_pdl(kernel, dim3(c->attn_ctas), dim3(threads), smem, stream, c->pool_map, p));
        return PI_OK;
    };
    int rc;
    if (headwise) rc = p.G <= 8 ? launch(attn_kernel<1, true>) : launch(attn_kernel<2, true>);
    else rc = p.G <= 8 ? launch(attn_kernel<1, false>) : launch(attn_kernel<2, false>);
    if (rc != PI_OK) return rc;
    PI_CUDA_TRY(cudaGetLastError());
    // merge of the split sequences: may start early, synchronises on the grid above by itself
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(cfg.n_kv_heads, batch);
    lc.blockDim = dim3(32 * (p.G < 16 ? p.G : 16));
    lc.dynamicSmemBytes = 0;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    PI_CUDA_TRY(cudaLaunchKernelEx(&lc, attn_merge_kernel, p, c->attn_ctas));
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
