// Pieces shared by the attention kernels: parameters, PTX wrappers (mbarrier, tiled TMA load, ldmatrix,
// movmatrix, bf16 mma), the arithmetic of one 16-token tile of one KV head, and the final write of a
// warp's query heads.
#pragma once

#include "pi_common.cuh"

namespace pi_attn {

constexpr int ATTN_MAX_STAGES = 8;

struct AttnParams {
    const __nv_bfloat16* q;
    const int32_t* sel_slots;
    const int32_t* sel_blocks;
    const int32_t* sel_count;
    const int32_t* ctx_len;
    __nv_bfloat16* out;
    float* lse;
    float* part_o;
    float* part_ml;
    unsigned int* counters;
    pi_status_ref st;
    int batch, Hq, Hkv, G, B, K, C, stages;
    int headwise;                 // 1: sel_slots / sel_blocks are [batch][Hkv][K], sel_count [batch][Hkv]
    int hold_last;                // test only: the producer never issues the loads of its CTA's last unit
    long long wait_cycles;        // bound of every wait on a barrier
    float scale_log2;
    // attention split around the recall (head-major form only): the step's recall list names the slots that are
    // being filled; `state` carries the softmax state of the first call to the second
    const pi_extent* rlist;
    const int32_t* rcount;
    int rcap;
    float* state;                 // [items][NT * 36][32] fp32, a warp's state as the merge regions hold it
};

// Blocks of sequence s that the unit list walks: the selection's count, or, when every KV head has
// its own selection, the largest count over the heads (a head with fewer blocks sees empty tiles).
// Counts outside [0, K] read as 0 (the main kernel reports them).
__device__ __forceinline__ int blocks_of_seq(const AttnParams& p, int s) {
    if (!p.headwise) {
        const int n = p.sel_count[s];
        return (n < 0 || n > p.K) ? 0 : n;
    }
    int n = 0;
    for (int h = 0; h < p.Hkv; ++h) {
        const int c = p.sel_count[s * p.Hkv + h];
        if (c >= 0 && c <= p.K) n = max(n, c);
    }
    return n;
}

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up when another warp raised `abort` or the cycle limit passes.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, long long limit) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity)) return true;
        if (*abort) return false;
        if (clock64() - t0 > limit) { *abort = 1; return false; }
    }
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3,
                                            unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t movm_t(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}


// One 16-token tile of one KV head (K and V rows in a stage of the ring, 128-byte swizzled halves of the
// head dimension) for the G query heads of this warp:  S^T = K q^T  (tokens on M, heads on N),
// online softmax over the tokens, O^T += V^T P.  State: o (accumulators), m (running maxima, exp2
// domain), l (per-lane partial sums of the weights).
template <int NT>
__device__ __forceinline__ void attn_tile(uint32_t base, int half_bytes, uint32_t offK, uint32_t offV, int r8, int cK, int cV,
                                          int row, int nvalid, float scale_log2, const uint32_t (&bq)[NT][8][2],
                                          float (&o)[NT][8][4], float (&m)[NT][2], float (&l)[NT][2]) {
            // ---- S^T = K q^T
            float c[NT][4];
    #pragma unroll
            for (int nt = 0; nt < NT; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
    #pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t a[4];
                const int chunk = 2 * (j & 3) + cK;
                ldsm_x4(base + (j >> 2) * half_bytes + offK + ((chunk ^ r8) << 4), a);
    #pragma unroll
                for (int nt = 0; nt < NT; ++nt) mma_bf16(c[nt], a, bq[nt][j][0], bq[nt][j][1]);
            }
            // ---- online softmax over tokens (rows), one state per query head (column)
            // P is split into a bf16 head and a bf16 remainder (two MMAs per V tile): value
            // channels with large magnitudes would otherwise see the 2^-9 rounding of P directly.
            uint32_t pb[NT][2], pl[NT][2];
    #pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float pr[4];
    #pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float s0 = row < nvalid ? c[nt][e] * scale_log2 : -INFINITY;
                    float s1 = row + 8 < nvalid ? c[nt][e + 2] * scale_log2 : -INFINITY;
                    float mx = fmaxf(s0, s1);
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                    const float m_new = fmaxf(m[nt][e], mx);
                    float alpha = 1.f, p0 = 0.f, p1 = 0.f;
                    if (m_new != -INFINITY) {
                        alpha = exp2f(m[nt][e] - m_new);
                        p0 = exp2f(s0 - m_new);
                        p1 = exp2f(s1 - m_new);
                    }
                    m[nt][e] = m_new;
                    l[nt][e] = l[nt][e] * alpha + p0 + p1;
                    pr[e] = p0; pr[e + 2] = p1;
    #pragma unroll
                    for (int i = 0; i < 8; ++i) { o[nt][i][e] *= alpha; o[nt][i][e + 2] *= alpha; }
                }
                // P^T fragments (rows = tokens) -> B operand (k = tokens, n = heads)
                const uint32_t h01 = pack_bf16(pr[0], pr[1]), h23 = pack_bf16(pr[2], pr[3]);
                const float2 f01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&h01));
                const float2 f23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&h23));
                pb[nt][0] = movm_t(h01);
                pb[nt][1] = movm_t(h23);
                pl[nt][0] = movm_t(pack_bf16(pr[0] - f01.x, pr[1] - f01.y));
                pl[nt][1] = movm_t(pack_bf16(pr[2] - f23.x, pr[3] - f23.y));
            }
            // ---- O^T += V^T P
    #pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint32_t a[4];
                const int chunk = 2 * (i & 3) + cV;
                ldsm_x4_t(base + (i >> 2) * half_bytes + offV + ((chunk ^ r8) << 4), a);
    #pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mma_bf16(o[nt][i], a, pb[nt][0], pb[nt][1]);
                    mma_bf16(o[nt][i], a, pl[nt][0], pl[nt][1]);
                }
            }
}

// Final result of this warp's query heads: O / l as bf16, and the natural-log-sum-exp.  l must be the
// full sum over the tile rows (reduced over the lanes of a column).
template <int NT>
__device__ __forceinline__ void attn_write_out(const AttnParams& p, int seq, int h, int row, int colp,
                                               const float (&o)[NT][8][4], const float (&m)[NT][2], const float (&l)[NT][2]) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int g = nt * 8 + colp + e;
            if (g >= p.G) continue;
            const size_t gh = static_cast<size_t>(seq) * p.Hq + static_cast<size_t>(h) * p.G + g;
            const float inv = l[nt][e] > 0.f ? 1.f / l[nt][e] : 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                p.out[gh * PI_HEAD_DIM + 16 * i + row] = __float2bfloat16(o[nt][i][e] * inv);
                p.out[gh * PI_HEAD_DIM + 16 * i + row + 8] = __float2bfloat16(o[nt][i][e + 2] * inv);
            }
            if (p.lse && row == 0)
                p.lse[gh] = l[nt][e] > 0.f ? (m[nt][e] + log2f(l[nt][e])) * 0.6931471805599453f : -INFINITY;
        }
}

}  // namespace pi_attn
