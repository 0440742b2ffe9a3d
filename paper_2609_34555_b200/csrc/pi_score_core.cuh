// Scoring arithmetic shared by the selection kernels: the order-preserving key of an fp32 score,
// the streaming 16-byte load, the per-lane part of the 256-long dot product of one block's digest
// with the summed positive / negative query parts, and the transposed warp reduction.  Both
// kernels that score (the ticket kernel and the cluster kernel) use exactly these routines, so
// their scores agree bit for bit.
#pragma once

#include "pi_common.cuh"

namespace pi_score {

constexpr int BLOCKS_PER_WARP = 8;               // 8 independent 16-byte loads per lane per group of blocks

// Shared arrays that one thread walks with a stride of several words are stored with one
// pad word every 32 entries, which keeps both the strided and the unit-stride walks free
// of bank conflicts.
__device__ __forceinline__ int padded(int i) { return i + (i >> 5); }

__device__ __forceinline__ uint32_t float_key(float s) {
    uint32_t u = __float_as_uint(s + 0.0f);       // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ uint4 ld_stream16(const uint4* p, unsigned long long policy) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy));
    return v;
}

__device__ __forceinline__ float dot8(uint4 v, const float (&w)[8]) {
    float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v.x));
    float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v.y));
    float2 c = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v.z));
    float2 d = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v.w));
    float s0 = a.x * w[0] + b.x * w[2];
    float s1 = a.y * w[1] + b.y * w[3];
    s0 = fmaf(c.x, w[4], s0); s1 = fmaf(c.y, w[5], s1);
    s0 = fmaf(d.x, w[6], s0); s1 = fmaf(d.y, w[7], s1);
    return s0 + s1;
}

// Weights of this lane's 8 channels: lanes 0-15 hold Q- (the sum over the group's query heads of
// min(q, 0)) for channels 8*lane.., lanes 16-31 hold Q+ for channels 8*(lane-16)...  qh points at
// the first query row of the group; the rows are fetched four at a time so their latencies overlap.
__device__ __forceinline__ void load_q_weights(const __nv_bfloat16* qh, int G, int lane, float (&w)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = 0.f;
    const int d0 = (lane & 15) * 8;
    const bool plus = lane >= 16;
    qh += d0;
    for (int g0 = 0; g0 < G; g0 += 4) {
        uint4 qv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            qv[j] = make_uint4(0, 0, 0, 0);
            if (g0 + j < G) qv[j] = *reinterpret_cast<const uint4*>(qh + static_cast<size_t>(g0 + j) * PI_HEAD_DIM);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&qv[j]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float2 fv = __bfloat1622float2(h2[i]);
                w[2 * i] += plus ? fmaxf(fv.x, 0.f) : fminf(fv.x, 0.f);
                w[2 * i + 1] += plus ? fmaxf(fv.y, 0.f) : fminf(fv.y, 0.f);
            }
        }
    }
}

// Transposed warp reduction: 8 partial sums per lane x 32 lanes -> the four lanes of group
// (lane >> 2) all end up with the full sum of block (lane >> 2); 9 shuffles for 8 blocks.
__device__ __forceinline__ float reduce8(float (&s)[BLOCKS_PER_WARP], int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const bool up = lane & 16;
        float send = up ? s[i] : s[i + 4];
        float keep = up ? s[i + 4] : s[i];
        s[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const bool up = lane & 8;
        float send = up ? s[i] : s[i + 2];
        float keep = up ? s[i + 2] : s[i];
        s[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    {
        const bool up = lane & 4;
        float send = up ? s[0] : s[1];
        float keep = up ? s[1] : s[0];
        s[0] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    s[0] += __shfl_xor_sync(0xffffffffu, s[0], 2);
    s[0] += __shfl_xor_sync(0xffffffffu, s[0], 1);
    return s[0];
}

}  // namespace pi_score
