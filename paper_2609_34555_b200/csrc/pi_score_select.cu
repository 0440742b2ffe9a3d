// Digest scoring of the retrieval head + exact top-k block selection, one launch.
//
// Grid (chunks, batch): every CTA scores SCORE_CHUNK consecutive blocks of one
// sequence (HBM-bound: 512 B of digest per block), writes fp32 scores, and takes a
// ticket; the CTA that takes the last ticket of a sequence selects for it.  No CTA
// ever waits for another one.
//
// Score of block b (Quest-style min/max digests, summed over the G query heads of
// the retrieval head):  sum_g sum_d max(q_g[d]*min_b[d], q_g[d]*max_b[d])
//   = sum_d Q+[d]*max_b[d] + Q-[d]*min_b[d],  Q+ = sum_g max(q_g,0), Q- = sum_g min(q_g,0)
// so each block costs one 256-long dot product whatever G is.
//
// Selection: sink and local blocks are always taken; among the middle blocks the
// k_mid largest scores win, ties to the lower index.  Keys are the order-preserving
// uint32 images of the fp32 scores; a bucket search over the 11 most significant
// *varying* bits narrows [lo, hi] until the k-th key is isolated, then one ordered
// compaction emits the result in ascending block order.
#include "pi_common.cuh"

namespace {

constexpr int SCORE_THREADS = 256;
constexpr int SCORE_WARPS = SCORE_THREADS / 32;
constexpr int SCORE_CHUNK = 128;                 // blocks per CTA
constexpr int BLOCKS_PER_ITER = 8;               // per warp: 8 independent 16-byte loads per lane
constexpr int BINS = PI_SELECT_BINS;
constexpr int BINS_PER_THREAD = BINS / SCORE_THREADS;

struct SelParams {
    const __nv_bfloat16* q;
    const uint4* digest;
    const int32_t* ctx_len;
    int32_t* sel;
    int32_t* sel_count;
    float* scores;
    unsigned int* counters;
    pi_status_ref st;
    int h_star, Hq, G, B, K, n_sink, n_local, max_blocks;
};

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

// Block-wide exclusive scan helpers (SCORE_THREADS threads, all must call).
__device__ __forceinline__ unsigned block_excl_scan(unsigned v, unsigned* warp_tot, unsigned& total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();                               // warp_tot may still be read from a previous call
    if (lane == 31) warp_tot[w] = inc;
    __syncthreads();
    unsigned base = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < SCORE_WARPS; ++i) {
        unsigned t = warp_tot[i];
        if (i < w) base += t;
        tot += t;
    }
    total = tot;
    return base + inc - v;
}

__global__ void __launch_bounds__(SCORE_THREADS)
score_select_kernel(SelParams p) {
    extern __shared__ uint32_t keys[];             // [n_blocks] in the selecting CTA
    __shared__ unsigned hist[BINS];
    __shared__ unsigned warp_tot[SCORE_WARPS];
    __shared__ uint32_t red_lo[SCORE_WARPS], red_hi[SCORE_WARPS];
    __shared__ uint32_t sh_lo, sh_hi;
    __shared__ unsigned sh_need, sh_cnt;
    __shared__ int sh_last;

    const int seq = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int ctx = p.ctx_len[seq];
    if (ctx < 0) ctx = 0;
    int n_blocks = (ctx + p.B - 1) / p.B;
    if (n_blocks > p.max_blocks) {
        if (tid == 0 && blockIdx.x == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_SELECT, seq, n_blocks, p.max_blocks);
        n_blocks = p.max_blocks;
    }

    // ---------------- phase 1: scores of this CTA's chunk
    const int c0 = blockIdx.x * SCORE_CHUNK;
    if (c0 < n_blocks) {
        // lanes 0-15 hold Q- for channels 8*lane.., lanes 16-31 hold Q+ for channels 8*(lane-16)..
        float w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = 0.f;
        const int d0 = (lane & 15) * 8;
        const bool plus = lane >= 16;
        const __nv_bfloat16* qh = p.q + (static_cast<size_t>(seq) * p.Hq + static_cast<size_t>(p.h_star) * p.G) * PI_HEAD_DIM + d0;
        for (int g = 0; g < p.G; ++g) {
            uint4 v = *reinterpret_cast<const uint4*>(qh + static_cast<size_t>(g) * PI_HEAD_DIM);
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float2 f = __bfloat1622float2(h2[i]);
                w[2 * i] += plus ? fmaxf(f.x, 0.f) : fminf(f.x, 0.f);
                w[2 * i + 1] += plus ? fmaxf(f.y, 0.f) : fminf(f.y, 0.f);
            }
        }
        const uint4* dg = p.digest + static_cast<size_t>(seq) * p.max_blocks * 32;   // 32 uint4 per block
        for (int b0 = c0 + warp * BLOCKS_PER_ITER; b0 < c0 + SCORE_CHUNK && b0 < n_blocks;
             b0 += SCORE_WARPS * BLOCKS_PER_ITER) {
            uint4 v[BLOCKS_PER_ITER];
#pragma unroll
            for (int i = 0; i < BLOCKS_PER_ITER; ++i) {
                v[i] = make_uint4(0, 0, 0, 0);
                if (b0 + i < n_blocks) v[i] = ld_stream16(dg + static_cast<size_t>(b0 + i) * 32 + lane);
            }
            float s[BLOCKS_PER_ITER];
#pragma unroll
            for (int i = 0; i < BLOCKS_PER_ITER; ++i) s[i] = dot8(v[i], w);
            // transposed warp reduction: 8 values x 32 lanes -> lane group (lane>>2) owns block (lane>>2)
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
            const int b = b0 + (lane >> 2);
            if ((lane & 3) == 0 && b < n_blocks) p.scores[static_cast<size_t>(seq) * p.max_blocks + b] = s[0];
        }
    }

    // ---------------- ticket: the last CTA of the sequence selects
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned t = atomicAdd(&p.counters[seq], 1u);
        sh_last = (t == gridDim.x - 1);
        if (sh_last) p.counters[seq] = 0;           // ready for the next launch
    }
    __syncthreads();
    if (!sh_last) return;
    __threadfence();

    // ---------------- phase 2: selection
    const int m_lo = min(p.n_sink, n_blocks);
    const int m_hi = max(n_blocks - p.n_local, m_lo);
    const int n_mid = m_hi - m_lo;
    const int k_mid = p.K - p.n_sink - p.n_local;
    const unsigned k = static_cast<unsigned>(min(k_mid, n_mid));

    uint32_t kmin = 0xffffffffu, kmax = 0u;
    const float* sc = p.scores + static_cast<size_t>(seq) * p.max_blocks;
    for (int i = tid; i < n_blocks; i += SCORE_THREADS) {
        uint32_t key = float_key(__ldcg(sc + i));
        keys[i] = key;
        if (i >= m_lo && i < m_hi) { kmin = min(kmin, key); kmax = max(kmax, key); }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane == 0) { red_lo[warp] = kmin; red_hi[warp] = kmax; }
    __syncthreads();
    if (tid == 0) {
        uint32_t a = red_lo[0], b = red_hi[0];
        for (int i = 1; i < SCORE_WARPS; ++i) { a = min(a, red_lo[i]); b = max(b, red_hi[i]); }
        sh_lo = a; sh_hi = b; sh_need = k; sh_cnt = static_cast<unsigned>(n_mid);
    }
    __syncthreads();

    // Narrow [lo, hi] until keys > hi are all winners and the first `need` keys (by index)
    // inside [lo, hi] complete the set.
    uint32_t lo = sh_lo, hi = sh_hi;
    unsigned need = k;
    if (k > 0 && k < static_cast<unsigned>(n_mid)) {
        for (int pass = 0; pass < 4; ++pass) {
            const uint32_t range = hi - lo;
            if (range == 0) break;                   // every key left is equal: ties by index
            const int bits = 32 - __clz(range);
            const int shift = bits > 11 ? bits - 11 : 0;
            for (int i = tid; i < BINS; i += SCORE_THREADS) hist[i] = 0;
            __syncthreads();
            for (int i = m_lo + tid; i < m_hi; i += SCORE_THREADS) {
                const uint32_t key = keys[i];
                if (key >= lo && key <= hi) atomicAdd(&hist[(key - lo) >> shift], 1u);
            }
            __syncthreads();
            // suffix sums from the top bin: thread t owns bins [t*BPT, t*BPT+BPT), reversed order
            const int top = BINS - 1 - tid * BINS_PER_THREAD;          // my highest bin
            unsigned local = 0;
#pragma unroll
            for (int j = 0; j < BINS_PER_THREAD; ++j) local += hist[top - j];
            unsigned total;
            const unsigned above = block_excl_scan(local, warp_tot, total);  // keys in bins above mine
            if (above < need && need <= above + local) {
                unsigned acc = above;
                for (int j = 0; j < BINS_PER_THREAD; ++j) {
                    const unsigned h = hist[top - j];
                    if (need <= acc + h) {
                        const uint32_t nlo = lo + (static_cast<uint32_t>(top - j) << shift);
                        const uint32_t span = shift ? ((1u << shift) - 1u) : 0u;
                        sh_lo = nlo;
                        sh_hi = (hi - nlo < span) ? hi : nlo + span;
                        sh_need = need - acc;
                        sh_cnt = h;
                        break;
                    }
                    acc += h;
                }
            }
            __syncthreads();
            lo = sh_lo; hi = sh_hi; need = sh_need;
            const unsigned cnt = sh_cnt;
            if (shift == 0 || cnt == need) break;
        }
    } else if (k == 0) {
        lo = 0xffffffffu; hi = 0xffffffffu; need = 0;       // nothing from the middle (keys are never all-ones for finite scores)
        // keys equal to 0xffffffff cannot occur for finite scores; `need` = 0 excludes them anyway
    } else {
        need = static_cast<unsigned>(n_mid);                // everything: [lo, hi] already spans all keys
    }

    // ordered compaction: thread owns a run of consecutive block indices
    const int ipt = (n_blocks + SCORE_THREADS - 1) / SCORE_THREADS;
    const int i0 = tid * ipt, i1 = min(i0 + ipt, n_blocks);
    unsigned c_sure = 0, c_eq = 0;
    for (int i = i0; i < i1; ++i) {
        if (i < m_lo || i >= m_hi) { ++c_sure; continue; }
        const uint32_t key = keys[i];
        if (k > 0 && key > hi) ++c_sure;
        else if (k > 0 && key >= lo) ++c_eq;
    }
    unsigned total;
    const unsigned before = block_excl_scan(c_sure | (c_eq << 16), warp_tot, total);
    unsigned sure_b = before & 0xffffu, eq_b = before >> 16;
    int32_t* out = p.sel + static_cast<size_t>(seq) * p.K;
    for (int i = i0; i < i1; ++i) {
        bool take;
        unsigned pos = sure_b + min(eq_b, need);
        if (i < m_lo || i >= m_hi) { take = true; ++sure_b; }
        else {
            const uint32_t key = keys[i];
            if (k > 0 && key > hi) { take = true; ++sure_b; }
            else if (k > 0 && key >= lo) { take = eq_b < need; ++eq_b; }
            else take = false;
        }
        if (take && pos < static_cast<unsigned>(p.K)) out[pos] = i;
    }
    const unsigned n_sel = min((total & 0xffffu) + min(total >> 16, need), static_cast<unsigned>(p.K));
    for (int i = n_sel + tid; i < p.K; i += SCORE_THREADS) out[i] = -1;
    if (tid == 0) p.sel_count[seq] = static_cast<int32_t>(n_sel);
}

}  // namespace

int pi_launch_score_select(pi_ctx* c, int h_star, int batch, const void* q, const void* digest,
                           const int32_t* ctx_len, int32_t* sel, int32_t* sel_count, float* scores,
                           unsigned int* counters, cudaStream_t stream) {
    SelParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.digest = static_cast<const uint4*>(digest);
    p.ctx_len = ctx_len;
    p.sel = sel;
    p.sel_count = sel_count;
    p.scores = scores;
    p.counters = counters;
    p.st = pi_status_of(c);
    p.h_star = h_star;
    p.Hq = c->cfg.n_q_heads;
    p.G = c->cfg.n_q_heads / c->cfg.n_kv_heads;
    p.B = c->cfg.block_tokens;
    p.K = c->cfg.budget_blocks;
    p.n_sink = c->cfg.n_sink_blocks;
    p.n_local = c->cfg.n_local_blocks;
    p.max_blocks = c->cfg.max_blocks;
    const size_t smem = static_cast<size_t>(c->cfg.max_blocks) * sizeof(uint32_t);
    if (smem > 40 * 1024)
        PI_CUDA_TRY(cudaFuncSetAttribute(score_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    dim3 grid((c->cfg.max_blocks + SCORE_CHUNK - 1) / SCORE_CHUNK, batch);
    score_select_kernel<<<grid, SCORE_THREADS, smem, stream>>>(p);
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
