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
#include "pi_score_core.cuh"

namespace {

using pi_score::BLOCKS_PER_WARP;
using pi_score::dot8;
using pi_score::float_key;
using pi_score::ld_stream16;
using pi_score::padded;

constexpr int SCORE_THREADS = 512;
constexpr int SCORE_WARPS = SCORE_THREADS / 32;
constexpr int SCORE_CHUNK = SCORE_WARPS * BLOCKS_PER_WARP;   // 128 blocks (64 KB of digests) per CTA
constexpr int BINS = PI_SELECT_BINS;
constexpr int BINS_PER_THREAD = BINS / SCORE_THREADS;
constexpr int RESOLVE_MAX = 32;                  // bucket sizes one warp resolves by direct ranking

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
    int batch, per;                                // (virtual) sequences in the launch, chunks per CTA
    // Which KV heads are scored.  A "virtual sequence" v is (sequence v / vh, slice v % vh); its score
    // sums n_sum heads starting at h_base + (v % vh) * hv_step; digests hold dig_heads heads per block.
    //   retrieval head only: vh 1, n_sum 1, h_base = that head, dig_heads 1
    //   averaged:            vh 1, n_sum Hkv, h_base 0,         dig_heads Hkv
    //   headwise:            vh Hkv, n_sum 1, h_base 0, hv_step 1, dig_heads Hkv
    int vh, n_sum, h_base, hv_step, dig_heads;
};

// Block-wide exclusive scan (SCORE_THREADS threads, all must call).
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
    unsigned mine = lane < SCORE_WARPS ? warp_tot[lane] : 0u;
    unsigned pre = mine;
#pragma unroll
    for (int o = 1; o < SCORE_WARPS; o <<= 1) {
        unsigned t = __shfl_up_sync(0xffffffffu, pre, o);
        if (lane >= o) pre += t;
    }
    total = __shfl_sync(0xffffffffu, pre, SCORE_WARPS - 1);
    const unsigned base = w == 0 ? 0u : __shfl_sync(0xffffffffu, pre, w - 1);
    return base + inc - v;
}

struct SelShared {
    uint32_t lo, hi;
    unsigned need, cnt, ncand;
};

// Selection for one sequence by the whole CTA, from the fp32 scores in global memory.
__device__ __forceinline__ void select_sequence(const SelParams& p, int seq, int n_blocks, uint32_t* keys, unsigned* hist,
                                                unsigned* warp_tot, uint32_t* red_lo, uint32_t* red_hi,
                                                uint32_t* cand_key, int* cand_idx, SelShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // ---------------- phase 2: selection
    const int m_lo = min(p.n_sink, n_blocks);
    const int m_hi = max(n_blocks - p.n_local, m_lo);
    const int n_mid = m_hi - m_lo;
    const int k_mid = p.K - p.n_sink - p.n_local;
    const unsigned k = static_cast<unsigned>(min(k_mid, n_mid));

    uint32_t kmin = 0xffffffffu, kmax = 0u;
    const float* sc = p.scores + static_cast<size_t>(seq) * p.max_blocks;
    for (int i = tid; i < BINS + BINS / 32 + 1; i += SCORE_THREADS) hist[i] = 0;   // overlaps the key loads below
    for (int i = tid; i < n_blocks; i += SCORE_THREADS) {
        uint32_t key = float_key(__ldcg(sc + i));
        keys[padded(i)] = key;
        if (i >= m_lo && i < m_hi) { kmin = min(kmin, key); kmax = max(kmax, key); }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane == 0) { red_lo[warp] = kmin; red_hi[warp] = kmax; }
    __syncthreads();
    {
        uint32_t a = red_lo[0], b = red_hi[0];
#pragma unroll
        for (int i = 1; i < SCORE_WARPS; ++i) { a = min(a, red_lo[i]); b = max(b, red_hi[i]); }
        kmin = a; kmax = b;
    }

    // Narrow [lo, hi] until keys > hi are all winners and the first `need` keys (by index)
    // inside [lo, hi] complete the set.
    uint32_t lo = kmin, hi = kmax;
    unsigned need = k;
    if (k > 0 && k < static_cast<unsigned>(n_mid)) {
        for (int pass = 0; pass < 4; ++pass) {
            const uint32_t range = hi - lo;
            if (range == 0) break;                   // every key left is equal: ties by index
            const int bits = 32 - __clz(range);
            const int shift = bits > 11 ? bits - 11 : 0;
            if (pass > 0) {                          // the first pass finds the histogram already cleared
                for (int i = tid; i < BINS + BINS / 32 + 1; i += SCORE_THREADS) hist[i] = 0;
                __syncthreads();
            }
            for (int i = m_lo + tid; i < m_hi; i += SCORE_THREADS) {
                const uint32_t key = keys[padded(i)];
                if (key >= lo && key <= hi) atomicAdd(&hist[padded((key - lo) >> shift)], 1u);
            }
            __syncthreads();
            // suffix sums from the top bin: thread t owns bins [top - BPT + 1, top], top = BINS-1 - t*BPT
            const int top = BINS - 1 - tid * BINS_PER_THREAD;
            unsigned hb[BINS_PER_THREAD], local = 0;
#pragma unroll
            for (int j = 0; j < BINS_PER_THREAD; ++j) { hb[j] = hist[padded(top - j)]; local += hb[j]; }
            unsigned total;
            const unsigned above = block_excl_scan(local, warp_tot, total);  // keys in bins above mine
            if (above < need && need <= above + local) {
                unsigned acc = above;
#pragma unroll
                for (int j = 0; j < BINS_PER_THREAD; ++j) {
                    if (need > acc && need <= acc + hb[j]) {
                        const uint32_t nlo = lo + (static_cast<uint32_t>(top - j) << shift);
                        const uint32_t span = shift ? ((1u << shift) - 1u) : 0u;
                        sh.lo = nlo;
                        sh.hi = (hi - nlo < span) ? hi : nlo + span;
                        sh.need = need - acc;
                        sh.cnt = hb[j];
                    }
                    acc += hb[j];
                }
                sh.ncand = 0;
            }
            __syncthreads();
            lo = sh.lo; hi = sh.hi; need = sh.need;
            const unsigned cnt = sh.cnt;
            if (shift == 0 || cnt == need) break;
            if (cnt <= RESOLVE_MAX) {
                // few keys left in the bucket: one warp ranks them by (key descending, index ascending)
                for (int i = m_lo + tid; i < m_hi; i += SCORE_THREADS) {
                    const uint32_t key = keys[padded(i)];
                    if (key >= lo && key <= hi) {
                        const unsigned pos = atomicAdd(&sh.ncand, 1u);
                        cand_key[pos] = key;
                        cand_idx[pos] = i;
                    }
                }
                __syncthreads();
                if (warp == 0) {
                    const bool have = lane < static_cast<int>(cnt);
                    const uint32_t mk = have ? cand_key[lane] : 0u;
                    const int mi = have ? cand_idx[lane] : 0x7fffffff;
                    unsigned rank = 0;
                    for (unsigned j = 0; j < cnt; ++j) {
                        const uint32_t ok = cand_key[j];
                        const int oi = cand_idx[j];
                        rank += (ok > mk || (ok == mk && oi < mi)) ? 1u : 0u;
                    }
                    // the need-th best candidate fixes the threshold key; ties at it go by index
                    const unsigned is_tau = __ballot_sync(0xffffffffu, have && rank == need - 1);
                    const uint32_t tau = __shfl_sync(0xffffffffu, mk, __ffs(is_tau) - 1);
                    const unsigned eq_taken = __popc(__ballot_sync(0xffffffffu, have && mk == tau && rank < need));
                    if (lane == 0) { sh.lo = tau; sh.hi = tau; sh.need = eq_taken; }
                }
                __syncthreads();
                lo = sh.lo; hi = sh.hi; need = sh.need;
                break;
            }
        }
    } else if (k == 0) {
        lo = 0xffffffffu; hi = 0xffffffffu; need = 0;       // nothing from the middle
    } else {
        need = static_cast<unsigned>(n_mid);                // everything: [lo, hi] already spans all keys
    }

    // ordered compaction: thread owns a run of consecutive block indices
    const int ipt = (n_blocks + SCORE_THREADS - 1) / SCORE_THREADS;
    const int i0 = tid * ipt, i1 = min(i0 + ipt, n_blocks);
    unsigned c_sure = 0, c_eq = 0;
    for (int i = i0; i < i1; ++i) {
        if (i < m_lo || i >= m_hi) { ++c_sure; continue; }
        const uint32_t key = keys[padded(i)];
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
            const uint32_t key = keys[padded(i)];
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

// Consecutive "chunks" (SCORE_CHUNK blocks of one sequence, sequence-major) are dealt out in
// equal runs to the CTAs; the grid is sized to what is resident at once (two CTAs per SM), so
// small workloads get one chunk per CTA and large ones loop.  Warps run through their run
// without CTA barriers; a barrier and a ticket follow only when the CTA leaves a sequence.
template <bool MULTI>                              // MULTI: head sets / all-head digests (the comparison strategies)
__global__ void __launch_bounds__(SCORE_THREADS, 2)
score_select_kernel(SelParams p) {
    const int vh = MULTI ? p.vh : 1, n_sum = MULTI ? p.n_sum : 1, dig_heads = MULTI ? p.dig_heads : 1;
    extern __shared__ uint32_t keys[];             // [padded(n_blocks)] in the selecting CTA
    __shared__ unsigned hist[BINS + BINS / 32 + 1];
    __shared__ unsigned warp_tot[SCORE_WARPS];
    __shared__ uint32_t red_lo[SCORE_WARPS], red_hi[SCORE_WARPS];
    __shared__ uint32_t cand_key[RESOLVE_MAX];
    __shared__ int cand_idx[RESOLVE_MAX];
    __shared__ SelShared sh;
    __shared__ int sh_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pi_grid_dependency_wait();
    pi_launch_dependents();
    const int n_chunks = (p.max_blocks + SCORE_CHUNK - 1) / SCORE_CHUNK;
    const int total = n_chunks * p.batch;
    const int f1 = min((static_cast<int>(blockIdx.x) + 1) * p.per, total);
    int f = blockIdx.x * p.per;

    while (f < f1) {
        const int seq = f / n_chunks;                          // virtual sequence
        const int fe = min(f1, (seq + 1) * n_chunks);          // this CTA's chunks of this sequence
        const int rseq = seq / vh, head0 = p.h_base + (seq - rseq * vh) * p.hv_step;
        float w[8];
        int n_blocks = 0;
        for (int c = f; c < fe; ++c) {
            const int b0 = (c - seq * n_chunks) * SCORE_CHUNK + warp * BLOCKS_PER_WARP;
            float acc[BLOCKS_PER_WARP];
#pragma unroll
            for (int i = 0; i < BLOCKS_PER_WARP; ++i) acc[i] = 0.f;
          for (int hh = 0; hh < n_sum; ++hh) {
            const int head = head0 + hh;
            // every load is issued before anything waits: digest rows up to max_blocks are
            // allocated, so they are read unguarded and masked at the store
            const uint4* dg = p.digest + (static_cast<size_t>(rseq) * p.max_blocks * dig_heads +
                                          (dig_heads > 1 ? head : 0)) * 32;            // 32 uint4 per (block, head)
            uint4 v[BLOCKS_PER_WARP];
            const unsigned long long stream_policy = pi_l2_stream_policy();
#pragma unroll
            for (int i = 0; i < BLOCKS_PER_WARP; ++i) {
                v[i] = make_uint4(0, 0, 0, 0);
                if (b0 + i < p.max_blocks) v[i] = ld_stream16(dg + static_cast<size_t>(b0 + i) * dig_heads * 32 + lane, stream_policy);
            }
            if (c == f || n_sum > 1) {
                pi_score::load_q_weights(p.q + (static_cast<size_t>(rseq) * p.Hq + static_cast<size_t>(head) * p.G) * PI_HEAD_DIM,
                                         p.G, lane, w);
            }
            if (c == f && hh == 0) {
                int ctx = p.ctx_len[rseq];
                if (ctx < 0) ctx = 0;
                n_blocks = (ctx + p.B - 1) / p.B;
                if (n_blocks > p.max_blocks) {
                    if (tid == 0 && c == seq * n_chunks) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_SELECT, rseq, n_blocks, p.max_blocks);
                    n_blocks = p.max_blocks;
                }
            }
#pragma unroll
            for (int i = 0; i < BLOCKS_PER_WARP; ++i) acc[i] += dot8(v[i], w);
          }
            float s[BLOCKS_PER_WARP];
#pragma unroll
            for (int i = 0; i < BLOCKS_PER_WARP; ++i) s[i] = acc[i];

            pi_score::reduce8(s, lane);
            const int b = b0 + (lane >> 2);
            if ((lane & 3) == 0 && b < n_blocks) p.scores[static_cast<size_t>(seq) * p.max_blocks + b] = s[0];
        }
        f = fe;

        // ---------------- ticket: the CTA that completes the sequence selects for it
        // (the CTA barrier orders every thread's score stores before thread 0's fence and ticket)
        const int first_cta = (seq * n_chunks) / p.per, last_cta = ((seq + 1) * n_chunks - 1) / p.per;
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            unsigned t = atomicAdd(&p.counters[seq], 1u);
            sh_last = (t == static_cast<unsigned>(last_cta - first_cta));
            if (sh_last) p.counters[seq] = 0;           // ready for the next launch
            __threadfence();
        }
        __syncthreads();
        if (sh_last) select_sequence(p, seq, n_blocks, keys, hist, warp_tot, red_lo, red_hi, cand_key, cand_idx, sh);
        __syncthreads();                                // shared arrays are reused by the next sequence
    }
}

}  // namespace

static int launch_score_select(SelParams& p, int batch, int n_sms, cudaStream_t stream);

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
    p.vh = 1; p.n_sum = 1; p.h_base = h_star; p.hv_step = 0; p.dig_heads = 1;
    return launch_score_select(p, batch, c->n_sms, stream);
}

// The comparison strategies of the paper's selection study: averaged scores shared by all heads,
// or one selection per KV head.  Same kernel over digests of every KV head.
int pi_launch_score_select_strategy(pi_ctx* c, int strategy, int batch, const void* q, const void* digest_all,
                                    const int32_t* ctx_len, int32_t* sel, int32_t* sel_count, float* scores,
                                    unsigned int* counters, cudaStream_t stream) {
    SelParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.digest = static_cast<const uint4*>(digest_all);
    p.ctx_len = ctx_len;
    p.sel = sel;
    p.sel_count = sel_count;
    p.scores = scores;
    p.counters = counters;
    p.st = pi_status_of(c);
    p.h_star = 0;
    p.Hq = c->cfg.n_q_heads;
    p.G = c->cfg.n_q_heads / c->cfg.n_kv_heads;
    p.B = c->cfg.block_tokens;
    p.K = c->cfg.budget_blocks;
    p.n_sink = c->cfg.n_sink_blocks;
    p.n_local = c->cfg.n_local_blocks;
    p.max_blocks = c->cfg.max_blocks;
    p.dig_heads = c->cfg.n_kv_heads;
    p.h_base = 0;
    if (strategy == PI_SELECT_AVERAGE) { p.vh = 1; p.n_sum = c->cfg.n_kv_heads; p.hv_step = 0; }
    else { p.vh = c->cfg.n_kv_heads; p.n_sum = 1; p.hv_step = 1; }
    return launch_score_select(p, batch * p.vh, c->n_sms, stream);
}

// Grid sizing shared by both entry points: as many CTAs as are resident at once (two per SM),
// each with an equal run of chunks.
static int launch_score_select(SelParams& p, int batch, int n_sms, cudaStream_t stream) {
    const int n_chunks = (p.max_blocks + SCORE_CHUNK - 1) / SCORE_CHUNK;
    const int total = n_chunks * batch;
    p.batch = batch;
    p.per = (total + 2 * n_sms - 1) / (2 * n_sms);
    const int grid = (total + p.per - 1) / p.per;
    const size_t smem = (static_cast<size_t>(p.max_blocks) + p.max_blocks / 32 + 1) * sizeof(uint32_t);
    const bool multi = p.vh > 1 || p.n_sum > 1 || p.dig_heads > 1;
    auto kern = multi ? score_select_kernel<true> : score_select_kernel<false>;
    // the kernel also holds about 9 KB of static shared memory: opt in before the two together pass 48 KB
    if (smem > 36 * 1024)
        PI_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    // a plain launch: this grid fills every SM's registers, so it must not sit resident waiting for
    // the kernel before it (it would keep the attention kernel of the other stream off the SMs)
    kern<<<grid, SCORE_THREADS, smem, stream>>>(p);
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}

// ------------------------------------------------------------------------------------------
// Allocation-free variant of the call above, for callers that must not allocate device
// memory (see the declaration in pulseinfer.h).  The scores and the per-sequence tickets,
// which the regular call keeps in memory that pi_create allocated, live in this fixed
// array instead.  Every GPU that loads the library holds one copy (2 MiB + 512 B) until the
// process exits.  The array's name is only a host-side handle: the device address comes from
// cudaGetSymbolAddress, once per device, on that device's first call.
#include <mutex>

constexpr int PI_NOALLOC_MAX_BATCH = 64;
constexpr int PI_NOALLOC_MAX_BLOCKS = 8192;
constexpr size_t PI_NOALLOC_HEAD_BYTES = 512;      // [0,256) status words, [256,512) tickets
constexpr size_t PI_NOALLOC_BYTES =
    PI_NOALLOC_HEAD_BYTES + static_cast<size_t>(PI_NOALLOC_MAX_BATCH) * PI_NOALLOC_MAX_BLOCKS * sizeof(float);
static __device__ __align__(256) unsigned char pi_noalloc_scratch[PI_NOALLOC_BYTES];

namespace {
constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mu;
unsigned char* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};
}  // namespace

extern "C" int pi_score_select_noalloc(int batch, int n_q_heads, int n_kv_heads, int block_tokens,
                                       int budget_blocks, int n_sink_blocks, int n_local_blocks,
                                       int max_blocks, int solo_head, const void* q_dev,
                                       const void* digest_dev, const int32_t* ctx_len_dev,
                                       int32_t* sel_blocks_dev, int32_t* sel_count_dev,
                                       int32_t* status_dev, void* stream) {
    if (!q_dev || !digest_dev || !ctx_len_dev || !sel_blocks_dev || !sel_count_dev) return PI_ERR_INVALID_ARG;
    if (batch < 1 || max_blocks < 1 || n_sink_blocks < 0 || n_local_blocks < 0) return PI_ERR_INVALID_ARG;
    if (batch > PI_NOALLOC_MAX_BATCH || max_blocks > PI_NOALLOC_MAX_BLOCKS) return PI_ERR_STATIC_LIMIT;
    if (n_kv_heads < 1 || n_q_heads < n_kv_heads || n_q_heads % n_kv_heads || n_q_heads / n_kv_heads > 16)
        return PI_ERR_UNSUPPORTED_DIM;
    if (block_tokens != 16 && block_tokens != 32 && block_tokens != 64) return PI_ERR_UNSUPPORTED_DIM;
    if (budget_blocks < 1 || budget_blocks > 4096 || budget_blocks < n_sink_blocks + n_local_blocks)
        return PI_ERR_INVALID_ARG;
    if (solo_head < 0 || solo_head >= n_kv_heads) return PI_ERR_INVALID_ARG;
    if (!pi_aligned16(q_dev) || !pi_aligned16(digest_dev)) return PI_ERR_BAD_ALIGN;

    // set-up, once per device, with that device current: resolve the array's device address
    int dev = -1;
    PI_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return PI_ERR_INVALID_ARG;
    unsigned char* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mu);
        if (!g_noalloc_ptr[dev]) {
            unsigned char* ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), pi_noalloc_scratch);
            if (e != cudaSuccess || !ptr) { (void)cudaGetLastError(); return PI_ERR_CUDA; }
            g_noalloc_ptr[dev] = ptr;
        }
        base = g_noalloc_ptr[dev];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the last call left: status words and tickets must start at zero
    PI_CUDA_TRY(cudaMemsetAsync(base, 0, PI_NOALLOC_HEAD_BYTES, s));
    if (status_dev) PI_CUDA_TRY(cudaMemsetAsync(status_dev, 0, 8 * sizeof(int32_t), s));

    SelParams p;
    p.q = static_cast<const __nv_bfloat16*>(q_dev);
    p.digest = static_cast<const uint4*>(digest_dev);
    p.ctx_len = ctx_len_dev;
    p.sel = sel_blocks_dev;
    p.sel_count = sel_count_dev;
    p.scores = reinterpret_cast<float*>(base + PI_NOALLOC_HEAD_BYTES);
    p.counters = reinterpret_cast<unsigned int*>(base + 256);
    p.st.flag = status_dev ? reinterpret_cast<int*>(status_dev + 7) : reinterpret_cast<int*>(base);
    p.st.mirror = status_dev ? status_dev : reinterpret_cast<int32_t*>(base + 64);
    p.h_star = solo_head;
    p.Hq = n_q_heads;
    p.G = n_q_heads / n_kv_heads;
    p.B = block_tokens;
    p.K = budget_blocks;
    p.n_sink = n_sink_blocks;
    p.n_local = n_local_blocks;
    p.max_blocks = max_blocks;
    p.vh = 1; p.n_sum = 1; p.h_base = solo_head; p.hv_step = 0; p.dig_heads = 1;
    // at most (8192 + 8192/32 + 1) keys: below the default dynamic shared-memory limit
    int n_sms = 0;
    PI_CUDA_TRY(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
    return launch_score_select(p, batch, n_sms, s);
}
