// Append of the decode step's new token: K/V rows into the pool slot of the current block
// and, through the mapped pinned pointer, into the host store; running min / max of the
// retrieval head's digest; a pool slot for a block that has just been opened.  One CTA per
// sequence; a few KB per sequence, latency-bound.
#include "pi_common.cuh"

namespace {

constexpr int APPEND_THREADS = 256;
constexpr int APPEND_WARPS = APPEND_THREADS / 32;

struct AppendParams {
    const uint4* k_new;            // [batch][Hkv][D] bf16, 16 uint4 per head row
    const uint4* v_new;
    const int32_t* ctx_len;
    unsigned char* host;
    unsigned char* pool;
    int32_t* table;
    int32_t* slot_block;
    uint32_t* slot_stamp;
    __nv_bfloat16* digest;
    pi_status_ref st;
    long long host_stride, pool_stride;
    const int32_t* page;           // paged host store (or null): block b of sequence s is arena page page[s * page_stride + b]
    long long page_stride;
    int n_pages;
    const uint32_t* step_dev;      // when set, the stamp is read from device memory (graph replay)
    uint32_t step;
    int B, Hkv, C, n_sink, n_local, max_blocks, h_star;
};

__global__ void __launch_bounds__(APPEND_THREADS)
append_kernel(AppendParams p) {
    __shared__ unsigned long long warp_min[APPEND_WARPS];
    __shared__ int s_slot;
    const int seq = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pi_grid_dependency_wait();
    pi_launch_dependents();
    const int pos = p.ctx_len[seq];
    if (pos < 0) return;
    const int b = pos / p.B, t = pos - b * p.B;
    if (b >= p.max_blocks) {
        if (tid == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_APPEND, seq, b, p.max_blocks);
        return;
    }
    int32_t* table = p.table + static_cast<size_t>(seq) * p.max_blocks;
    int32_t* slot_block = p.slot_block + static_cast<size_t>(seq) * p.C;
    uint32_t* slot_stamp = p.slot_stamp + static_cast<size_t>(seq) * p.C;
    const long long block_bytes = static_cast<long long>(p.Hkv) * 2 * p.B * PI_HEAD_DIM * 2;
    int slot = table[b];
    long long host_off = seq * p.host_stride + b * block_bytes;
    if (p.page) {
        // a block index beyond the sequence's row of the table is not followed (rows are page_stride long)
        const int pg = b < p.page_stride ? p.page[seq * p.page_stride + b] : -1;
        if (pg < 0 || pg >= p.n_pages) {
            if (tid == 0) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_APPEND, seq, b, pg);
            return;
        }
        host_off = pg * block_bytes;
    }

    if (t == 0 && slot < 0) {
        // the block just opened is part of the local window: it takes the least recently selected
        // slot whose block is neither sink nor local under the new length (free slots first)
        const int nb_new = b + 1;
        unsigned long long best = ~0ull;
        for (int s = tid; s < p.C; s += APPEND_THREADS) {
            const int ob = slot_block[s];
            const bool pinned = ob >= 0 && (ob < p.n_sink || ob >= nb_new - p.n_local);
            if (!pinned) best = min(best, (static_cast<unsigned long long>(slot_stamp[s]) << 32) | static_cast<unsigned>(s));
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
        if (lane == 0) warp_min[warp] = best;
        __syncthreads();
        if (tid == 0) {
            unsigned long long g = warp_min[0];
            for (int w = 1; w < APPEND_WARPS; ++w) g = min(g, warp_min[w]);
            int sl = -1;
            if (g != ~0ull) {
                sl = static_cast<int>(g & 0xffffffffull);
                const int old = slot_block[sl];
                if (old >= 0 && old < p.max_blocks) table[old] = -1;
                table[b] = sl;
                slot_block[sl] = b;
            }
            s_slot = sl;
        }
        __syncthreads();
        slot = s_slot;
        if (slot < 0) {
            if (tid == 0) pi_report(p.st, PI_ERR_POOL_TOO_SMALL, PI_STAGE_APPEND, seq, b, p.C);
            return;
        }
    } else if (slot < 0 || slot >= p.C) {
        if (tid == 0) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_APPEND, seq, b, slot);
        return;
    }
    unsigned char* pool_blk = p.pool + seq * p.pool_stride + slot * block_bytes;
    unsigned char* host_blk = p.host + host_off;
    if (t == 0) {
        // a fresh block starts zeroed, in the pool and in the host store
        const uint4 z = make_uint4(0, 0, 0, 0);
        for (long long i = tid; i < block_bytes / 16; i += APPEND_THREADS) {
            reinterpret_cast<uint4*>(pool_blk)[i] = z;
            reinterpret_cast<uint4*>(host_blk)[i] = z;
        }
        __syncthreads();                                   // zeros land before the rows below
    }
    if (tid == 0) slot_stamp[slot] = p.step_dev ? *p.step_dev : p.step;
    // rows: [Hkv][2][B][D]; one head row is 256 B = 16 uint4
    for (int i = tid; i < p.Hkv * 32; i += APPEND_THREADS) {
        const int h = i >> 5, kv = (i >> 4) & 1, c = i & 15;
        const uint4 x = (kv ? p.v_new : p.k_new)[(static_cast<size_t>(seq) * p.Hkv + h) * 16 + c];
        const long long off = ((static_cast<long long>(h) * 2 + kv) * p.B + t) * (PI_HEAD_DIM * 2) + c * 16;
        *reinterpret_cast<uint4*>(pool_blk + off) = x;
        *reinterpret_cast<uint4*>(host_blk + off) = x;
    }
    // running min / max of the retrieval head's keys in this block (exact: bf16 values only)
    if (tid < PI_HEAD_DIM) {
        const __nv_bfloat16 x = reinterpret_cast<const __nv_bfloat16*>(p.k_new)[(static_cast<size_t>(seq) * p.Hkv + p.h_star) * PI_HEAD_DIM + tid];
        __nv_bfloat16* lo = p.digest + (static_cast<size_t>(seq) * p.max_blocks + b) * 2 * PI_HEAD_DIM + tid;
        __nv_bfloat16* hi = lo + PI_HEAD_DIM;
        if (t == 0) { *lo = x; *hi = x; }
        else {
            if (__bfloat162float(x) < __bfloat162float(*lo)) *lo = x;
            if (__bfloat162float(x) > __bfloat162float(*hi)) *hi = x;
        }
    }
}

}  // namespace

int pi_launch_append(pi_ctx* c, int h_star, int batch, uint32_t step, const void* k_new, const void* v_new,
                     const int32_t* ctx_len, void* host_kv, int64_t host_stride, void* pool, int32_t* table,
                     int32_t* slot_block, uint32_t* slot_stamp, void* digest, const int32_t* page_table,
                     int64_t page_stride, int32_t n_pages, const uint32_t* step_dev, cudaStream_t stream) {
    AppendParams p;
    p.step_dev = step_dev;
    p.page = page_table; p.page_stride = page_stride; p.n_pages = n_pages;
    p.k_new = static_cast<const uint4*>(k_new);
    p.v_new = static_cast<const uint4*>(v_new);
    p.ctx_len = ctx_len;
    p.host = static_cast<unsigned char*>(host_kv);
    p.pool = static_cast<unsigned char*>(pool);
    p.table = table; p.slot_block = slot_block; p.slot_stamp = slot_stamp;
    p.digest = static_cast<__nv_bfloat16*>(digest);
    p.st = pi_status_of(c);
    p.host_stride = host_stride;
    p.pool_stride = static_cast<long long>(c->cfg.pool_slots) * c->cfg.n_kv_heads * 2 * c->cfg.block_tokens * PI_HEAD_DIM * 2;
    p.step = step;
    p.B = c->cfg.block_tokens; p.Hkv = c->cfg.n_kv_heads; p.C = c->cfg.pool_slots;
    p.n_sink = c->cfg.n_sink_blocks; p.n_local = c->cfg.n_local_blocks; p.max_blocks = c->cfg.max_blocks;
    p.h_star = h_star;
    PI_CUDA_TRY(pi_launch_pdl(append_kernel, dim3(batch), dim3(APPEND_THREADS), 0, stream, p));
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
