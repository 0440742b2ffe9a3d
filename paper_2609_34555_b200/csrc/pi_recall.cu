// Gather-scatter recall: the GPU pulls the missing units out of the pinned host store
// with wide loads and writes them into their pool slots.
//
// A small, fixed number of persistent CTAs (sized for the host link, not for the miss
// count: requests beyond what the link can absorb only queue up in the memory system and
// slow the HBM traffic of kernels running beside this one) walks one flat space of 4 KB
// pieces covering every extent of every list.
// Lists and counts are read from device memory, so the kernel can be enqueued right
// behind the diff kernel without a host round trip.  Neighbouring warps take
// neighbouring pieces, so an extent of merged units is read as one long sequential
// burst of 512-byte warp requests with many requests in flight per warp.
#include "pi_common.cuh"

namespace {

constexpr int RECALL_THREADS = 256;
constexpr int RECALL_WARPS = RECALL_THREADS / 32;
constexpr int PIECE_BYTES = 4096;                 // per warp per iteration: 8 x 16 B per lane
constexpr int LOADS_PER_LANE = PIECE_BYTES / (32 * 16);
// Extents cached in shared memory.  Kept to 12 KB on purpose: the attention kernel that runs
// beside this one leaves about 20 KB of an SM's shared memory free, and a recall CTA that
// does not fit next to an attention CTA costs the attention kernel a whole extra wave.
constexpr int RECALL_CACHE_EXTENTS = 768;

struct RecallParams {
    const unsigned char* host;
    unsigned char* pool;
    const pi_extent* list;
    const int32_t* count;
    pi_status_ref st;
    long long host_stride, pool_stride, unit_bytes;
    long long unit_stride, list_offset;            // distance between consecutive units; byte offset of list (l % lists_per_seq)
    int n_lists, lists_per_seq, cap, cache_cap;
    long long pool_units, host_units;              // units one sequence's pool region / host region holds
    // paged host store: unit u of sequence s is page page[s * page_stride + u] of the arena at `host`
    const int32_t* page;
    long long page_stride;
    int n_pages;
};

__device__ __forceinline__ uint4 ld_host16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Block-wide exclusive scan of one value per thread over RECALL_THREADS threads, continued
// from `run` (updated to the new running total).  All threads must call.
__device__ __forceinline__ long long block_scan_add(long long v, long long* warp_tot, long long& run) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    long long base = run, tot = 0;
#pragma unroll
    for (int i = 0; i < RECALL_WARPS; ++i) {
        if (i < warp) base += warp_tot[i];
        tot += warp_tot[i];
    }
    run += tot;
    return base + inc - v;
}

template <bool PAGED>
__global__ void __launch_bounds__(RECALL_THREADS)
recall_kernel(RecallParams p) {
    extern __shared__ long long s_dyn[];
    long long* s_pref = s_dyn;                                  // [n_lists + 1] units before each list
    int* s_eoff = reinterpret_cast<int*>(s_pref + p.n_lists + 1);      // [n_lists + 1] extents before each list
    pi_extent* s_ext = reinterpret_cast<pi_extent*>(s_pref + p.n_lists + 1 + (p.n_lists + 2) / 2);   // [cache_cap]
    __shared__ long long warp_tot[RECALL_WARPS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pi_grid_dependency_wait();
    pi_launch_dependents();

    // 1. extents before each list (counts are validated once, here)
    long long run = 0;
    for (int l0 = 0; l0 < p.n_lists; l0 += RECALL_THREADS) {
        const int l = l0 + tid;
        int n = 0;
        if (l < p.n_lists) {
            n = p.count[l];
            if (n < 0 || n > p.cap) {
                if (blockIdx.x == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_RECALL, l, n, p.cap);
                n = 0;
            }
        }
        const long long off = block_scan_add(n, warp_tot, run);
        if (l < p.n_lists) s_eoff[l] = static_cast<int>(off);
    }
    if (tid == 0) s_eoff[p.n_lists] = static_cast<int>(run);
    __syncthreads();
    const int n_ext = s_eoff[p.n_lists];
    const bool cached = n_ext <= p.cache_cap;

    // 2. all extents into shared memory in one round of loads (when they fit), so that finding
    //    a piece's extent later costs no global round trip
    if (cached) {
        for (int i = tid; i < n_ext; i += RECALL_THREADS) {
            int lo = 0, hi = p.n_lists;                          // last l with s_eoff[l] <= i
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (s_eoff[mid] <= i) lo = mid; else hi = mid;
            }
            s_ext[i] = p.list[static_cast<size_t>(lo) * p.cap + (i - s_eoff[lo])];
        }
        __syncthreads();
    }

    // 3. units before each list: a list's total is units_before + n_units of its last extent
    run = 0;
    for (int l0 = 0; l0 < p.n_lists; l0 += RECALL_THREADS) {
        const int l = l0 + tid;
        long long u = 0;
        if (l < p.n_lists) {
            const int n = s_eoff[l + 1] - s_eoff[l];
            if (n > 0) {
                const pi_extent e = cached ? s_ext[s_eoff[l + 1] - 1] : p.list[static_cast<size_t>(l) * p.cap + n - 1];
                u = static_cast<long long>(e.units_before) + e.n_units;
                if (u < 0) u = 0;
                // a list cannot move more units than its sequence's pool region holds: a larger total is a
                // damaged list, and walking it would keep the kernel busy for nothing
                if (u > p.pool_units) {
                    if (blockIdx.x == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_RECALL, l, static_cast<int>(min(u, 0x7fffffffLL)), static_cast<int>(min(p.pool_units, 0x7fffffffLL)));
                    u = 0;
                }
            }
        }
        const long long off = block_scan_add(u, warp_tot, run);
        if (l < p.n_lists) s_pref[l] = off;
    }
    if (tid == 0) s_pref[p.n_lists] = run;
    __syncthreads();

    const long long pieces_per_unit = p.unit_bytes / PIECE_BYTES;
    const long long total = s_pref[p.n_lists] * pieces_per_unit;
    const long long stride = static_cast<long long>(gridDim.x) * RECALL_WARPS;

    // piece -> (source, destination) of this lane's 16-byte column; src == nullptr: skip the piece
    auto resolve = [&](long long piece, const unsigned char*& src, unsigned char*& dst) {
        src = nullptr; dst = nullptr;
        if (piece >= total) return;
        const long long unit = piece / pieces_per_unit;
        const long long in_unit = (piece - unit * pieces_per_unit) * PIECE_BYTES;
        // list that holds this unit: last l with s_pref[l] <= unit
        int lo = 0, hi = p.n_lists;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_pref[mid] <= unit) lo = mid; else hi = mid;
        }
        const int l = lo;
        const int u_in_list = static_cast<int>(unit - s_pref[l]);
        // extent inside the list: last e with units_before <= u_in_list
        const pi_extent* ext = cached ? s_ext + s_eoff[l] : p.list + static_cast<size_t>(l) * p.cap;
        int elo = 0, ehi = s_eoff[l + 1] - s_eoff[l];
        while (ehi - elo > 1) {
            const int mid = (elo + ehi) >> 1;
            if (ext[mid].units_before <= u_in_list) elo = mid; else ehi = mid;
        }
        const pi_extent e = ext[elo];
        const int k = u_in_list - e.units_before;
        if (e.src_unit < 0 || e.dst_unit < 0 || k < 0 || k >= e.n_units) {
            if (lane == 0) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_RECALL, l, elo, e.src_unit);
            return;
        }
        // a unit beyond the sequence's pool region (or, block-major store, its host region) is skipped
        if (static_cast<long long>(e.dst_unit) + k >= p.pool_units) {
            if (lane == 0) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_RECALL, l, elo, e.dst_unit + k);
            return;
        }
        if (!PAGED && static_cast<long long>(e.src_unit) + k >= p.host_units) {
            if (lane == 0) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_RECALL, l, elo, e.src_unit + k);
            return;
        }
        const int seq = l / p.lists_per_seq;
        const long long loff = (l - seq * p.lists_per_seq) * p.list_offset + in_unit + lane * 16;
        if (PAGED) {
            // one table lookup per 4 KB piece; the pieces of a page stay one sequential burst
            // a unit index beyond the sequence's row of the table is not followed (rows are page_stride long)
            const long long ui = static_cast<long long>(e.src_unit) + k;
            const int pg = ui < p.page_stride ? p.page[seq * p.page_stride + ui] : -1;
            if (pg < 0 || pg >= p.n_pages) {
                if (lane == 0) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_RECALL, l, e.src_unit + k, pg);
                return;
            }
            src = p.host + static_cast<long long>(pg) * p.unit_stride + loff;
        } else {
            src = p.host + seq * p.host_stride + (static_cast<long long>(e.src_unit) + k) * p.unit_stride + loff;
        }
        dst = p.pool + seq * p.pool_stride + (static_cast<long long>(e.dst_unit) + k) * p.unit_stride + loff;
    };

    // the next piece is resolved (searches, page lookup) while this piece's host loads are in flight
    long long piece = static_cast<long long>(warp) * gridDim.x + blockIdx.x;
    const unsigned char* src;
    unsigned char* dst;
    resolve(piece, src, dst);
    while (piece < total) {
        uint4 v[LOADS_PER_LANE];
        if (src) {
#pragma unroll
            for (int i = 0; i < LOADS_PER_LANE; ++i) v[i] = ld_host16(src + i * 512);
        }
        const unsigned char* nsrc;
        unsigned char* ndst;
        piece += stride;
        resolve(piece, nsrc, ndst);
        if (src) {
#pragma unroll
            for (int i = 0; i < LOADS_PER_LANE; ++i) *reinterpret_cast<uint4*>(dst + i * 512) = v[i];
        }
        src = nsrc; dst = ndst;
    }
}

}  // namespace

int pi_launch_recall(pi_ctx* c, int n_lists, int lists_per_seq, const void* host_kv, int64_t host_stride,
                     void* pool, int64_t pool_stride, const pi_extent* list, int32_t cap,
                     const int32_t* count, int64_t unit_bytes, int64_t unit_stride, int64_t list_offset,
                     const int32_t* page_table, int64_t page_stride, int32_t n_pages, cudaStream_t stream) {
    RecallParams p;
    p.page = page_table; p.page_stride = page_stride; p.n_pages = n_pages;
    p.host = static_cast<const unsigned char*>(host_kv);
    p.pool = static_cast<unsigned char*>(pool);
    p.list = list; p.count = count;
    p.st = pi_status_of(c);
    p.host_stride = host_stride; p.pool_stride = pool_stride; p.unit_bytes = unit_bytes;
    p.unit_stride = unit_stride > 0 ? unit_stride : unit_bytes;
    p.list_offset = list_offset;
    p.n_lists = n_lists; p.lists_per_seq = lists_per_seq; p.cap = cap;
    // capacities of one sequence's regions in units (pool: C blocks, host: NB blocks of block_bytes)
    const long long block_bytes = static_cast<long long>(c->cfg.n_kv_heads) * c->cfg.block_tokens * PI_HEAD_DIM * 4;
    p.pool_units = static_cast<long long>(c->cfg.pool_slots) * block_bytes / p.unit_stride;
    p.host_units = static_cast<long long>(c->cfg.max_blocks) * block_bytes / p.unit_stride;
    // shared memory: two prefix arrays over the lists + the extent cache
    const long long want = static_cast<long long>(n_lists) * cap;
    p.cache_cap = static_cast<int>(want < RECALL_CACHE_EXTENTS ? want : RECALL_CACHE_EXTENTS);
    const size_t smem = (static_cast<size_t>(n_lists) + 1) * sizeof(long long) +
                        ((static_cast<size_t>(n_lists) + 2) / 2) * sizeof(long long) +
                        static_cast<size_t>(p.cache_cap) * sizeof(pi_extent);
    auto kernel = page_table ? recall_kernel<true> : recall_kernel<false>;
    if (smem > 40 * 1024)
        PI_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    // ask for the largest shared-memory carve-out although this kernel hardly uses any: an SM
    // keeps one L1/shared split for all resident CTAs, and the attention kernel that overlaps
    // this one needs nearly all of it -- with the default split its CTAs could not join ours
    PI_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared));
    PI_CUDA_TRY(pi_launch_pdl(kernel, dim3(c->recall_ctas), dim3(RECALL_THREADS), smem, stream, p));
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
