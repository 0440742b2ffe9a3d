// Gather-scatter recall: the GPU pulls the missing units out of the pinned host store
// with wide loads and writes them into their pool slots.
//
// A small, fixed number of persistent CTAs (sized for the host link, not for the miss
// count) walks one flat space of 4 KB pieces covering every extent of every list.
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

struct RecallParams {
    const unsigned char* host;
    unsigned char* pool;
    const pi_extent* list;
    const int32_t* count;
    pi_status_ref st;
    long long host_stride, pool_stride, unit_bytes;
    int n_lists, lists_per_seq, cap;
};

__device__ __forceinline__ uint4 ld_host16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(RECALL_THREADS)
recall_kernel(RecallParams p) {
    extern __shared__ long long s_pref[];          // [n_lists + 1] exclusive prefix of units per list
    __shared__ long long warp_tot[RECALL_WARPS];
    __shared__ long long s_run;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // units per list = units_before + n_units of its last extent; prefix over lists
    if (tid == 0) s_run = 0;
    __syncthreads();
    for (int l0 = 0; l0 < p.n_lists; l0 += RECALL_THREADS) {
        const int l = l0 + tid;
        long long u = 0;
        if (l < p.n_lists) {
            int n = p.count[l];
            if (n < 0 || n > p.cap) {
                if (blockIdx.x == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_RECALL, l, n, p.cap);
                n = 0;
            }
            if (n > 0) {
                const pi_extent e = p.list[static_cast<size_t>(l) * p.cap + n - 1];
                u = static_cast<long long>(e.units_before) + e.n_units;
                if (u < 0) u = 0;
            }
        }
        long long inc = u;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            long long t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        long long base = s_run;
        for (int i = 0; i < warp; ++i) base += warp_tot[i];
        if (l < p.n_lists) s_pref[l] = base + inc - u;
        __syncthreads();
        if (tid == RECALL_THREADS - 1) s_run = base + inc;
        __syncthreads();
    }
    if (tid == 0) s_pref[p.n_lists] = s_run;
    __syncthreads();

    const long long pieces_per_unit = p.unit_bytes / PIECE_BYTES;
    const long long total = s_pref[p.n_lists] * pieces_per_unit;
    const long long stride = static_cast<long long>(gridDim.x) * RECALL_WARPS;
    for (long long piece = static_cast<long long>(warp) * gridDim.x + blockIdx.x; piece < total; piece += stride) {
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
        const pi_extent* ext = p.list + static_cast<size_t>(l) * p.cap;
        int elo = 0, ehi = p.count[l];
        while (ehi - elo > 1) {
            const int mid = (elo + ehi) >> 1;
            if (ext[mid].units_before <= u_in_list) elo = mid; else ehi = mid;
        }
        const pi_extent e = ext[elo];
        const int k = u_in_list - e.units_before;
        if (e.src_unit < 0 || e.dst_unit < 0 || k < 0 || k >= e.n_units) {
            if (lane == 0) pi_report(p.st, PI_ERR_INDEX_RANGE, PI_STAGE_RECALL, l, elo, e.src_unit);
            continue;
        }
        const int seq = l / p.lists_per_seq;
        const unsigned char* src = p.host + seq * p.host_stride + (static_cast<long long>(e.src_unit) + k) * p.unit_bytes + in_unit + lane * 16;
        unsigned char* dst = p.pool + seq * p.pool_stride + (static_cast<long long>(e.dst_unit) + k) * p.unit_bytes + in_unit + lane * 16;
        uint4 v[LOADS_PER_LANE];
#pragma unroll
        for (int i = 0; i < LOADS_PER_LANE; ++i) v[i] = ld_host16(src + i * 512);
#pragma unroll
        for (int i = 0; i < LOADS_PER_LANE; ++i) *reinterpret_cast<uint4*>(dst + i * 512) = v[i];
    }
}

}  // namespace

int pi_launch_recall(pi_ctx* c, int n_lists, int lists_per_seq, const void* host_kv, int64_t host_stride,
                     void* pool, int64_t pool_stride, const pi_extent* list, int32_t cap,
                     const int32_t* count, int64_t unit_bytes, cudaStream_t stream) {
    RecallParams p;
    p.host = static_cast<const unsigned char*>(host_kv);
    p.pool = static_cast<unsigned char*>(pool);
    p.list = list; p.count = count;
    p.st = pi_status_of(c);
    p.host_stride = host_stride; p.pool_stride = pool_stride; p.unit_bytes = unit_bytes;
    p.n_lists = n_lists; p.lists_per_seq = lists_per_seq; p.cap = cap;
    const size_t smem = (static_cast<size_t>(n_lists) + 1) * sizeof(long long);
    if (smem > 40 * 1024)
        PI_CUDA_TRY(cudaFuncSetAttribute(recall_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    recall_kernel<<<c->recall_ctas, RECALL_THREADS, smem, stream>>>(p);
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
