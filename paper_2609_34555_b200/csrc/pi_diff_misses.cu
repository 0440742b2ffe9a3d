// Miss diff of the selection against the device-resident block table, victim choice,
// table update and the coalesced recall list, as a call of its own: one CTA per sequence,
// everything the sequence needs (selection, slot arrays, victim keys) in shared memory.
// The per-sequence routine is shared with the kernel that also scores and selects.
#include "pi_common.cuh"
#include "pi_diff_core.cuh"

namespace {

constexpr int DIFF_THREADS = 256;

struct DiffParams {
    const int32_t* ctx_len;
    const int32_t* sel;
    const int32_t* sel_count;
    int32_t* table;
    int32_t* slot_block;
    uint32_t* slot_stamp;
    int32_t* sel_slots;
    pi_extent* list;
    int32_t* count;
    pi_status_ref st;
    unsigned long long* stats;
    uint32_t step;
    const uint32_t* step_dev;      // when set, the step is read from device memory (a captured graph replays with a new step)
    int B, K, C, Cpad, n_sink, n_local, max_blocks;
};

__global__ void __launch_bounds__(DIFF_THREADS)
diff_kernel(DiffParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ pi_select::Scratch<DIFF_THREADS / 32> sc;
    __shared__ int warp_tot[2 * (DIFF_THREADS / 32)];
    __shared__ int s_ncand;
    pi_grid_dependency_wait();
    pi_launch_dependents();
    const int seq = blockIdx.x, tid = threadIdx.x;

    pi_diff::SeqArgs a;
    a.step = p.step_dev ? *p.step_dev : p.step;
    int ctx = p.ctx_len[seq];
    if (ctx < 0) ctx = 0;
    a.n_blocks = min((ctx + p.B - 1) / p.B, p.max_blocks);
    int cnt = p.sel_count[seq];
    if (cnt < 0 || cnt > p.K) {
        if (tid == 0) pi_report(p.st, PI_ERR_CAPACITY, PI_STAGE_DIFF, seq, cnt, p.K);
        cnt = max(0, min(cnt, p.K));
    }
    a.cnt = cnt;
    a.seq = seq; a.K = p.K; a.C = p.C; a.Cpad = p.Cpad; a.n_sink = p.n_sink; a.n_local = p.n_local; a.max_blocks = p.max_blocks;
    a.table = p.table + static_cast<size_t>(seq) * p.max_blocks;
    a.slot_block = p.slot_block + static_cast<size_t>(seq) * p.C;
    a.slot_stamp = p.slot_stamp + static_cast<size_t>(seq) * p.C;
    a.sel_slots = p.sel_slots + static_cast<size_t>(seq) * p.K;
    a.list = p.list + static_cast<size_t>(seq) * p.K;
    a.count = p.count + seq;
    a.stats = p.stats; a.st = p.st;

    pi_diff::Smem m = pi_diff::carve(smem_raw + pi_diff::smem_keys_bytes(p.C, p.Cpad), p.K, p.C);
    m.keys = reinterpret_cast<uint32_t*>(smem_raw);
    m.warp_tot = warp_tot;
    m.n_cand = &s_ncand;

    const int32_t* sel = p.sel + static_cast<size_t>(seq) * p.K;
    for (int j = tid; j < cnt; j += DIFF_THREADS) m.sel[j] = sel[j];
    for (int s = tid; s < p.C; s += DIFF_THREADS) {
        m.sb[s] = a.slot_block[s];
        m.stp[s] = a.slot_stamp[s];
        m.used[s] = 0;
    }
    if (tid == 0) s_ncand = 0;
    pi_select::clear<DIFF_THREADS>(sc);
    __syncthreads();
    pi_diff::diff_sequence<DIFF_THREADS>(a, m, sc);
}

}  // namespace

int pi_launch_diff(pi_ctx* c, int batch, uint32_t step, const uint32_t* step_dev, const int32_t* ctx_len, const int32_t* sel,
                   const int32_t* sel_count, int32_t* table, int32_t* slot_block, uint32_t* slot_stamp,
                   int32_t* sel_slots, pi_extent* list, int32_t* count, cudaStream_t stream) {
    DiffParams p;
    p.ctx_len = ctx_len; p.sel = sel; p.sel_count = sel_count;
    p.table = table; p.slot_block = slot_block; p.slot_stamp = slot_stamp;
    p.sel_slots = sel_slots; p.list = list; p.count = count;
    p.st = pi_status_of(c);
    p.stats = c->stats_dev;
    p.step = step;
    p.step_dev = step_dev;
    p.B = c->cfg.block_tokens; p.K = c->cfg.budget_blocks; p.C = c->cfg.pool_slots;
    int cpad = 2;
    while (cpad < p.C) cpad <<= 1;
    p.Cpad = cpad;
    p.n_sink = c->cfg.n_sink_blocks; p.n_local = c->cfg.n_local_blocks; p.max_blocks = c->cfg.max_blocks;
    const size_t smem = pi_diff::smem_keys_bytes(p.C, p.Cpad) + pi_diff::smem_lists_bytes(p.K, p.C);
    // the kernel also holds about 9 KB of static shared memory
    auto kern = diff_kernel;
    if (smem > 36 * 1024)
        PI_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    PI_CUDA_TRY(pi_launch_pdl(kern, dim3(batch), dim3(DIFF_THREADS), smem, stream, p));
    PI_CUDA_TRY(cudaGetLastError());
    return PI_OK;
}
