/*
 * CPU oracle for the per-layer decode recall path of sparse KV-cache offloading:
 * digest -> score -> select -> diff -> recall -> sparse attention.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain loops, fp64 arithmetic on the exact values of
 * the bf16 inputs, no blocking, no fusion.  It shares no code with the CUDA
 * library and must never be called from the product path.
 *
 * What the paper fixes and what it leaves open
 *   - Workflow (Sec. 2.2, "Sparse KV Cache Offloading"): (1) sparse selection gives
 *     B_topk, (2) B_recall = B_topk \ B_gpu, (3) B_recall moves from DRAM to the GPU.
 *   - SoloHead (Sec. 4.4.1): digests exist for one retrieval KV head per layer; its
 *     top-k block set is shared by all KV heads of the layer.
 *   - Budget (Sec. 5, Setup): sink + local tokens are always resident and always
 *     attended; only middle blocks compete for the top-k.
 *   - The digest formula is NOT in the paper (it only says "compact per-head
 *     digests", following Quest).  Reading used here: channel-wise min and max of
 *     the block's keys; score = sum over the group's query heads and channels of
 *     max(q*min, q*max).  parity unpinned by the paper: pinned by the hand-worked
 *     example and the upper-bound invariant in tests/.
 *   - The eviction rule is NOT in the paper.  Reading used here: least recently
 *     selected slot first, ties to the lower slot.  parity unpinned by the paper.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define PIO_OK 0
#define PIO_POOL_TOO_SMALL (-4)

static double bf16_val(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int pio_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads of the loop over sequences in pio_layer_step (timing only; no effect on results). */
void pio_set_num_threads(int n) {
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Offset (in elements) of token t of kv head h, plane kv (0 = K, 1 = V) in one block
 * stored as [Hkv][2][B][D]. */
static size_t in_block(int h, int kv, int t, int B, int D) {
    return (((size_t)h * 2 + kv) * B + t) * D;
}

/* ---- O1: block digests of the layer's retrieval head (Sec. 4.4.1; Quest-style
 * min/max reading).  kv_seq: [n_blocks][Hkv][2][B][D] bf16 bits; digest:
 * [n_blocks][2][D], row 0 = channel-wise min, row 1 = max over the valid tokens
 * t < ctx of the block.  min/max of bf16 values are bf16 values: no rounding. */
void pio_build_digest(const uint16_t* kv_seq, int ctx, int B, int Hkv, int D, int h_star,
                      uint16_t* digest) {
    int n_blocks = (ctx + B - 1) / B;
    size_t blk = (size_t)Hkv * 2 * B * D;
    for (int b = 0; b < n_blocks; ++b) {
        int valid = ctx - b * B < B ? ctx - b * B : B;
        for (int d = 0; d < D; ++d) {
            uint16_t lo = kv_seq[b * blk + in_block(h_star, 0, 0, B, D) + d], hi = lo;
            for (int t = 1; t < valid; ++t) {
                uint16_t x = kv_seq[b * blk + in_block(h_star, 0, t, B, D) + d];
                if (bf16_val(x) < bf16_val(lo)) lo = x;
                if (bf16_val(x) > bf16_val(hi)) hi = x;
            }
            digest[((size_t)b * 2 + 0) * D + d] = lo;
            digest[((size_t)b * 2 + 1) * D + d] = hi;
        }
    }
}

/* ---- O2: query-digest score of every block (Sec. 4.4.1 "query-digest scores").
 * q: [Hq][D]; only the G = Hq/Hkv query heads mapped to kv head h_star by GQA are
 * used and their per-head scores are summed (the paper averages per-KV-head
 * quantities over the group; a sum ranks identically). */
void pio_score(const uint16_t* q, const uint16_t* digest, int n_blocks, int Hq, int Hkv, int D,
               int h_star, double* score) {
    int G = Hq / Hkv;
    for (int b = 0; b < n_blocks; ++b) {
        double s = 0.0;
        for (int g = h_star * G; g < (h_star + 1) * G; ++g) {
            for (int d = 0; d < D; ++d) {
                double qv = bf16_val(q[(size_t)g * D + d]);
                double a = qv * bf16_val(digest[((size_t)b * 2 + 0) * D + d]);
                double c = qv * bf16_val(digest[((size_t)b * 2 + 1) * D + d]);
                s += a > c ? a : c;
            }
        }
        score[b] = s;
    }
}

/* ---- O3: selection (Sec. 2.2 step 1; Sec. 5 budget).  Sink blocks [0, n_sink) and
 * local blocks [n_blocks - n_local, n_blocks) are always taken; the k_mid =
 * K - n_sink - n_local best middle blocks by (score descending, index ascending)
 * join them.  Output ascending by block index, padded with -1 up to K. */
typedef struct { double s; int32_t b; } pio_cand;

static int cmp_cand(const void* x, const void* y) {
    const pio_cand* a = (const pio_cand*)x;
    const pio_cand* c = (const pio_cand*)y;
    if (a->s > c->s) return -1;
    if (a->s < c->s) return 1;
    return (a->b > c->b) - (a->b < c->b);
}

static int cmp_i32(const void* x, const void* y) {
    int32_t a = *(const int32_t*)x, c = *(const int32_t*)y;
    return (a > c) - (a < c);
}

static int is_pinned(int b, int n_blocks, int n_sink, int n_local) {
    return b < n_sink || b >= n_blocks - n_local;
}

void pio_select(const double* score, int n_blocks, int n_sink, int n_local, int K,
                int32_t* sel, int32_t* sel_count) {
    int k_mid = K - n_sink - n_local;
    if (k_mid < 0) k_mid = 0;
    pio_cand* mid = (pio_cand*)malloc(sizeof(pio_cand) * (size_t)(n_blocks > 0 ? n_blocks : 1));
    int n_mid = 0, n = 0;
    for (int b = 0; b < n_blocks; ++b) {
        if (is_pinned(b, n_blocks, n_sink, n_local)) {
            if (n < K) sel[n++] = b;
        } else {
            mid[n_mid].s = score[b];
            mid[n_mid].b = b;
            ++n_mid;
        }
    }
    qsort(mid, (size_t)n_mid, sizeof(pio_cand), cmp_cand);
    int take = n_mid < k_mid ? n_mid : k_mid;
    for (int i = 0; i < take && n < K; ++i) sel[n++] = mid[i].b;
    qsort(sel, (size_t)n, sizeof(int32_t), cmp_i32);
    *sel_count = n;
    for (int i = n; i < K; ++i) sel[i] = -1;
    free(mid);
}

/* ---- O4: miss diff against the resident set (Sec. 2.2 step 2) with the LRU victim
 * reading.  table[n_blocks] = slot or -1; slot_block[C] = block or -1;
 * slot_stamp[C] = step at which the slot's block was last selected (0 = never).
 * Outputs: sel_slots[K] (slot of every selected block after the update, -1
 * padding), miss_pairs[2*K] = (block, slot) ascending by block, n_miss.
 * Returns PIO_POOL_TOO_SMALL (tables untouched, n_miss = 0, sel_slots of the missing
 * blocks = -1) when fewer victim candidates exist than misses. */
int pio_diff(const int32_t* sel, int sel_count, int n_blocks, int C, int n_sink, int n_local,
             uint32_t step, int32_t* table, int32_t* slot_block, uint32_t* slot_stamp,
             int32_t* sel_slots, int K, int32_t* miss_pairs, int32_t* n_miss) {
    int32_t* miss = (int32_t*)malloc(sizeof(int32_t) * (size_t)(K > 0 ? K : 1));
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)(C > 0 ? C : 1));
    int m = 0, nc = 0;
    for (int j = 0; j < sel_count; ++j)
        if (table[sel[j]] < 0) miss[m++] = sel[j];
    /* candidates: slots whose block is neither selected nor pinned; free slots count */
    for (int s = 0; s < C; ++s) {
        int b = slot_block[s], in_sel = 0;
        for (int j = 0; j < sel_count; ++j) in_sel |= (sel[j] == b);
        if (b < 0 || (!in_sel && !is_pinned(b, n_blocks, n_sink, n_local))) cand[nc++] = s;
    }
    /* order candidates by (stamp ascending, slot ascending): insertion sort, stable */
    for (int i = 1; i < nc; ++i) {
        int32_t s = cand[i];
        int j = i - 1;
        while (j >= 0 && slot_stamp[cand[j]] > slot_stamp[s]) { cand[j + 1] = cand[j]; --j; }
        cand[j + 1] = s;
    }
    int rc = PIO_OK;
    if (nc < m) {
        rc = PIO_POOL_TOO_SMALL;
        *n_miss = 0;
    } else {
        for (int i = 0; i < m; ++i) {
            int32_t s = cand[i], old = slot_block[s];
            if (old >= 0) table[old] = -1;
            table[miss[i]] = s;
            slot_block[s] = miss[i];
            miss_pairs[2 * i] = miss[i];
            miss_pairs[2 * i + 1] = s;
        }
        *n_miss = m;
        for (int j = 0; j < sel_count; ++j) slot_stamp[table[sel[j]]] = step;
    }
    for (int j = 0; j < K; ++j) sel_slots[j] = j < sel_count ? table[sel[j]] : -1;
    free(miss);
    free(cand);
    return rc;
}

/* ---- O5: recall (Sec. 2.2 step 3; Sec. 4.4.2): byte copy of each missing unit from
 * the host store into its pool position.  pairs = (src_unit, dst_unit); a unit is a
 * whole block (all KV heads share the selection) or one (block, head) fragment. */
void pio_recall(const uint8_t* host_seq, uint8_t* pool_seq, const int32_t* pairs, int n,
                int64_t unit_bytes) {
    for (int i = 0; i < n; ++i)
        memcpy(pool_seq + (size_t)pairs[2 * i + 1] * unit_bytes,
               host_seq + (size_t)pairs[2 * i] * unit_bytes, (size_t)unit_bytes);
}

/* ---- O6: sparse GQA decode attention over the selected blocks (Sec. 4.2.1: the
 * offload batch "performs attention ... using the recalled KV blocks").
 * store: blocks laid out [.][Hkv][2][B][D]; entry j of the selection lives at
 * store index where[j] (a pool slot, or the block index itself when reading the
 * host copy) and is logical block blocks[j], so its token t is position
 * blocks[j]*B + t, attended only if < ctx.  out[Hq][D], lse[Hq] (natural log). */
void pio_attention(const uint16_t* q, const uint16_t* store, const int32_t* where,
                   const int32_t* blocks, int count, int ctx, int B, int Hq, int Hkv, int D,
                   double* out, double* lse) {
    int G = Hq / Hkv;
    size_t blk = (size_t)Hkv * 2 * B * D;
    double scale = 1.0 / sqrt((double)D);
    double* s = (double*)malloc(sizeof(double) * (size_t)(count > 0 ? count : 1) * B);
    for (int g = 0; g < Hq; ++g) {
        int h = g / G;
        double mx = -INFINITY;
        for (int j = 0; j < count; ++j)
            for (int t = 0; t < B; ++t) {
                double acc = -INFINITY;
                if (blocks[j] * B + t < ctx) {
                    const uint16_t* k = store + (size_t)where[j] * blk + in_block(h, 0, t, B, D);
                    acc = 0.0;
                    for (int d = 0; d < D; ++d) acc += bf16_val(q[(size_t)g * D + d]) * bf16_val(k[d]);
                    acc *= scale;
                }
                s[(size_t)j * B + t] = acc;
                if (acc > mx) mx = acc;
            }
        double den = 0.0;
        for (int d = 0; d < D; ++d) out[(size_t)g * D + d] = 0.0;
        if (mx == -INFINITY) { lse[g] = -INFINITY; continue; }
        for (int j = 0; j < count; ++j)
            for (int t = 0; t < B; ++t) {
                double a = s[(size_t)j * B + t];
                if (a == -INFINITY) continue;
                double p = exp(a - mx);
                den += p;
                const uint16_t* v = store + (size_t)where[j] * blk + in_block(h, 1, t, B, D);
                for (int d = 0; d < D; ++d) out[(size_t)g * D + d] += p * bf16_val(v[d]);
            }
        for (int d = 0; d < D; ++d) out[(size_t)g * D + d] /= den;
        lse[g] = mx + log(den);
    }
    free(s);
}

/* ---- One whole layer-step for a batch: O2..O6 in order, sequences independent
 * (the loop over sequences may run on several cores; used for timing and for
 * full-batch expected values).  All arrays are per-layer, sequence-major with the
 * strides a dense [batch][...] array has; ctx_len[batch]. */
int pio_layer_step(int batch, const int32_t* ctx_len, int max_blocks, int B, int Hq, int Hkv, int D,
                   int h_star, int K, int n_sink, int n_local, int C, uint32_t step,
                   const uint16_t* q, const uint16_t* digest, const uint8_t* host_kv,
                   int32_t* table, int32_t* slot_block, uint32_t* slot_stamp, uint8_t* pool,
                   double* score, int32_t* sel, int32_t* sel_count, int32_t* sel_slots,
                   int32_t* miss_pairs, int32_t* n_miss, double* out, double* lse) {
    int64_t block_bytes = (int64_t)Hkv * 2 * B * D * 2;
    int rc_all = PIO_OK;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int s = 0; s < batch; ++s) {
        int nb = (ctx_len[s] + B - 1) / B;
        const uint16_t* qs = q + (size_t)s * Hq * D;
        double* sc = score + (size_t)s * max_blocks;
        pio_score(qs, digest + (size_t)s * max_blocks * 2 * D, nb, Hq, Hkv, D, h_star, sc);
        pio_select(sc, nb, n_sink, n_local, K, sel + (size_t)s * K, sel_count + s);
        int rc = pio_diff(sel + (size_t)s * K, sel_count[s], nb, C, n_sink, n_local, step,
                          table + (size_t)s * max_blocks, slot_block + (size_t)s * C,
                          slot_stamp + (size_t)s * C, sel_slots + (size_t)s * K, K,
                          miss_pairs + (size_t)s * 2 * K, n_miss + s);
        if (rc != PIO_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
            rc_all = rc;
            continue;
        }
        uint8_t* pool_s = pool + (size_t)s * C * block_bytes;
        pio_recall(host_kv + (size_t)s * max_blocks * block_bytes, pool_s,
                   miss_pairs + (size_t)s * 2 * K, n_miss[s], block_bytes);
        pio_attention(qs, (const uint16_t*)pool_s, sel_slots + (size_t)s * K, sel + (size_t)s * K,
                      sel_count[s], ctx_len[s], B, Hq, Hkv, D, out + (size_t)s * Hq * D,
                      lse + (size_t)s * Hq);
    }
    return rc_all;
}

/* ---- Append of the step's new token (the step before the recall path; the paper
 * implies it -- the full KV of an offloaded request lives in CPU memory while sink, local
 * and hot middle tokens stay on the GPU, Sec. 4.2 / Sec. 5 Setup -- but never describes it:
 * parity unpinned by the paper, pinned by rebuild-from-scratch invariants in tests/).
 * The token lands at position p = ctx (length before the append), block b = p / B, row
 * t = p % B.  A new block (t == 0) belongs to the local window, so it takes a pool slot:
 * the least recently selected slot whose block is neither sink nor local under the new
 * length (ties to the lower slot, free slots first); its rows are zeroed in the pool and in
 * the host store.  The K/V rows of all heads are written to the pool slot and to the host
 * store, the slot's stamp becomes `step`, and the digest row of block b takes the new key of
 * the retrieval head into its running min / max.  Returns PIO_OK, or PIO_POOL_TOO_SMALL when
 * no slot can be evicted, or -8 when a block that must be resident is not. */
int pio_append(const uint16_t* k_new, const uint16_t* v_new, int ctx, int B, int Hkv, int D, int h_star,
               int n_sink, int n_local, int C, uint32_t step, uint16_t* host_seq, uint16_t* pool_seq,
               int32_t* table, int32_t* slot_block, uint32_t* slot_stamp, uint16_t* digest) {
    int b = ctx / B, t = ctx % B, nb_new = b + 1;
    size_t blk = (size_t)Hkv * 2 * B * D;
    int slot = table[b];
    if (t == 0) {
        if (slot < 0) {
            int best = -1;
            for (int s = 0; s < C; ++s) {
                int ob = slot_block[s];
                if (ob >= 0 && is_pinned(ob, nb_new, n_sink, n_local)) continue;
                if (best < 0 || slot_stamp[s] < slot_stamp[best]) best = s;
            }
            if (best < 0) return PIO_POOL_TOO_SMALL;
            if (slot_block[best] >= 0) table[slot_block[best]] = -1;
            slot = best;
            table[b] = slot;
            slot_block[slot] = b;
        }
        memset(pool_seq + (size_t)slot * blk, 0, blk * sizeof(uint16_t));
        memset(host_seq + (size_t)b * blk, 0, blk * sizeof(uint16_t));
    } else if (slot < 0) {
        return -8;
    }
    slot_stamp[slot] = step;
    for (int h = 0; h < Hkv; ++h)
        for (int d = 0; d < D; ++d) {
            uint16_t kx = k_new[(size_t)h * D + d], vx = v_new[(size_t)h * D + d];
            pool_seq[(size_t)slot * blk + in_block(h, 0, t, B, D) + d] = kx;
            pool_seq[(size_t)slot * blk + in_block(h, 1, t, B, D) + d] = vx;
            host_seq[(size_t)b * blk + in_block(h, 0, t, B, D) + d] = kx;
            host_seq[(size_t)b * blk + in_block(h, 1, t, B, D) + d] = vx;
        }
    for (int d = 0; d < D; ++d) {
        uint16_t x = k_new[(size_t)h_star * D + d];
        uint16_t* lo = digest + ((size_t)b * 2 + 0) * D + d;
        uint16_t* hi = digest + ((size_t)b * 2 + 1) * D + d;
        if (t == 0) { *lo = x; *hi = x; }
        else {
            if (bf16_val(x) < bf16_val(*lo)) *lo = x;
            if (bf16_val(x) > bf16_val(*hi)) *hi = x;
        }
    }
    return PIO_OK;
}

/* ---- The comparison strategies of Sec. 4.4.1 (headwise: every KV head selects for itself;
 * average: the per-head query-digest scores are combined and one top-k is shared).  They need
 * the digests of all KV heads: digest_all[n_blocks][Hkv][2][D].  The score of a set of KV heads
 * [h_lo, h_hi) is the sum of their per-head scores (a sum ranks like the paper's average):
 * headwise uses one head at a time, average uses all of them. */
void pio_build_digest_all(const uint16_t* kv_seq, int ctx, int B, int Hkv, int D, uint16_t* digest_all) {
    int n_blocks = (ctx + B - 1) / B;
    size_t blk = (size_t)Hkv * 2 * B * D;
    for (int b = 0; b < n_blocks; ++b) {
        int valid = ctx - b * B < B ? ctx - b * B : B;
        for (int h = 0; h < Hkv; ++h)
            for (int d = 0; d < D; ++d) {
                uint16_t lo = kv_seq[b * blk + in_block(h, 0, 0, B, D) + d], hi = lo;
                for (int t = 1; t < valid; ++t) {
                    uint16_t x = kv_seq[b * blk + in_block(h, 0, t, B, D) + d];
                    if (bf16_val(x) < bf16_val(lo)) lo = x;
                    if (bf16_val(x) > bf16_val(hi)) hi = x;
                }
                digest_all[(((size_t)b * Hkv + h) * 2 + 0) * D + d] = lo;
                digest_all[(((size_t)b * Hkv + h) * 2 + 1) * D + d] = hi;
            }
    }
}

void pio_score_heads(const uint16_t* q, const uint16_t* digest_all, int n_blocks, int Hq, int Hkv, int D,
                     int h_lo, int h_hi, double* score) {
    int G = Hq / Hkv;
    for (int b = 0; b < n_blocks; ++b) {
        double s = 0.0;
        for (int h = h_lo; h < h_hi; ++h)
            for (int g = h * G; g < (h + 1) * G; ++g)
                for (int d = 0; d < D; ++d) {
                    double qv = bf16_val(q[(size_t)g * D + d]);
                    double a = qv * bf16_val(digest_all[(((size_t)b * Hkv + h) * 2 + 0) * D + d]);
                    double c = qv * bf16_val(digest_all[(((size_t)b * Hkv + h) * 2 + 1) * D + d]);
                    s += a > c ? a : c;
                }
        score[b] = s;
    }
}

/* Recall of units that are `unit_bytes` long but `unit_stride` apart, starting `offset` bytes into
 * the sequence's region: the per-head form of Sec. 3.4 (one (block, head) fragment per transfer). */
void pio_recall_strided(const uint8_t* host_seq, uint8_t* pool_seq, const int32_t* pairs, int n,
                        int64_t unit_bytes, int64_t unit_stride, int64_t offset) {
    for (int i = 0; i < n; ++i)
        memcpy(pool_seq + offset + (size_t)pairs[2 * i + 1] * unit_stride,
               host_seq + offset + (size_t)pairs[2 * i] * unit_stride, (size_t)unit_bytes);
}

/* Recall from a paged host store (Sec. 4.4.2: the recalled blocks lie scattered across host
 * memory): logical block b of the sequence is page page_table[b] of an arena of unit_bytes-long
 * pages.  Everything else as in pio_recall. */
void pio_recall_paged(const uint8_t* arena, const int32_t* page_table, uint8_t* pool_seq, const int32_t* pairs,
                      int n, int64_t unit_bytes) {
    for (int i = 0; i < n; ++i)
        memcpy(pool_seq + (size_t)pairs[2 * i + 1] * unit_bytes,
               arena + (size_t)page_table[pairs[2 * i]] * unit_bytes, (size_t)unit_bytes);
}
