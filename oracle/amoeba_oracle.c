/*
 * CPU oracle for the TP a->b re-layout of an LLM instance's state (Amoeba, runtime TP transformation).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the re-layout computes.
 * It is used by the tests, by the smoke check and by the benchmark's CPU-baseline leg; the product
 * library never links, loads or calls it, and it shares no header, helper or table with the CUDA path.
 *
 * Everything is an element-by-element loop over the *logical* (unsharded) tensors.  The result of a
 * TP a->b transformation is a permutation of bytes, so the definition is exact: the expected TP=b state is
 * "shard the logical state for TP=b", and the logical state is "un-shard the TP=a state".
 *
 * Definitions followed (paper section numbers):
 *   - Head partition of the KV cache (Sec. 3.1, "Base solution"): worker W_i, i = 1..TP, keeps the headers
 *     (H/TP)(i-1)+1 ... (H/TP)(i-1)+H/TP.  The functions below keep the paper's 1-indexed workers and headers.
 *     With grouped-query attention (Sec. 2.1 footnote) H is the number of K/V heads.
 *   - Header-centric KV layout (Sec. 3.1, "Improvement 1"): storage order [Block, Header, K/V, Token]; the
 *     head dimension is innermost and every layer has its own array of blocks (the paper omits both).
 *   - Token-first KV layout (Sec. 3.1: the layout of mainstream engines, the paper's starting point): K and V each
 *     occupy one contiguous region of the layer's pool, and inside a region a token's headers are stored together:
 *     order [K/V, Block, Token, Header], head dimension innermost.
 *   - FFN partition (Sec. 3.2, Eq. 1): up_proj split column-wise, down_proj split row-wise in the paper's
 *     [in,out] algebra FFN = f(I x U) x D.  Weights are stored [out,in] row-major here, so the paper's columns
 *     of U are rows of up/gate (contiguous) and the paper's rows of D are columns of down (strided).
 *     Attention projections follow the same rule by heads: q/k/v like U, o_proj like D.
 *   - Destination block bookkeeping (Sec. 3.1: every worker sets pages aside for the KV it will receive): the
 *     paper gives no order; the reading used here is sequences in index order, logical blocks in order, each
 *     taking the next id of the ordered free list (list order, or ascending id when a mask is given).
 *
 *   - In-place migration (Sec. 3.1, "Improvement 1"; the scenario of Sec. 3.1's example, N x TP1 -> TP N, here
 *     N x TP a -> TP N*a): every worker keeps its memory.  A worker retains, for the requests of its own instance, the
 *     headers the target TP assigns to it, sends the other headers to their workers, and the room they leave is
 *     reused by reshaping blocks: an old block of Hkv/a headers becomes N new blocks of Hkv/(N*a) headers.
 *     The paper names no block numbering; the reading used here: the worker r of instance i becomes worker r*N+i of
 *     the merged instance (so that, with a = 1, W_i keeps header group i as in the paper's example), and block p of
 *     instance i becomes block p*N+i of the merged instance (on every worker: the block table stays shared).  With
 *     the header-centric layout that new block is, on the worker that retains it, exactly the retained segment of
 *     the old block: nothing of it moves.
 *
 *   - Weight padding (Sec. 3.2, "Improvement 1", Eq. 2): padding is added at every potential partition boundary
 *     so that each partition starts on an allocation-page boundary (2 MB in the paper, Table 2 counts such pages per
 *     tensor).  With P = the largest TP degree the instance may take, a tensor is P partitions; a worker of TP = t
 *     holds P/t consecutive partitions, each stored dense at a pitch rounded up to whole pages:
 *     U' = [U_1, 0, U_2, 0, ...], D' = [D_1^T, 0, D_2^T, 0, ...]^T.  A partition of a tensor split by rows is its
 *     rows; a partition of a tensor split by columns (o_proj, down_proj) is stored as its own dense
 *     [hidden, columns/P] matrix (the paper's D_i).  A fused buffer pads after each partition's [q;k;v] or [gate;up].
 *     The pad words themselves are never written here.
 *
 * Elements are opaque 16-bit words (fp16 or bf16 makes no difference to movement).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t L;      /* layers */
    int32_t hidden; /* model width */
    int32_t Hq;     /* query heads */
    int32_t Hkv;    /* key/value heads ("headers") */
    int32_t D;      /* head dim */
    int32_t I;      /* FFN intermediate width */
} oracle_model;

enum { ORACLE_OK = 0, ORACLE_INVALID_ARG = 1, ORACLE_NO_FREE_BLOCKS = 4, ORACLE_BAD_BLOCK_ID = 5 };
enum { ORACLE_HEADER_CENTRIC = 0, ORACLE_TOKEN_FIRST = 1 };

/* Element offset inside one layer of a worker's pool (NB blocks, Hs headers per worker, T tokens per block). */
static int64_t pool_offset(int order, int64_t NB, int Hs, int T, int D, int64_t blk, int hl, int c, int tok, int d) {
    if (order == ORACLE_TOKEN_FIRST) /* [K/V][Block][Token][Header][dim] */
        return ((((int64_t)c * NB + blk) * T + tok) * Hs + hl) * (int64_t)D + d;
    /* [Block][Header][K/V][Token][dim] */
    return ((((blk * Hs + hl) * 2 + c) * T + tok) * (int64_t)D) + d;
}

/* ---- Sec. 3.1: which headers worker W_i keeps (1-indexed, inclusive range) ---- */
void oracle_header_range(int H, int TP, int i, int* first, int* last) {
    *first = (H / TP) * (i - 1) + 1;
    *last = (H / TP) * (i - 1) + H / TP;
}

/* The worker that keeps a header: search the ranges, no closed form on purpose. */
int oracle_worker_of_header(int H, int TP, int header) {
    for (int i = 1; i <= TP; ++i) {
        int first, last;
        oracle_header_range(H, TP, i, &first, &last);
        if (header >= first && header <= last) return i;
    }
    return 0;
}

static int64_t blocks_of(int32_t len, int T) { return ((int64_t)len + T - 1) / T; }

/* Number of padded tokens (whole blocks) before sequence s in the logical KV array. */
static int64_t token_base(const int32_t* seq_lens, int s, int T) {
    int64_t g = 0;
    for (int j = 0; j < s; ++j) g += blocks_of(seq_lens[j], T) * T;
    return g;
}

int64_t oracle_padded_tokens(int S, const int32_t* seq_lens, int T) { return token_base(seq_lens, S, T); }

/*
 * Logical KV: KV[l][g][h][c][d]; g = padded global token (sequence s, token t -> token_base(s) + t, every
 * sequence rounded up to whole blocks, slack tokens included), h = K/V head 0..Hkv-1, c = 0 (K) / 1 (V).
 * Pool of worker r (0-indexed pointer array, worker r+1 in the paper's numbering):
 *   pool[r][l*layer_stride + pool_offset(order, ...)],  Hs = Hkv/TP headers per worker, NB blocks per layer.
 * dir = 0: logical -> pools (shard).  dir = 1: pools -> logical (reconstruct).
 */
static void kv_walk(uint16_t* KV, const oracle_model* m, int T, int TP, int NB, int order,
                    int64_t layer_stride_elems, int S, const int32_t* seq_lens, const int32_t* bt, int maxb,
                    uint16_t* const* pools, int dir) {
    const int Hs = m->Hkv / TP;
    const int64_t G = token_base(seq_lens, S, T);
#pragma omp parallel for schedule(static)
    for (int l = 0; l < m->L; ++l) {
        for (int s = 0; s < S; ++s) {
            const int64_t g0 = token_base(seq_lens, s, T);
            const int64_t ntok = blocks_of(seq_lens[s], T) * T;
            for (int64_t t = 0; t < ntok; ++t) {
                const int64_t blk = bt[(int64_t)s * maxb + t / T];
                const int tok = (int)(t % T);
                for (int header = 1; header <= m->Hkv; ++header) {
                    const int w = oracle_worker_of_header(m->Hkv, TP, header); /* 1-indexed */
                    int first, last;
                    oracle_header_range(m->Hkv, TP, w, &first, &last);
                    const int hl = header - first; /* position among the worker's own headers */
                    uint16_t* pool = pools[w - 1] + (int64_t)l * layer_stride_elems;
                    for (int c = 0; c < 2; ++c) {
                        for (int d = 0; d < m->D; ++d) {
                            const int64_t lo = ((((int64_t)l * G + g0 + t) * m->Hkv + (header - 1)) * 2 + c) * m->D + d;
                            const int64_t po = pool_offset(order, NB, Hs, T, m->D, blk, hl, c, tok, d);
                            if (dir == 0) pool[po] = KV[lo];
                            else KV[lo] = pool[po];
                        }
                    }
                }
            }
        }
    }
}

void oracle_kv_shard(const uint16_t* KV, const oracle_model* m, int T, int TP, int NB, int order,
                     int64_t layer_stride_elems, int S, const int32_t* seq_lens, const int32_t* bt, int maxb,
                     uint16_t* const* pools) {
    kv_walk((uint16_t*)KV, m, T, TP, NB, order, layer_stride_elems, S, seq_lens, bt, maxb, pools, 0);
}

void oracle_kv_reconstruct(uint16_t* KV, const oracle_model* m, int T, int TP, int NB, int order,
                           int64_t layer_stride_elems, int S, const int32_t* seq_lens, const int32_t* bt, int maxb,
                           const uint16_t* const* pools) {
    kv_walk(KV, m, T, TP, NB, order, layer_stride_elems, S, seq_lens, bt, maxb, (uint16_t* const*)pools, 1);
}

/* TP a -> b on the KV cache: un-shard the TP=a pools into the logical array, shard that for TP=b. */
int oracle_kv_transform(const oracle_model* m, int T, int S, const int32_t* seq_lens, int maxb, int a, int NB_src,
                        int src_order, int64_t src_layer_stride, const int32_t* src_bt,
                        const uint16_t* const* src_pools, int b, int NB_dst, int dst_order, int64_t dst_layer_stride,
                        const int32_t* dst_bt, uint16_t* const* dst_pools) {
    const int64_t G = token_base(seq_lens, S, T);
    const int64_t n = (int64_t)m->L * G * m->Hkv * 2 * m->D;
    uint16_t* KV = (uint16_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(uint16_t));
    if (!KV) return ORACLE_INVALID_ARG;
    oracle_kv_reconstruct(KV, m, T, a, NB_src, src_order, src_layer_stride, S, seq_lens, src_bt, maxb, src_pools);
    oracle_kv_shard(KV, m, T, b, NB_dst, dst_order, dst_layer_stride, S, seq_lens, dst_bt, maxb, dst_pools);
    free(KV);
    return ORACLE_OK;
}

/*
 * One layer's logical weights, all [out,in] row-major:
 *   q [Hq*D, hidden]  k,v [Hkv*D, hidden]  o [hidden, Hq*D]  gate,up [I, hidden]  down [hidden, I]
 * Worker r (0-indexed here) of TP holds
 *   q_r  = rows of its Hq/TP query heads        k_r, v_r = rows of its Hkv/TP K/V heads
 *   gate_r, up_r = rows r*I/TP ...               (the paper's column-wise split of U, Eq. 1)
 *   o_r  = columns of its query heads of o       down_r = columns r*I/TP ... of down   (row-wise split of D)
 * each stored dense.  Fused buffers: qkv_r = [q_r; k_r; v_r], gate_up_r = [gate_r; up_r] (row concatenation).
 * A shard set is 7 pointers {q,k,v,o,gate,up,down}; with fused_qkv the q pointer is the fused buffer and k,v are
 * ignored, with fused_gate_up the gate pointer is the fused buffer and up is ignored.
 * dir = 0: logical -> shard.  dir = 1: shard -> logical.
 */
typedef struct { uint16_t *q, *k, *v, *o, *gate, *up, *down; } oracle_weights;

static void rows_walk(uint16_t* logical, int64_t rows_total, int64_t cols, int TP, int r, uint16_t* shard, int dir) {
    const int64_t rows_r = rows_total / TP;
    for (int64_t i = 0; i < rows_r; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            const int64_t lo = (r * rows_r + i) * cols + j;
            if (dir == 0) shard[i * cols + j] = logical[lo];
            else logical[lo] = shard[i * cols + j];
        }
}

static void cols_walk(uint16_t* logical, int64_t rows, int64_t cols_total, int TP, int r, uint16_t* shard, int dir) {
    const int64_t cols_r = cols_total / TP;
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols_r; ++j) {
            const int64_t lo = i * cols_total + r * cols_r + j;
            if (dir == 0) shard[i * cols_r + j] = logical[lo];
            else logical[lo] = shard[i * cols_r + j];
        }
}

static void weights_walk(const oracle_model* m, int TP, int r, int fused_qkv, int fused_gate_up,
                         const oracle_weights* lg, const oracle_weights* sh, int dir) {
    const int64_t hid = m->hidden, qrows = (int64_t)m->Hq * m->D, kvrows = (int64_t)m->Hkv * m->D, I = m->I;
    uint16_t* q_r = sh->q;
    uint16_t* k_r = fused_qkv ? q_r + (qrows / TP) * hid : sh->k;
    uint16_t* v_r = fused_qkv ? k_r + (kvrows / TP) * hid : sh->v;
    uint16_t* gate_r = sh->gate;
    uint16_t* up_r = fused_gate_up ? gate_r + (I / TP) * hid : sh->up;
    rows_walk(lg->q, qrows, hid, TP, r, q_r, dir);
    rows_walk(lg->k, kvrows, hid, TP, r, k_r, dir);
    rows_walk(lg->v, kvrows, hid, TP, r, v_r, dir);
    rows_walk(lg->gate, I, hid, TP, r, gate_r, dir);
    rows_walk(lg->up, I, hid, TP, r, up_r, dir);
    cols_walk(lg->o, hid, qrows, TP, r, sh->o, dir);
    cols_walk(lg->down, hid, I, TP, r, sh->down, dir);
}

void oracle_weights_shard(const oracle_model* m, int TP, int r, int fused_qkv, int fused_gate_up,
                          const oracle_weights* logical, const oracle_weights* shard) {
    weights_walk(m, TP, r, fused_qkv, fused_gate_up, logical, shard, 0);
}

void oracle_weights_reconstruct(const oracle_model* m, int TP, int r, int fused_qkv, int fused_gate_up,
                                const oracle_weights* logical, const oracle_weights* shard) {
    weights_walk(m, TP, r, fused_qkv, fused_gate_up, logical, shard, 1);
}

/* TP a -> b on one layer's weights: un-shard the a shard sets into logical tensors, shard those b ways. */
int oracle_weights_transform(const oracle_model* m, int fused_qkv, int fused_gate_up, int a,
                             const oracle_weights* src /*[a]*/, int b, const oracle_weights* dst /*[b]*/) {
    const int64_t hid = m->hidden, qrows = (int64_t)m->Hq * m->D, kvrows = (int64_t)m->Hkv * m->D, I = m->I;
    oracle_weights lg;
    lg.q = (uint16_t*)malloc((size_t)(qrows * hid) * 2);
    lg.k = (uint16_t*)malloc((size_t)(kvrows * hid) * 2);
    lg.v = (uint16_t*)malloc((size_t)(kvrows * hid) * 2);
    lg.o = (uint16_t*)malloc((size_t)(qrows * hid) * 2);
    lg.gate = (uint16_t*)malloc((size_t)(I * hid) * 2);
    lg.up = (uint16_t*)malloc((size_t)(I * hid) * 2);
    lg.down = (uint16_t*)malloc((size_t)(I * hid) * 2);
    int rc = ORACLE_OK;
    if (!lg.q || !lg.k || !lg.v || !lg.o || !lg.gate || !lg.up || !lg.down) rc = ORACLE_INVALID_ARG;
    if (rc == ORACLE_OK) {
        for (int r = 0; r < a; ++r) oracle_weights_reconstruct(m, a, r, fused_qkv, fused_gate_up, &lg, &src[r]);
        for (int r = 0; r < b; ++r) oracle_weights_shard(m, b, r, fused_qkv, fused_gate_up, &lg, &dst[r]);
    }
    free(lg.q); free(lg.k); free(lg.v); free(lg.o); free(lg.gate); free(lg.up); free(lg.down);
    return rc;
}

/*
 * Destination block bookkeeping (Sec. 3.1, reserved pages for received KV; order = the reading stated above).
 *
 * in : seq_lens[S]; src_bt[S][maxb] (entries past a sequence's blocks are -1); either free_list[n] (ids in the
 *      order they are to be handed out) or free_mask[n] (n = NB_dst; non-zero = free, handed out in ascending id).
 * out: dst_bt[S][maxb] (-1 padded), pairs[N][2] = (src block, dst block) for the k-th block in (sequence, logical
 *      block) order, *num_pairs = N, *free_count_out = free blocks left, *status.
 *
 * Whole-call errors (nothing is assigned: dst_bt all -1, N = 0, free count unchanged):
 *   a negative length or a sequence longer than maxb blocks -> INVALID_ARG; more blocks than pairs_cap ->
 *   INVALID_ARG; more blocks than free blocks -> NO_FREE_BLOCKS (checked in this order).
 * Per-block errors -> BAD_BLOCK_ID: a free-list id outside [0, NB_dst), or one that an earlier block of this walk
 *   has already taken (a list that names an id twice: two blocks must never share a destination), gives dst_bt
 *   entry -1 and pair (-1,-1);
 *   a source id outside [0, NB_src) keeps the dst_bt entry but gives pair (-1,-1), so nothing is copied for it.
 * status is sticky: it is only written while it still holds 0.
 */
void oracle_assign_blocks(int S, const int32_t* seq_lens, int T, const int32_t* src_bt, int maxb, int NB_src,
                          const int32_t* free_list, const uint8_t* free_mask, int n, int NB_dst, int32_t* dst_bt,
                          int32_t* pairs, int pairs_cap, int32_t* num_pairs, int32_t* free_count_out,
                          int32_t* status) {
    int32_t* ordered = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    int64_t n_free = 0;
    if (free_list) {
        for (int i = 0; i < n; ++i) ordered[n_free++] = free_list[i];
    } else {
        for (int id = 0; id < n; ++id)
            if (free_mask[id]) ordered[n_free++] = id;
    }
    for (int64_t i = 0; i < (int64_t)S * maxb; ++i) dst_bt[i] = -1;
    *num_pairs = 0;
    *free_count_out = (int32_t)n_free;

    int err = ORACLE_OK;
    int64_t total = 0;
    for (int s = 0; s < S; ++s) {
        if (seq_lens[s] < 0 || blocks_of(seq_lens[s], T) > maxb) err = ORACLE_INVALID_ARG;
        else total += blocks_of(seq_lens[s], T);
    }
    if (err == ORACLE_OK && total > pairs_cap) err = ORACLE_INVALID_ARG;
    if (err == ORACLE_OK && total > n_free) err = ORACLE_NO_FREE_BLOCKS;
    if (err != ORACLE_OK) {
        if (*status == 0) *status = err;
        free(ordered);
        return;
    }

    uint8_t* taken = (uint8_t*)calloc((size_t)(NB_dst > 0 ? NB_dst : 1), 1);
    int64_t k = 0;
    for (int s = 0; s < S; ++s) {
        for (int64_t i = 0; i < blocks_of(seq_lens[s], T); ++i) {
            const int32_t src = src_bt[(int64_t)s * maxb + i];
            const int32_t dst = ordered[k];
            int dst_ok = dst >= 0 && dst < NB_dst;
            if (dst_ok && taken[dst]) dst_ok = 0;
            if (dst_ok) taken[dst] = 1;
            const int src_ok = src >= 0 && src < NB_src;
            dst_bt[(int64_t)s * maxb + i] = dst_ok ? dst : -1;
            pairs[2 * k + 0] = (dst_ok && src_ok) ? src : -1;
            pairs[2 * k + 1] = (dst_ok && src_ok) ? dst : -1;
            if (!(dst_ok && src_ok) && *status == 0) *status = ORACLE_BAD_BLOCK_ID;
            ++k;
        }
    }
    *num_pairs = (int32_t)k;
    *free_count_out = (int32_t)(n_free - k);
    free(taken);
    free(ordered);
}

/*
 * Copy the blocks named in a pair list, for every layer and every header: the same expected result as
 * oracle_kv_transform when the pair list comes from oracle_assign_blocks, but usable when a pair is (-1,-1)
 * (skipped) or a block id is out of range (skipped, BAD_BLOCK_ID).  Element loops through the logical
 * coordinates (header -> source worker / destination worker), no run copies.
 */
void oracle_kv_copy_pairs(const oracle_model* m, int T, int a, int NB_src, int src_order, int64_t src_layer_stride,
                          const uint16_t* const* src_pools, int b, int NB_dst, int dst_order,
                          int64_t dst_layer_stride, uint16_t* const* dst_pools, const int32_t* pairs, int num_pairs,
                          int32_t* status) {
    const int Ha = m->Hkv / a, Hb = m->Hkv / b;
    for (int k = 0; k < num_pairs; ++k) {
        const int64_t p = pairs[2 * k], q = pairs[2 * k + 1];
        if (p < 0 || q < 0) continue;
        if (p >= NB_src || q >= NB_dst) {
            if (*status == 0) *status = ORACLE_BAD_BLOCK_ID;
            continue;
        }
        for (int l = 0; l < m->L; ++l)
            for (int header = 1; header <= m->Hkv; ++header) {
                const int wa = oracle_worker_of_header(m->Hkv, a, header);
                const int wb = oracle_worker_of_header(m->Hkv, b, header);
                int fa, fb, last;
                oracle_header_range(m->Hkv, a, wa, &fa, &last);
                oracle_header_range(m->Hkv, b, wb, &fb, &last);
                const uint16_t* sp = src_pools[wa - 1] + (int64_t)l * src_layer_stride;
                uint16_t* dp = dst_pools[wb - 1] + (int64_t)l * dst_layer_stride;
                for (int c = 0; c < 2; ++c)
                    for (int tok = 0; tok < T; ++tok)
                        for (int d = 0; d < m->D; ++d)
                            dp[pool_offset(dst_order, NB_dst, Hb, T, m->D, q, header - fb, c, tok, d)] =
                                sp[pool_offset(src_order, NB_src, Ha, T, m->D, p, header - fa, c, tok, d)];
            }
    }
}


/*
 * In-place merge of N instances of TP = a into one instance of TP = N*a (Sec. 3.1, Improvement 1).
 *
 * in : seq_lens[N][S], bt[N][S][maxb] (each instance's own block table over its own pool of NB blocks; -1 padded;
 *      an instance with fewer than S sequences pads with length 0);
 *      pools[i*a + r] = pool of worker r (0-indexed) of instance i, header-centric, [L][NB][Hkv/a][K/V][T][D],
 *      layer_stride elements between layers.
 * out: the same pools, now read as pools of the merged instance: pools[i*a + r] is worker r*N+i (0-indexed) with
 *      [L][NB*N][Hkv/(N*a)][K/V][T][D]; new_bt[N][S][maxb] = the merged instance's block table rows of the N
 *      request sets (entry p -> p*N+i); live[N][NB] = 1 for every old block named by instance i's table.
 *
 * Every word is read from a snapshot of the old pools and written to its new place, element by element through
 * the logical coordinates (instance, block, token, header, K/V, dim); words whose new place equals their old place
 * are written with the value they already have.  Words of blocks no table names are never touched.
 *
 * Errors.  Whole call (nothing moves, new_bt all -1, live all 0): a negative length or a sequence longer than maxb
 * blocks -> INVALID_ARG.  Per block -> BAD_BLOCK_ID: an id outside [0, NB) or -1 inside a sequence gives new_bt
 * entry -1 and the block does not move; an id named twice by one instance moves once, both entries get p*N+i.
 * status is sticky.
 */
void oracle_kv_merge_inplace(const oracle_model* m, int T, int N, int a, int NB, int64_t layer_stride, int S,
                             const int32_t* seq_lens, int maxb, const int32_t* bt, uint16_t* const* pools,
                             int32_t* new_bt, uint8_t* live, int32_t* status) {
    const int TPn = N * a;               /* target TP */
    const int Ha = m->Hkv / a;           /* headers per worker before */
    const int Hn = m->Hkv / TPn;         /* headers per worker after */
    const int64_t pool_elems = (int64_t)m->L * layer_stride;
    for (int64_t k = 0; k < (int64_t)N * S * maxb; ++k) new_bt[k] = -1;
    for (int64_t k = 0; k < (int64_t)N * NB; ++k) live[k] = 0;
    for (int64_t k = 0; k < (int64_t)N * S; ++k)
        if (seq_lens[k] < 0 || blocks_of(seq_lens[k], T) > maxb) {
            if (*status == 0) *status = ORACLE_INVALID_ARG;
            return;
        }
    /* snapshot of every pool before anything moves */
    uint16_t** old = (uint16_t**)malloc(sizeof(uint16_t*) * (size_t)(N * a));
    for (int w = 0; w < N * a; ++w) {
        old[w] = (uint16_t*)malloc((size_t)pool_elems * sizeof(uint16_t));
        memcpy(old[w], pools[w], (size_t)pool_elems * sizeof(uint16_t));
    }
    for (int i = 0; i < N; ++i) {
        for (int s = 0; s < S; ++s) {
            for (int64_t j = 0; j < blocks_of(seq_lens[i * S + s], T); ++j) {
                const int64_t e = ((int64_t)i * S + s) * maxb + j;
                const int64_t p = bt[e];
                if (p < 0 || p >= NB) {
                    if (*status == 0) *status = ORACLE_BAD_BLOCK_ID;
                    continue;
                }
                new_bt[e] = (int32_t)(p * N + i);
                if (live[(int64_t)i * NB + p]) { /* named twice by this instance: already moved */
                    if (*status == 0) *status = ORACLE_BAD_BLOCK_ID;
                    continue;
                }
                live[(int64_t)i * NB + p] = 1;
                for (int l = 0; l < m->L; ++l)
                    for (int header = 1; header <= m->Hkv; ++header) {
                        /* before: worker wa of instance i (1-indexed within the instance) */
                        const int wa = oracle_worker_of_header(m->Hkv, a, header);
                        int fa, fn, last;
                        oracle_header_range(m->Hkv, a, wa, &fa, &last);
                        /* after: worker wn of the merged instance, which is worker (wn-1)/N of instance (wn-1)%N */
                        const int wn = oracle_worker_of_header(m->Hkv, TPn, header);
                        oracle_header_range(m->Hkv, TPn, wn, &fn, &last);
                        const int inst_after = (wn - 1) % N, rank_after = (wn - 1) / N;
                        const uint16_t* sp = old[i * a + (wa - 1)] + (int64_t)l * layer_stride;
                        uint16_t* dp = pools[inst_after * a + rank_after] + (int64_t)l * layer_stride;
                        for (int c = 0; c < 2; ++c)
                            for (int tok = 0; tok < T; ++tok)
                                for (int d = 0; d < m->D; ++d)
                                    dp[pool_offset(ORACLE_HEADER_CENTRIC, (int64_t)NB * N, Hn, T, m->D, p * N + i,
                                                   header - fn, c, tok, d)] =
                                        sp[pool_offset(ORACLE_HEADER_CENTRIC, NB, Ha, T, m->D, p, header - fa, c, tok, d)];
                    }
            }
        }
    }
    for (int w = 0; w < N * a; ++w) free(old[w]);
    free(old);
}


/* ---- Sec. 3.2, Improvement 1: padded partitions ---- */

/* Table 2: allocation pages one tensor of rows x cols elements of elem_bytes occupies when split TP ways. */
double oracle_pages_per_tensor(int64_t rows, int64_t cols, int elem_bytes, int TP, int64_t page_bytes) {
    return (double)rows * (double)cols * (double)elem_bytes / (double)TP / (double)page_bytes;
}

/* Elements from the start of one partition to the start of the next: the partition rounded up to whole pages. */
int64_t oracle_padded_pitch(int64_t partition_elems, int64_t page_elems) {
    return (partition_elems + page_elems - 1) / page_elems * page_elems;
}

/*
 * Worker r (0-indexed) of TP holds partitions r*P/TP ... (r+1)*P/TP - 1 of every tensor, partition j of its own at
 * element offset j*pitch of the buffer (pitch = the buffer's partition size rounded up to pages).
 * Buffers: q,k,v,gate,up: partition = its rows, [rows/P, hidden]; o, down: partition = [hidden, cols/P] dense;
 * fused_qkv: partition = [q_p; k_p; v_p] under the q pointer; fused_gate_up: [gate_p; up_p] under the gate pointer.
 * dir = 0: logical -> shard, dir = 1: shard -> logical.
 */
static void padded_rows(uint16_t* logical, int64_t rows_total, int64_t cols, int P, int p, uint16_t* part, int dir) {
    const int64_t rows_p = rows_total / P;
    for (int64_t i = 0; i < rows_p; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            const int64_t lo = (p * rows_p + i) * cols + j;
            if (dir == 0) part[i * cols + j] = logical[lo];
            else logical[lo] = part[i * cols + j];
        }
}

static void padded_cols(uint16_t* logical, int64_t rows, int64_t cols_total, int P, int p, uint16_t* part, int dir) {
    const int64_t cols_p = cols_total / P;
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols_p; ++j) {
            const int64_t lo = i * cols_total + p * cols_p + j;
            if (dir == 0) part[i * cols_p + j] = logical[lo];
            else logical[lo] = part[i * cols_p + j];
        }
}

void oracle_weights_padded_walk(const oracle_model* m, int TP, int r, int P, int64_t page_elems, int fused_qkv,
                                int fused_gate_up, const oracle_weights* lg, const oracle_weights* sh, int dir) {
    const int64_t hid = m->hidden, qrows = (int64_t)m->Hq * m->D, kvrows = (int64_t)m->Hkv * m->D, I = m->I;
    const int n = P / TP;
    const int64_t q_part = qrows / P * hid, kv_part = kvrows / P * hid, ffn_part = I / P * hid;
    const int64_t pitch_q = oracle_padded_pitch(fused_qkv ? q_part + 2 * kv_part : q_part, page_elems);
    const int64_t pitch_kv = oracle_padded_pitch(kv_part, page_elems);
    const int64_t pitch_gate = oracle_padded_pitch(fused_gate_up ? 2 * ffn_part : ffn_part, page_elems);
    const int64_t pitch_up = oracle_padded_pitch(ffn_part, page_elems);
    const int64_t pitch_o = oracle_padded_pitch(q_part, page_elems);      /* [hidden, qrows/P] */
    const int64_t pitch_down = oracle_padded_pitch(ffn_part, page_elems); /* [hidden, I/P] */
    for (int j = 0; j < n; ++j) {
        const int p = r * n + j; /* partition index among the P */
        uint16_t* q_p = sh->q + j * pitch_q;
        uint16_t* k_p = fused_qkv ? q_p + q_part : sh->k + j * pitch_kv;
        uint16_t* v_p = fused_qkv ? k_p + kv_part : sh->v + j * pitch_kv;
        uint16_t* gate_p = sh->gate + j * pitch_gate;
        uint16_t* up_p = fused_gate_up ? gate_p + ffn_part : sh->up + j * pitch_up;
        padded_rows(lg->q, qrows, hid, P, p, q_p, dir);
        padded_rows(lg->k, kvrows, hid, P, p, k_p, dir);
        padded_rows(lg->v, kvrows, hid, P, p, v_p, dir);
        padded_rows(lg->gate, I, hid, P, p, gate_p, dir);
        padded_rows(lg->up, I, hid, P, p, up_p, dir);
        padded_cols(lg->o, hid, qrows, P, p, sh->o + j * pitch_o, dir);
        padded_cols(lg->down, hid, I, P, p, sh->down + j * pitch_down, dir);
    }
}


/*
 * The way back (Sec. 3.3, scale-down: "KV first", each new instance must hold all headers of its own requests),
 * in place: one instance of TP = N*a becomes N instances of TP = a on the same workers' memory.  It undoes
 * oracle_kv_merge_inplace and uses the same reading: merged worker r*N+i becomes worker r of instance i, and a block
 * whose merged id is q = p*N+i belongs to instance i and becomes its block p (the N new-size slots p*N .. p*N+N-1 of
 * that instance's pools).  The scheduler decides which request goes to which instance; a request may go to instance
 * i only while its blocks have ids = i (mod N) - other blocks are first renumbered by an ordinary block-table
 * rewrite with a free list of such ids.
 *
 * in : seq_lens[N][S], bt[N][S][maxb]: row block i = the merged instance's table rows of the requests that go to
 *      instance i (ids over the merged pools of NB*N blocks); pools[i*a + r] = merged worker r*N+i,
 *      [L][NB*N][Hkv/(N*a)][K/V][T][D].
 * out: pools[i*a + r] = worker r of instance i, [L][NB][Hkv/a][K/V][T][D]; old_bt[N][S][maxb] (entry q -> q/N);
 *      live[N][NB] = 1 for every block of instance i that now holds a request's data.
 * Errors as in the merge; in addition an id q with q mod N != i is BAD_BLOCK_ID (entry -1, block not moved).
 */
void oracle_kv_split_inplace(const oracle_model* m, int T, int N, int a, int NB, int64_t layer_stride, int S,
                             const int32_t* seq_lens, int maxb, const int32_t* bt, uint16_t* const* pools,
                             int32_t* old_bt, uint8_t* live, int32_t* status) {
    const int TPn = N * a, Ha = m->Hkv / a, Hn = m->Hkv / TPn;
    const int64_t pool_elems = (int64_t)m->L * layer_stride;
    for (int64_t k = 0; k < (int64_t)N * S * maxb; ++k) old_bt[k] = -1;
    for (int64_t k = 0; k < (int64_t)N * NB; ++k) live[k] = 0;
    for (int64_t k = 0; k < (int64_t)N * S; ++k)
        if (seq_lens[k] < 0 || blocks_of(seq_lens[k], T) > maxb) {
            if (*status == 0) *status = ORACLE_INVALID_ARG;
            return;
        }
    uint16_t** old = (uint16_t**)malloc(sizeof(uint16_t*) * (size_t)(N * a));
    for (int w = 0; w < N * a; ++w) {
        old[w] = (uint16_t*)malloc((size_t)pool_elems * sizeof(uint16_t));
        memcpy(old[w], pools[w], (size_t)pool_elems * sizeof(uint16_t));
    }
    for (int i = 0; i < N; ++i)
        for (int s = 0; s < S; ++s)
            for (int64_t j = 0; j < blocks_of(seq_lens[i * S + s], T); ++j) {
                const int64_t e = ((int64_t)i * S + s) * maxb + j;
                const int64_t q = bt[e];
                if (q < 0 || q >= (int64_t)NB * N || q % N != i) {
                    if (*status == 0) *status = ORACLE_BAD_BLOCK_ID;
                    continue;
                }
                const int64_t p = q / N;
                old_bt[e] = (int32_t)p;
                if (live[(int64_t)i * NB + p]) {
                    if (*status == 0) *status = ORACLE_BAD_BLOCK_ID;
                    continue;
                }
                live[(int64_t)i * NB + p] = 1;
                for (int l = 0; l < m->L; ++l)
                    for (int header = 1; header <= m->Hkv; ++header) {
                        /* before: merged worker wn, which lives in the memory of worker (wn-1)/N of instance (wn-1)%N */
                        const int wn = oracle_worker_of_header(m->Hkv, TPn, header);
                        /* after: worker wa of instance i */
                        const int wa = oracle_worker_of_header(m->Hkv, a, header);
                        int fa, fn, last;
                        oracle_header_range(m->Hkv, TPn, wn, &fn, &last);
                        oracle_header_range(m->Hkv, a, wa, &fa, &last);
                        const uint16_t* sp = old[((wn - 1) % N) * a + (wn - 1) / N] + (int64_t)l * layer_stride;
                        uint16_t* dp = pools[i * a + (wa - 1)] + (int64_t)l * layer_stride;
                        for (int c = 0; c < 2; ++c)
                            for (int tok = 0; tok < T; ++tok)
                                for (int d = 0; d < m->D; ++d)
                                    dp[pool_offset(ORACLE_HEADER_CENTRIC, NB, Ha, T, m->D, p, header - fa, c, tok, d)] =
                                        sp[pool_offset(ORACLE_HEADER_CENTRIC, (int64_t)NB * N, Hn, T, m->D, q,
                                                       header - fn, c, tok, d)];
                    }
            }
    for (int w = 0; w < N * a; ++w) free(old[w]);
    free(old);
}


/*
 * In-place block reshaping of ONE instance (Sec. 3.1, "Improvement 1": a worker retains the headers the new TP degree
 * assigns to it where they are, and the room the migrated headers leave inside a block is reused by reshaping the
 * block into smaller blocks).  TP = a becomes TP = N*a (split) or TP = N*a becomes TP = a (merge back).
 *
 * Reading (the paper names no numbering): the header ranges are contiguous, so old worker r (0-indexed) of TP = a
 * holds exactly the headers of workers r*N .. r*N+N-1 of TP = N*a; it becomes worker r*N, the one whose headers are
 * the first N-th of each of its blocks.  Its pool of NB blocks of Hkv/a headers is re-read as NB*N blocks of
 * Hkv/(N*a) headers, and old block p becomes new block p*N ON EVERY WORKER (the block table stays shared): on worker
 * r*N that is the same memory, so the retained headers do not move; the headers of group k = 1..N-1 go to block p*N of
 * worker r*N+k, whose pool (same capacity, NB*N blocks) is fresh.  Afterwards every id that is not p*N for a live p is
 * free - in particular the ids p*N+1 .. p*N+N-1, which on worker r*N are the segments the migrated headers left.
 *
 * pools[w], w = 0 .. N*a-1, is the pool of worker w of the TP = N*a side; worker r of the TP = a side is pools[r*N].
 * Both views use layer_stride elements between layers.
 *
 * split (dir = 0)  in : seq_lens[S], bt[S][maxb] over NB ids.   out: new_bt (p -> p*N), free_mask[NB*N].
 * merge (dir = 1)  in : bt over NB*N ids; only ids = 0 (mod N) can be reshaped back (the caller first renumbers other
 *                       blocks with the ordinary block-table rewrite and a free list of such ids whose N-1 followers
 *                       are free).                              out: new_bt (q -> q/N), free_mask[NB].
 * Both: pairs[k] = (old id, new id) of the k-th block in (sequence, logical block) order, (-1,-1) for a block that
 * is not moved; *num_pairs; *free_count = number of set bytes of free_mask (1 = free).
 *
 * Every word is read from a snapshot of the pools taken before anything moves and written through its logical
 * coordinates (block, token, header, K/V, dim); a word whose new place is its old place is written with the value
 * it has.  Words of blocks no table names, and the segments the migrated headers leave, are never written.
 *
 * Errors.  Whole call (nothing moves; new_bt all -1, no pairs, free_mask all 1): a negative length, a sequence
 * longer than maxb blocks, or more blocks than pairs_cap -> INVALID_ARG.  Per block -> BAD_BLOCK_ID, table entry -1,
 * pair (-1,-1), block not moved: an id outside the pool, -1 inside a sequence, an id named a second time, and for the
 * merge an id that is not a multiple of N.  status is sticky.
 */
static void kv_reshape_inplace(int dir, const oracle_model* m, int T, int N, int a, int NB, int64_t layer_stride,
                               int S, const int32_t* seq_lens, int maxb, const int32_t* bt, uint16_t* const* pools,
                               int32_t* new_bt, int32_t* pairs, int pairs_cap, int32_t* num_pairs,
                               uint8_t* free_mask, int32_t* free_count, int32_t* status) {
    const int TPn = N * a, Ha = m->Hkv / a, Hn = m->Hkv / TPn;
    const int64_t NBn = (int64_t)NB * N;                 /* blocks of the TP = N*a side */
    const int64_t ids_in = dir == 0 ? NB : NBn, ids_out = dir == 0 ? NBn : NB;
    const int64_t pool_elems = (int64_t)m->L * layer_stride;
    for (int64_t k = 0; k < (int64_t)S * maxb; ++k) new_bt[k] = -1;
    for (int64_t k = 0; k < ids_out; ++k) free_mask[k] = 1;
    *num_pairs = 0;
    *free_count = (int32_t)ids_out;
    int64_t total = 0;
    int err = ORACLE_OK;
    for (int s = 0; s < S; ++s) {
        if (seq_lens[s] < 0 || blocks_of(seq_lens[s], T) > maxb) err = ORACLE_INVALID_ARG;
        else total += blocks_of(seq_lens[s], T);
    }
    if (err == ORACLE_OK && total > pairs_cap) err = ORACLE_INVALID_ARG;
    if (err != ORACLE_OK) {
        if (*status == 0) *status = err;
        return;
    }
    uint16_t** old = (uint16_t**)malloc(sizeof(uint16_t*) * (size_t)TPn);
    for (int w = 0; w < TPn; ++w) {
        old[w] = (uint16_t*)malloc((size_t)(pool_elems > 0 ? pool_elems : 1) * sizeof(uint16_t));
        memcpy(old[w], pools[w], (size_t)pool_elems * sizeof(uint16_t));
    }
    int64_t k = 0, n_live = 0;
    for (int s = 0; s < S; ++s)
        for (int64_t j = 0; j < blocks_of(seq_lens[s], T); ++j, ++k) {
            const int64_t e = (int64_t)s * maxb + j;
            const int64_t id = bt[e];
            pairs[2 * k] = pairs[2 * k + 1] = -1;
            int ok = id >= 0 && id < ids_in && (dir == 0 || id % N == 0);
            const int64_t nid = dir == 0 ? id * N : id / N;
            if (ok && !free_mask[nid]) ok = 0; /* named a second time */
            if (!ok) {
                if (*status == 0) *status = ORACLE_BAD_BLOCK_ID;
                continue;
            }
            new_bt[e] = (int32_t)nid;
            pairs[2 * k] = (int32_t)id;
            pairs[2 * k + 1] = (int32_t)nid;
            free_mask[nid] = 0;
            ++n_live;
            const int64_t blk_a = dir == 0 ? id : nid;  /* the block's id on the TP = a side */
            const int64_t blk_n = dir == 0 ? nid : id;  /* ... and on the TP = N*a side */
            for (int l = 0; l < m->L; ++l)
                for (int header = 1; header <= m->Hkv; ++header) {
                    const int wa = oracle_worker_of_header(m->Hkv, a, header);   /* 1-indexed worker at TP = a */
                    const int wn = oracle_worker_of_header(m->Hkv, TPn, header); /* ... at TP = N*a */
                    int fa, fn, last;
                    oracle_header_range(m->Hkv, a, wa, &fa, &last);
                    oracle_header_range(m->Hkv, TPn, wn, &fn, &last);
                    const int mem_a = (wa - 1) * N; /* whose memory the TP = a worker lives in */
                    const int mem_n = wn - 1;
                    const int64_t lo = (int64_t)l * layer_stride;
                    for (int c = 0; c < 2; ++c)
                        for (int tok = 0; tok < T; ++tok)
                            for (int d = 0; d < m->D; ++d) {
                                const int64_t oa = lo + pool_offset(ORACLE_HEADER_CENTRIC, NB, Ha, T, m->D, blk_a,
                                                                    header - fa, c, tok, d);
                                const int64_t on = lo + pool_offset(ORACLE_HEADER_CENTRIC, NBn, Hn, T, m->D, blk_n,
                                                                    header - fn, c, tok, d);
                                if (dir == 0) pools[mem_n][on] = old[mem_a][oa];
                                else pools[mem_a][oa] = old[mem_n][on];
                            }
                }
        }
    *num_pairs = (int32_t)k;
    *free_count = (int32_t)(ids_out - n_live);
    for (int w = 0; w < TPn; ++w) free(old[w]);
    free(old);
}

void oracle_kv_reshape_split(const oracle_model* m, int T, int N, int a, int NB, int64_t layer_stride, int S,
                             const int32_t* seq_lens, int maxb, const int32_t* bt, uint16_t* const* pools,
                             int32_t* new_bt, int32_t* pairs, int pairs_cap, int32_t* num_pairs, uint8_t* free_mask,
                             int32_t* free_count, int32_t* status) {
    kv_reshape_inplace(0, m, T, N, a, NB, layer_stride, S, seq_lens, maxb, bt, pools, new_bt, pairs, pairs_cap,
                       num_pairs, free_mask, free_count, status);
}

void oracle_kv_reshape_merge(const oracle_model* m, int T, int N, int a, int NB, int64_t layer_stride, int S,
                             const int32_t* seq_lens, int maxb, const int32_t* bt, uint16_t* const* pools,
                             int32_t* new_bt, int32_t* pairs, int pairs_cap, int32_t* num_pairs, uint8_t* free_mask,
                             int32_t* free_count, int32_t* status) {
    kv_reshape_inplace(1, m, T, N, a, NB, layer_stride, S, seq_lens, maxb, bt, pools, new_bt, pairs, pairs_cap,
                       num_pairs, free_mask, free_count, status);
}
