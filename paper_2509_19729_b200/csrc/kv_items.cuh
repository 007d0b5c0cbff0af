// Work items of the KV cache migration (Sec. 3.1): how one (block pair, layer) is cut into 2-D copies, shared by the
// KV kernels and by the kernel that moves KV and weights of a layer range in one launch.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "copy_engine.cuh"
#include "plan.hpp"

namespace amoeba {

struct KvParams {
    const char* src[AMOEBA_MAX_TP];
    char* dst[AMOEBA_MAX_TP];
    const int32_t* pairs;      // [cap][2]
    const int32_t* num_pairs;  // device scalar
    int32_t* status;
    int64_t vec_bytes, src_layer_stride, dst_layer_stride;
    int64_t row_bytes, src_row_pitch, dst_row_pitch;
    int32_t pairs_cap, layer_begin, n_layers;
    int32_t nb_src, nb_dst, block_tokens;
    int32_t src_token_major, dst_token_major;
    int32_t heads_src, heads_dst, heads_per_unit, head_units, planes;
    int32_t rows, rows_per_item, row_groups, col_chunks, chunk_bytes;
    // box items (tensor-map path)
    int32_t heads_per_run, runs_per_block, box_heads, box_tokens, box_sub_runs, box_tok_groups;
    // In-place block reshaping of one instance (0 = off): +N, the destination has N times the source's workers and
    // destination worker r*N IS source worker r; -N, the other way round.  The header unit a worker retains
    // (every N-th) is not a work item at all: `moving_units` counts the others.
    int32_t reshape, moving_units;
    int64_t src_span, dst_span;  // bytes of a source / destination pool the layers of this call reach into
};

// Tensor maps of the token-first pools, one per worker: dimensions {dim, token of the layer's K or V region,
// K/V, local header, layer}, box {head_dim, box_tokens, 2, box_heads, 1}.
struct KvMaps {
    CUtensorMap src[AMOEBA_MAX_TP];
    CUtensorMap dst[AMOEBA_MAX_TP];
};

// Byte offset, inside one layer of a worker's pool, of token 0 of (block, local header, K/V plane).
__device__ __forceinline__ int64_t pool_offset(bool token_major, int32_t nb, int32_t heads, int32_t T, int64_t vec,
                                               int32_t blk, int32_t hl, int32_t c) {
    return token_major ? ((((int64_t)c * nb + blk) * T) * heads + hl) * vec
                       : ((((int64_t)blk * heads + hl) * 2 + c) * T) * vec;
}

// Least significant digit of `rem` in a mixed-radix number; `rem` keeps the higher digits.
__device__ __forceinline__ int32_t take_digit(uint32_t& rem, int32_t radix) {
    if (radix == 1) return 0;
    const uint32_t q = rem / (uint32_t)radix;
    const int32_t d = (int32_t)(rem - q * (uint32_t)radix);
    rem = q;
    return d;
}

struct KvItems {
    const KvParams& p;
    int32_t n_pairs;
    __device__ __forceinline__ int32_t items_per_pair() const {
        return p.planes * p.moving_units * p.row_groups * p.col_chunks;
    }
    __device__ __forceinline__ int64_t count() const { return (int64_t)n_pairs * p.n_layers * items_per_pair(); }
    // n_rows == 0 marks a skipped pair.
    __device__ __forceinline__ Item operator()(int64_t w) const {
        // Two 64-bit divisions (by the items of one pair, by the pair count); everything inside a pair is 32-bit,
        // and a digit whose radix is 1 costs nothing.
        const int32_t ipp = items_per_pair();
        const int64_t lp = w / ipp;
        uint32_t rem = (uint32_t)(w - lp * ipp);
        const int32_t col = take_digit(rem, p.col_chunks);
        const int32_t rg = take_digit(rem, p.row_groups);
        int32_t hu = take_digit(rem, p.moving_units);
        const int32_t c = (int32_t)rem;  // < planes
        if (p.reshape) {  // skip every N-th unit: the m-th moving unit is unit (m / (N-1)) * N + 1 + m % (N-1)
            const int32_t n = p.reshape > 0 ? p.reshape : -p.reshape;
            const int32_t grp = hu / (n - 1);
            hu = grp * n + 1 + (hu - grp * (n - 1));
        }
        const int32_t pair = (int32_t)(lp % n_pairs);
        const int32_t layer = p.layer_begin + (int32_t)(lp / n_pairs);
        const int2 ids = __ldg(reinterpret_cast<const int2*>(p.pairs) + pair);
        Item it;
        it.src_map = it.dst_map = nullptr;
        it.src_pitch = p.src_row_pitch;
        it.dst_pitch = p.dst_row_pitch;
        it.n_rows = 0;
        it.row_bytes = 0;
        it.src = nullptr;
        it.dst = nullptr;
        if (ids.x < 0 || ids.y < 0) return it;  // the table rewrite already reported this one
        // Reshaping in place: the retained headers only stay where they are if the finer side's id is N times the other.
        const bool reshaped_ok = p.reshape == 0 || (p.reshape > 0 ? (int64_t)ids.x * p.reshape == ids.y
                                                                  : (int64_t)ids.y * -p.reshape == ids.x);
        if (ids.x >= p.nb_src || ids.y >= p.nb_dst || !reshaped_ok) {
            if (c == 0 && rg == 0 && col == 0) atomicCAS(p.status, 0, (int)AMOEBA_ERR_BAD_BLOCK_ID);
            return it;
        }
        const int32_t h0 = hu * p.heads_per_unit;  // first header of the unit
        const int32_t ra = h0 / p.heads_src, ha = h0 - ra * p.heads_src;
        const int32_t rb = h0 / p.heads_dst, hb = h0 - rb * p.heads_dst;
        const int32_t r0 = rg * p.rows_per_item;
        const int64_t in_row = (int64_t)col * p.chunk_bytes;
        it.n_rows = min(p.rows_per_item, p.rows - r0);
        it.row_bytes = p.chunk_bytes;
        it.src = p.src[ra] + layer * p.src_layer_stride +
                 pool_offset(p.src_token_major, p.nb_src, p.heads_src, p.block_tokens, p.vec_bytes, ids.x, ha, c) +
                 r0 * p.src_row_pitch + in_row;
        it.dst = p.dst[rb] + layer * p.dst_layer_stride +
                 pool_offset(p.dst_token_major, p.nb_dst, p.heads_dst, p.block_tokens, p.vec_bytes, ids.y, hb, c) +
                 r0 * p.dst_row_pitch + in_row;
#ifdef AMOEBA_CHECK_ITEMS
        if (!rows_inside(it.src - p.src[ra], it.src_pitch, it.n_rows, it.row_bytes, p.src_span) ||
            !rows_inside(it.dst - p.dst[rb], it.dst_pitch, it.n_rows, it.row_bytes, p.dst_span)) {
            atomicCAS(p.status, 0, (int)AMOEBA_ERR_INTERNAL);
            it.n_rows = 0;
        }
#endif
        return it;
    }
};

// Box items: (layer, pair, run, sub-run of headers, token group); K and V travel together.
struct KvBoxItems {
    const KvParams& p;
    const KvMaps& maps;
    int32_t n_pairs;
    __device__ __forceinline__ int32_t items_per_pair() const {
        return p.runs_per_block * p.box_sub_runs * p.box_tok_groups;
    }
    __device__ __forceinline__ int64_t count() const { return (int64_t)n_pairs * p.n_layers * items_per_pair(); }
    __device__ __forceinline__ Item operator()(int64_t w) const {
        const int32_t ipp = items_per_pair();
        const int64_t lp = w / ipp;
        uint32_t rem = (uint32_t)(w - lp * ipp);
        const int32_t tg = take_digit(rem, p.box_tok_groups);
        const int32_t sub = take_digit(rem, p.box_sub_runs);
        const int32_t run = (int32_t)rem;  // < runs_per_block
        const int32_t pair = (int32_t)(lp % n_pairs);
        const int32_t layer = p.layer_begin + (int32_t)(lp / n_pairs);
        const int2 ids = __ldg(reinterpret_cast<const int2*>(p.pairs) + pair);
        Item it;
        it.src_map = it.dst_map = nullptr;
        it.n_rows = 0;
        it.row_bytes = 0;
        it.src = nullptr;
        it.dst = nullptr;
        it.src_pitch = it.dst_pitch = (int64_t)p.block_tokens * p.vec_bytes;  // header-centric side: (header, K/V) rows
        if (ids.x < 0 || ids.y < 0) return it;
        if (ids.x >= p.nb_src || ids.y >= p.nb_dst) {
            if (run == 0 && sub == 0 && tg == 0) atomicCAS(p.status, 0, (int)AMOEBA_ERR_BAD_BLOCK_ID);
            return it;
        }
        const int32_t h0 = run * p.heads_per_run + sub * p.box_heads;
        const int32_t ra = h0 / p.heads_src, ha = h0 - ra * p.heads_src;
        const int32_t rb = h0 / p.heads_dst, hb = h0 - rb * p.heads_dst;
        const int32_t t0 = tg * p.box_tokens;
        it.n_rows = 2 * p.box_heads;
        it.row_bytes = (int32_t)(p.box_tokens * p.vec_bytes);
        it.layer = layer;
        if (p.src_token_major) {
            it.src_map = &maps.src[ra];
            it.src_tok = ids.x * p.block_tokens + t0;
            it.src_head = ha;
        } else {
            it.src = p.src[ra] + layer * p.src_layer_stride +
                     pool_offset(false, p.nb_src, p.heads_src, p.block_tokens, p.vec_bytes, ids.x, ha, 0) +
                     t0 * p.vec_bytes;
        }
        if (p.dst_token_major) {
            it.dst_map = &maps.dst[rb];
            it.dst_tok = ids.y * p.block_tokens + t0;
            it.dst_head = hb;
        } else {
            it.dst = p.dst[rb] + layer * p.dst_layer_stride +
                     pool_offset(false, p.nb_dst, p.heads_dst, p.block_tokens, p.vec_bytes, ids.y, hb, 0) +
                     t0 * p.vec_bytes;
        }
#ifdef AMOEBA_CHECK_ITEMS  // the header-centric sides; a tensor map checks its own coordinates against its extents
        if ((it.src && !rows_inside(it.src - p.src[ra], it.src_pitch, it.n_rows, it.row_bytes, p.src_span)) ||
            (it.dst && !rows_inside(it.dst - p.dst[rb], it.dst_pitch, it.n_rows, it.row_bytes, p.dst_span))) {
            atomicCAS(p.status, 0, (int)AMOEBA_ERR_INTERNAL);
            it.n_rows = 0;
        }
#endif
        return it;
    }
};

__device__ __forceinline__ int32_t clamp_pairs(const KvParams& p) {
    const int32_t n = *p.num_pairs;
    return n < 0 ? 0 : (n > p.pairs_cap ? p.pairs_cap : n);
}

// Copies the plan's geometry into the kernel parameters (pools, pair list, status, layer range and `reshape` are the
// caller's to set).
inline void kv_fill_geometry(const amoeba_plan* plan, KvParams& p) {
    const KvGeom& g = plan->kv;
    p.vec_bytes = plan->vec_bytes;
    p.row_bytes = g.row_bytes;
    p.src_row_pitch = g.src_row_pitch;
    p.dst_row_pitch = g.dst_row_pitch;
    p.block_tokens = plan->src.block_tokens;
    p.src_token_major = plan->src.kv_order == AMOEBA_KV_TOKEN_MAJOR;
    p.dst_token_major = plan->dst.kv_order == AMOEBA_KV_TOKEN_MAJOR;
    p.heads_per_unit = g.heads_per_unit;
    p.head_units = g.head_units;
    p.planes = g.planes;
    p.rows = g.rows;
    p.rows_per_item = g.rows_per_item;
    p.row_groups = g.row_groups;
    p.col_chunks = g.col_chunks;
    p.chunk_bytes = g.chunk_bytes;
    const KvBoxGeom& bx = plan->kvbox;
    p.heads_per_run = plan->heads_per_run;
    p.runs_per_block = plan->runs_per_block;
    p.box_heads = bx.heads;
    p.box_tokens = bx.tokens;
    p.box_sub_runs = bx.sub_runs;
    p.box_tok_groups = bx.tok_groups;
    p.src_layer_stride = plan->src_layer_stride;
    p.dst_layer_stride = plan->dst_layer_stride;
    p.nb_src = plan->src.num_blocks;
    p.nb_dst = plan->dst.num_blocks;
    p.heads_src = plan->heads_src;
    p.heads_dst = plan->heads_dst;
    p.src_span = (int64_t)(p.layer_begin + p.n_layers) * plan->src_layer_stride;
    p.dst_span = (int64_t)(p.layer_begin + p.n_layers) * plan->dst_layer_stride;
    p.moving_units = g.head_units;
    if (p.reshape) {  // one unit = the headers of one worker of the finer side; every N-th stays
        const int n = p.reshape > 0 ? p.reshape : -p.reshape;
        p.moving_units = g.head_units - g.head_units / n;
    }
}

// Checks the pools of an out-of-place KV call and puts them into the parameters.
inline amoeba_status kv_set_pools(const amoeba_plan* plan, const void* const* src_pools, void* const* dst_pools,
                                  KvParams& p) {
    for (int r = 0; r < plan->src.tp; ++r) {
        if (!src_pools[r]) return AMOEBA_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(src_pools[r]) % 16) return AMOEBA_ERR_ALIGNMENT;
        p.src[r] = static_cast<const char*>(src_pools[r]);
    }
    for (int r = 0; r < plan->dst.tp; ++r) {
        if (!dst_pools[r]) return AMOEBA_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(dst_pools[r]) % 16) return AMOEBA_ERR_ALIGNMENT;
        for (int q = 0; q < plan->src.tp; ++q)  // out of place: a destination pool is never a source pool
            if (dst_pools[r] == src_pools[q]) return AMOEBA_ERR_INVALID_ARG;
        p.dst[r] = static_cast<char*>(dst_pools[r]);
    }
    return AMOEBA_OK;
}

}  // namespace amoeba
