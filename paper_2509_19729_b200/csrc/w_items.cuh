// Work items of the weight re-partition (Sec. 3.2, Eq. 1): the planner's per-layer copy descriptors cut into 2-D
// copies, shared by the weight kernels and by the kernel that moves KV and weights of a layer range in one launch.
#pragma once
#include <cuda_runtime.h>

#include <vector>

#include "copy_engine.cuh"
#include "plan.hpp"

namespace amoeba {

struct WParams {
    WDescDev descs[kMaxWeightDescs];
    void* ptrs[kMaxWeightPtrs];  // [layer][src rank][tensor] then, from dst_base, [layer][dst rank][tensor]
    int32_t n_descs, items_per_layer, n_layers, src_tp, dst_tp, dst_base;
    int32_t* status;                                         // where an item outside its buffer is reported (checked build)
    int64_t src_bytes[kNumTensors], dst_bytes[kNumTensors];  // size of a worker's buffer of each kind (checked build)
};

struct WItems {
    const WParams& p;
    __device__ __forceinline__ int64_t count() const { return (int64_t)p.items_per_layer * p.n_layers; }
    __device__ __forceinline__ Item operator()(int64_t w) const {
        const int32_t layer = (int32_t)(w / p.items_per_layer);
        const int32_t rem = (int32_t)(w - (int64_t)layer * p.items_per_layer);
        int lo = 0, hi = p.n_descs - 1;  // last descriptor with item_begin <= rem
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (p.descs[mid].item_begin <= rem) lo = mid;
            else hi = mid - 1;
        }
        const WDescDev& d = p.descs[lo];
        const int32_t local = rem - d.item_begin;
        const int32_t rg = local / d.col_chunks, cc = local - rg * d.col_chunks;
        const int32_t r0 = rg * d.rows_per_item;
        const int64_t off = (int64_t)cc * d.chunk_bytes;
        Item it;
        it.src_map = it.dst_map = nullptr;
        it.n_rows = min(d.rows_per_item, d.n_rows - r0);
        it.row_bytes = (int32_t)min((int64_t)d.chunk_bytes, d.row_bytes - off);
        it.src_pitch = d.src_pitch;
        it.dst_pitch = d.dst_pitch;
        const char* s = static_cast<const char*>(p.ptrs[(layer * p.src_tp) * kNumTensors + d.src_slot]);
        char* t = static_cast<char*>(p.ptrs[p.dst_base + (layer * p.dst_tp) * kNumTensors + d.dst_slot]);
        if (!t) {  // this destination worker's buffers were not given: its shard is not produced by this call
            it.n_rows = 0;
            it.row_bytes = 0;
            it.src = nullptr;
            it.dst = nullptr;
            return it;
        }
        it.src = s + d.src_off + r0 * d.src_pitch + off;
        it.dst = t + d.dst_off + r0 * d.dst_pitch + off;
#ifdef AMOEBA_CHECK_ITEMS
        if (!rows_inside(it.src - s, it.src_pitch, it.n_rows, it.row_bytes, p.src_bytes[d.src_slot % kNumTensors]) ||
            !rows_inside(it.dst - t, it.dst_pitch, it.n_rows, it.row_bytes, p.dst_bytes[d.dst_slot % kNumTensors])) {
            atomicCAS(p.status, 0, (int)AMOEBA_ERR_INTERNAL);
            it.n_rows = 0;
        }
#endif
        return it;
    }
};

inline void* const* slots(const amoeba_layer_weights* w) { return reinterpret_cast<void* const*>(w); }

// Layers one launch can take: its pointer table holds (a + b) * kNumTensors pointers per layer.
inline int weight_layers_per_launch(int a, int b) { return std::max(1, kMaxWeightPtrs / ((a + b) * kNumTensors)); }

// Descriptors and the pointer table of layers [l0, l0 + nl) into the kernel parameters: src is [a][L], dst is [b][L]
// (worker-major host arrays of device pointers).
inline void w_fill_params(WParams& p, const std::vector<WDescDev>& descs, int32_t items_per_layer,
                          const amoeba_layer_weights* src, int a, const amoeba_layer_weights* dst, int b, int L, int l0,
                          int nl) {
    p.n_descs = (int32_t)descs.size();
    p.items_per_layer = items_per_layer;
    p.src_tp = a;
    p.dst_tp = b;
    for (int i = 0; i < p.n_descs; ++i) p.descs[i] = descs[i];
    p.n_layers = nl;
    p.dst_base = nl * a * kNumTensors;
    for (int l = 0; l < nl; ++l) {
        for (int r = 0; r < a; ++r)
            for (int t = 0; t < kNumTensors; ++t)
                p.ptrs[(l * a + r) * kNumTensors + t] = slots(&src[(size_t)r * L + l0 + l])[t];
        for (int r = 0; r < b; ++r)
            for (int t = 0; t < kNumTensors; ++t)
                p.ptrs[p.dst_base + (l * b + r) * kNumTensors + t] = slots(&dst[(size_t)r * L + l0 + l])[t];
    }
}

// Every buffer a descriptor names must be present, aligned and not the same on both sides, for every requested layer -
// except that a destination worker may be left out of a layer altogether (all seven pointers NULL): its shard is then
// not produced.
inline amoeba_status w_check_ptrs(const amoeba_plan* plan, const amoeba_layer_weights* src,
                                  const amoeba_layer_weights* dst, int layer_begin, int layer_end) {
    const int L = plan->src.model.num_layers;
    auto left_out = [&](int rank, int l) {
        void* const* sl = slots(&dst[(size_t)rank * L + l]);
        for (int t = 0; t < kNumTensors; ++t)
            if (sl[t]) return false;
        return true;
    };
    for (int l = layer_begin; l < layer_end; ++l)
        for (const WDescDev& d : plan->wdev) {
            const int dst_rank = d.dst_slot / kNumTensors;
            const void* t = slots(&dst[(size_t)dst_rank * L + l])[d.dst_slot % kNumTensors];
            if (!t && left_out(dst_rank, l)) continue;
            const void* s = slots(&src[(size_t)(d.src_slot / kNumTensors) * L + l])[d.src_slot % kNumTensors];
            if (!s || !t || s == t) return AMOEBA_ERR_INVALID_ARG;  // out of place: never the same buffer
            if (reinterpret_cast<uintptr_t>(s) % 16 || reinterpret_cast<uintptr_t>(t) % 16) return AMOEBA_ERR_ALIGNMENT;
        }
    return AMOEBA_OK;
}

// Largest work item of a descriptor list, in bytes (the ring kernels' stage size).
inline int w_stage_bytes(const std::vector<WDescDev>& descs) {
    int64_t stage_bytes = 16;
    for (const WDescDev& d : descs) stage_bytes = std::max<int64_t>(stage_bytes, (int64_t)d.rows_per_item * d.chunk_bytes);
    return (int)stage_bytes;
}

}  // namespace amoeba
