// Model weight transformation (Sec. 3.2): the copy that re-partitions one instance's projection weights from
// TP = a shards to TP = b shards.  Which rows / columns a worker holds is Eq. 1's partition (storage [out,in]):
// q/k/v/gate/up by output rows - contiguous runs; o_proj/down_proj by input columns - `hidden` strided runs per
// (source worker, destination worker) pair.  The planner has reduced all of it to a short per-layer list of 2-D copy
// descriptors; this kernel cuts them into work items and deals the items of all requested layers to a persistent grid.
#include <cuda_runtime.h>

#include "copy_engine.cuh"
#include "launch.hpp"
#include "plan.hpp"

namespace amoeba {

struct WParams {
    WDescDev descs[kMaxWeightDescs];
    void* ptrs[kMaxWeightPtrs];  // [layer][src rank][tensor] then, from dst_base, [layer][dst rank][tensor]
    int32_t n_descs, items_per_layer, n_layers, src_tp, dst_tp, dst_base;
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
        return it;
    }
};

template <int UNROLL, int CTAS_PER_SM>
__global__ void __launch_bounds__(256, CTAS_PER_SM) w_reshard_ldst(const __grid_constant__ WParams p) {
    const WItems items{p};
    const int64_t n = items.count();
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < n; w += n_warps)
        warp_copy_item<UNROLL>(items(w));
}

__global__ void __launch_bounds__(1024) w_reshard_bulk(const __grid_constant__ WParams p, const RingShape rs,
                                                        int32_t* status) {
    extern __shared__ __align__(128) char smem[];
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem) + warp * rs.stages;
    char* stages = smem + kBarrierBytes + (int64_t)warp * rs.stages * rs.stage_bytes;
    const WItems items{p};
    const bool ok = warp_bulk_ring(items, items.count(), (int64_t)blockIdx.x * nwarps + warp,
                                   (int64_t)gridDim.x * nwarps, stages, bars, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

__global__ void __launch_bounds__(1024) w_reshard_pair(const __grid_constant__ WParams p, const RingShape rs,
                                                        int32_t* status) {
    extern __shared__ __align__(128) char smem[];
    const int warp = threadIdx.x >> 5, ring = warp >> 1, role = warp & 1, nrings = blockDim.x >> 6;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem) + ring * 2 * rs.stages;
    uint64_t* empty = full + rs.stages;
    char* stages = smem + kBarrierBytes + (int64_t)ring * rs.stages * rs.stage_bytes;
    if (role == 0 && (threadIdx.x & 31) == 0) pair_ring_init(full, empty, rs.stages);
    __syncthreads();
    const WItems items{p};
    const bool ok = pair_bulk_ring(role, items, items.count(), (int64_t)blockIdx.x * nrings + ring,
                                   (int64_t)gridDim.x * nrings, stages, full, empty, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

static void* const* slots(const amoeba_layer_weights* w) { return reinterpret_cast<void* const*>(w); }

}  // namespace amoeba

using namespace amoeba;

extern "C" amoeba_status amoeba_reshard_weights(const amoeba_plan* plan, const amoeba_layer_weights* src,
                                                const amoeba_layer_weights* dst, int32_t layer_begin,
                                                int32_t layer_end, int32_t* d_status, void* cuda_stream) {
    static_assert(sizeof(amoeba_layer_weights) == kNumTensors * sizeof(void*), "slot view of the weight struct");
    if (!plan || !src || !dst || !d_status) return AMOEBA_ERR_INVALID_ARG;
    const int L = plan->src.model.num_layers, a = plan->src.tp, b = plan->dst.tp;
    if (layer_begin < 0 || layer_end > L || layer_begin > layer_end) return AMOEBA_ERR_INVALID_ARG;
    const int n_descs = (int)plan->wdev.size();
    // Every buffer a descriptor names must be present and aligned, for every requested layer - except that a
    // destination worker may be left out of a layer altogether (all seven pointers NULL): its shard is then not produced.
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
            if (!s || !t) return AMOEBA_ERR_INVALID_ARG;
            if (reinterpret_cast<uintptr_t>(s) % 16 || reinterpret_cast<uintptr_t>(t) % 16) return AMOEBA_ERR_ALIGNMENT;
        }
    if (layer_begin == layer_end || n_descs == 0) return AMOEBA_OK;

    DeviceInfo dev;
    if (!device_info(&dev)) return AMOEBA_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const KernelOpts& opt = plan->opt.w;
    const int path = opt.copy_path ? opt.copy_path : kWDefaults.copy_path;
    int stage_bytes = 16;
    for (const WDescDev& d : plan->wdev)
        stage_bytes = std::max<int64_t>(stage_bytes, (int64_t)d.rows_per_item * d.chunk_bytes);
    const int layers_per_launch = std::max(1, kMaxWeightPtrs / ((a + b) * kNumTensors));

    WParams p;  // large: filled per launch
    p.n_descs = n_descs;
    p.items_per_layer = plan->items_per_layer;
    p.src_tp = a;
    p.dst_tp = b;
    for (int i = 0; i < n_descs; ++i) p.descs[i] = plan->wdev[i];
    for (int l0 = layer_begin; l0 < layer_end; l0 += layers_per_launch) {
        const int nl = std::min(layers_per_launch, layer_end - l0);
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
        const int64_t n_items = (int64_t)p.items_per_layer * nl;
        cudaError_t e;
        if (path == 1) {
            const int per_sm = opt.ctas_per_sm ? opt.ctas_per_sm : kLdstCtasPerSm;
            const int grid = (int)std::min<int64_t>((n_items + 7) / 8, grid_cap(opt, (int64_t)dev.sms * per_sm));
            if (per_sm <= 2) w_reshard_ldst<8, 2><<<grid, 256, 0, stream>>>(p);
            else if (per_sm == 3) w_reshard_ldst<6, 3><<<grid, 256, 0, stream>>>(p);
            else w_reshard_ldst<4, 4><<<grid, 256, 0, stream>>>(p);
            e = cudaGetLastError();
        } else {
            const BulkShape bs = bulk_shape(dev, opt, kWDefaults, path, stage_bytes);
            const int grid = (int)std::min<int64_t>((n_items + bs.rings - 1) / bs.rings, grid_cap(opt, (int64_t)dev.sms * bs.ctas_per_sm));
            auto kernel = path == 3 ? w_reshard_pair : w_reshard_bulk;
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bs.smem);
            if (e == cudaSuccess) {
                kernel<<<grid, bs.threads, bs.smem, stream>>>(p, bs.ring, d_status);
                e = cudaGetLastError();
            }
        }
        if (e != cudaSuccess) return AMOEBA_ERR_CUDA;
        count_launch();
    }
    return AMOEBA_OK;
}
