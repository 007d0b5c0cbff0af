// KV cache migration in the head dimension (Sec. 3.1) as an on-GPU gather/scatter between the pools of the
// source workers (TP = a) and of the destination workers (TP = b).  Either side may use the header-centric order
// [layer][block][header][K/V][token][dim] (Sec. 3.1, Improvement 1) or the token-first order
// [layer][K/V][block][token][header][dim] of mainstream engines.
//
// Work decomposition: (layer, pair, K/V plane, header unit, row group, column chunk).  A header unit is a group of
// consecutive headers that lives in exactly one source pool and one destination pool and is a regular 2-D copy on
// both sides (see KvGeom): with both sides header-centric it is a run of gcd(Hkv/a, Hkv/b) headers, K and V
// together, one contiguous row; with token-first on a side it is one row per token.  Units are cut into copy work
// items, dealt round-robin to a persistent grid; layer is the slowest index so that concurrently running CTAs touch
// neighbouring DRAM pages.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>
#include <new>

#include "copy_engine.cuh"
#include "kv_items.cuh"
#include "launch.hpp"
#include "plan.hpp"

namespace amoeba {

// Vector load/store path: one work item per warp at a time, warps strided over the items.
template <int UNROLL, int CTAS_PER_SM>
__global__ void __launch_bounds__(256, CTAS_PER_SM) kv_reshard_ldst(const __grid_constant__ KvParams p) {
    const KvItems items{p, clamp_pairs(p)};
    const int64_t n = items.count();
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < n; w += n_warps) {
        const Item it = items(w);
        if (it.n_rows) warp_copy_item<UNROLL>(it);
    }
}

// Dynamic shared memory: [kBarrierBytes of mbarriers][rings x stages x stage_bytes].
__global__ void __launch_bounds__(1024) kv_reshard_bulk(const __grid_constant__ KvParams p, const RingShape rs) {
    extern __shared__ __align__(128) char smem[];
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem) + warp * rs.stages;
    char* stages = smem + kBarrierBytes + (int64_t)warp * rs.stages * rs.stage_bytes;
    const KvItems items{p, clamp_pairs(p)};
    const bool ok = warp_bulk_ring(items, items.count(), (int64_t)blockIdx.x * nwarps + warp,
                                   (int64_t)gridDim.x * nwarps, stages, bars, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(p.status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

// Warps 2r and 2r+1 are the producer and the consumer of ring r.
__global__ void __launch_bounds__(1024) kv_reshard_pair(const __grid_constant__ KvParams p, const RingShape rs) {
    extern __shared__ __align__(128) char smem[];
    const PairRing r = pair_ring_setup(smem, rs);
    const KvItems items{p, clamp_pairs(p)};
    const bool ok = pair_bulk_ring(r.role, items, items.count(), (int64_t)blockIdx.x * r.nrings + r.ring,
                                   (int64_t)gridDim.x * r.nrings, r.stages, r.full, r.empty, r.abort, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(p.status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

// The same two ring kernels over box items (a side that is token-first goes through its tensor map).
__global__ void __launch_bounds__(1024) kv_reshard_bulk_box(const __grid_constant__ KvParams p,
                                                            const __grid_constant__ KvMaps maps, const RingShape rs) {
    extern __shared__ __align__(128) char smem[];
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem) + warp * rs.stages;
    char* stages = smem + kBarrierBytes + (int64_t)warp * rs.stages * rs.stage_bytes;
    const KvBoxItems items{p, maps, clamp_pairs(p)};
    const bool ok = warp_bulk_ring(items, items.count(), (int64_t)blockIdx.x * nwarps + warp,
                                   (int64_t)gridDim.x * nwarps, stages, bars, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(p.status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

__global__ void __launch_bounds__(1024) kv_reshard_pair_box(const __grid_constant__ KvParams p,
                                                            const __grid_constant__ KvMaps maps, const RingShape rs) {
    extern __shared__ __align__(128) char smem[];
    const PairRing r = pair_ring_setup(smem, rs);
    const KvBoxItems items{p, maps, clamp_pairs(p)};
    const bool ok = pair_bulk_ring(r.role, items, items.count(), (int64_t)blockIdx.x * r.nrings + r.ring,
                                   (int64_t)gridDim.x * r.nrings, r.stages, r.full, r.empty, r.abort, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(p.status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

// ---------------------------------------------------------------- in-place merge of N instances (Sec. 3.1, Impr. 1)
// Pools: [instance i][worker r] -> pools[i*a + r]; old block p of such a pool is N segments of Hkv/(N*a) headers;
// segment k is what merged worker r*N+k keeps.  For i < k the pair of segments (pool (i,r), block p, segment k) and
// (pool (k,r), block p, segment i) trade places; segment i of pool (i,r) stays.  A work item is one chunk of such a
// pair: both live -> a two-row item whose rows are read from A and B and written to B and A (the rings read a whole
// item into a stage before they write any of it); one live -> a plain copy; none -> skipped.
struct MergeParams {
    char* pools[AMOEBA_MAX_TP];
    const uint8_t* live;  // [N][nb]
    int64_t layer_stride, block_bytes, seg_bytes, chunk_bytes;
    int32_t n_inst, a, nb, layer_begin, n_layers, chunks_per_seg, n_pairs;
    int32_t split;  // 0: merge (a live block sends its segments away), 1: the way back (a live block gathers them)
    int32_t* status;
    int64_t span;   // bytes of a pool the layers of this call reach into
};

struct MergeItems {
    const MergeParams& p;
    __device__ __forceinline__ int64_t count() const {
        return (int64_t)p.n_layers * p.nb * p.a * p.n_pairs * p.chunks_per_seg;
    }
    __device__ __forceinline__ Item operator()(int64_t w) const {
        const int32_t ipb = p.a * p.n_pairs * p.chunks_per_seg;  // items of one (layer, block)
        const int64_t lb = w / ipb;
        uint32_t rem = (uint32_t)(w - lb * ipb);
        const int32_t chunk = take_digit(rem, p.chunks_per_seg);
        int32_t pr = take_digit(rem, p.n_pairs);
        const int32_t r = (int32_t)rem;  // < a
        const int32_t blk = (int32_t)(lb % p.nb);
        const int32_t layer = p.layer_begin + (int32_t)(lb / p.nb);
        int32_t i = 0;  // pr-th pair (i, k) with i < k, in lexicographic order
        while (pr >= p.n_inst - 1 - i) {
            pr -= p.n_inst - 1 - i;
            ++i;
        }
        const int32_t k = i + 1 + pr;
        const bool live_i = p.live[(int64_t)i * p.nb + blk] != 0, live_k = p.live[(int64_t)k * p.nb + blk] != 0;
        Item it;
        it.src_map = it.dst_map = nullptr;
        it.n_rows = 0;
        it.row_bytes = (int32_t)p.chunk_bytes;
        it.src = nullptr;
        it.dst = nullptr;
        it.src_pitch = it.dst_pitch = 0;
        if (!live_i && !live_k) return it;
        const int64_t base = layer * p.layer_stride + (int64_t)blk * p.block_bytes + (int64_t)chunk * p.chunk_bytes;
        char* A = p.pools[i * p.a + r] + base + k * p.seg_bytes;  // leaves instance i's worker for merged worker r*N+k
        char* B = p.pools[k * p.a + r] + base + i * p.seg_bytes;  // leaves instance k's worker for merged worker r*N+i
#ifdef AMOEBA_CHECK_ITEMS
        if (!rows_inside(A - p.pools[i * p.a + r], 0, 1, (int32_t)p.chunk_bytes, p.span) ||
            !rows_inside(B - p.pools[k * p.a + r], 0, 1, (int32_t)p.chunk_bytes, p.span)) {
            atomicCAS(p.status, 0, (int)AMOEBA_ERR_INTERNAL);
            return it;
        }
#endif
        if (live_i && live_k) {
            it.n_rows = 2;
            it.src = A;
            it.src_pitch = B - A;
            it.dst = B;
            it.dst_pitch = A - B;
        } else {
            // merge: the live block's segment leaves for the other worker; split: the live block fetches its segment
            const bool a_to_b = (live_i != 0) != (p.split != 0);
            it.n_rows = 1;
            it.src = a_to_b ? A : B;
            it.dst = a_to_b ? B : A;
        }
        return it;
    }
};

__global__ void __launch_bounds__(1024) kv_merge_bulk(const __grid_constant__ MergeParams p, const RingShape rs,
                                                      int32_t* status) {
    extern __shared__ __align__(128) char smem[];
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem) + warp * rs.stages;
    char* stages = smem + kBarrierBytes + (int64_t)warp * rs.stages * rs.stage_bytes;
    const MergeItems items{p};
    const bool ok = warp_bulk_ring(items, items.count(), (int64_t)blockIdx.x * nwarps + warp,
                                   (int64_t)gridDim.x * nwarps, stages, bars, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

__global__ void __launch_bounds__(1024) kv_merge_pair(const __grid_constant__ MergeParams p, const RingShape rs,
                                                      int32_t* status) {
    extern __shared__ __align__(128) char smem[];
    const PairRing r = pair_ring_setup(smem, rs);
    const MergeItems items{p};
    const bool ok = pair_bulk_ring(r.role, items, items.count(), (int64_t)blockIdx.x * r.nrings + r.ring,
                                   (int64_t)gridDim.x * r.nrings, r.stages, r.full, r.empty, r.abort, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

// cuTensorMapEncodeTiled, looked up through the runtime so that the library does not link against the driver.
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

// Tensor map of one worker's token-first pool [layer][K/V][block][token][header][dim] (1-, 2- or 4-byte elements), with the
// dimensions ordered {dim, token, K/V, header, layer} so that a box lands in shared memory as
// [header][K/V][token][dim]: the header-centric order of the same data.
constexpr int kDefaultL2Promotion = 1;  // 1 + CU_TENSOR_MAP_L2_PROMOTION_NONE
static bool encode_pool_map(CUtensorMap* out, const void* pool, const amoeba_layout& lay, int64_t layer_stride,
                            int32_t heads, int64_t vec_bytes, const KvBoxGeom& bx, int l2_promotion) {
    const int promo = (l2_promotion ? l2_promotion : kDefaultL2Promotion) - 1;
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return false;
    const cuuint64_t T = (cuuint64_t)lay.block_tokens, NB = (cuuint64_t)lay.num_blocks;
    const cuuint64_t dims[5] = {(cuuint64_t)lay.model.head_dim, NB * T, 2, (cuuint64_t)heads,
                                (cuuint64_t)lay.model.num_layers};
    const cuuint64_t strides[4] = {(cuuint64_t)heads * vec_bytes,           // next token
                                   NB * T * (cuuint64_t)heads * vec_bytes,   // K region -> V region
                                   (cuuint64_t)vec_bytes,                    // next header of the same token
                                   (cuuint64_t)layer_stride};
    const cuuint32_t box[5] = {(cuuint32_t)lay.model.head_dim, (cuuint32_t)bx.tokens, 2, (cuuint32_t)bx.heads, 1};
    const cuuint32_t elem_strides[5] = {1, 1, 1, 1, 1};
    const int e = lay.model.elem_bytes;  // the elements are opaque: any unsigned type of their size will do
    const CUtensorMapDataType type = e == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                            : e == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32;
    return encode(out, type, 5, const_cast<void*>(pool), dims, strides, box, elem_strides,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, (CUtensorMapL2promotion)promo,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace amoeba

using namespace amoeba;

// Encoded tensor maps of a plan's token-first pools, kept while the pool addresses and the plan's options stay the same.
struct LaunchCache {
    std::mutex mutex;
    uint64_t generation = 0;  // plan generation the maps were encoded for (0 = none yet)
    const void* src[AMOEBA_MAX_TP] = {};
    const void* dst[AMOEBA_MAX_TP] = {};
    amoeba::KvMaps maps;
};

amoeba_plan::~amoeba_plan() { delete cache; }

namespace amoeba {

// Fills *maps for the given pools: from the plan's cache when nothing changed since they were last encoded.
static bool pool_maps(const amoeba_plan* plan, const KvParams& p, KvMaps* maps) {
    static std::mutex create_mutex;
    amoeba_plan* mp = const_cast<amoeba_plan*>(plan);  // the cache is the plan's only state that data calls change
    {
        std::lock_guard<std::mutex> lock(create_mutex);
        if (!mp->cache) mp->cache = new (std::nothrow) LaunchCache();
        if (!mp->cache) return false;
    }
    LaunchCache& c = *mp->cache;
    std::lock_guard<std::mutex> lock(c.mutex);
    const uint64_t gen = plan->generation.load(std::memory_order_relaxed);
    bool same = c.generation == gen;
    for (int r = 0; same && r < plan->src.tp; ++r) same = c.src[r] == p.src[r];
    for (int r = 0; same && r < plan->dst.tp; ++r) same = c.dst[r] == p.dst[r];
    if (!same) {
        c.generation = 0;
        std::memset(&c.maps, 0, sizeof(c.maps));
        if (p.src_token_major)
            for (int r = 0; r < plan->src.tp; ++r)
                if (!encode_pool_map(&c.maps.src[r], p.src[r], plan->src, plan->src_layer_stride, plan->heads_src,
                                     plan->vec_bytes, plan->kvbox, plan->opt.kv.l2_promotion))
                    return false;
        if (p.dst_token_major)
            for (int r = 0; r < plan->dst.tp; ++r)
                if (!encode_pool_map(&c.maps.dst[r], p.dst[r], plan->dst, plan->dst_layer_stride, plan->heads_dst,
                                     plan->vec_bytes, plan->kvbox, plan->opt.kv.l2_promotion))
                    return false;
        for (int r = 0; r < plan->src.tp; ++r) c.src[r] = p.src[r];
        for (int r = 0; r < plan->dst.tp; ++r) c.dst[r] = p.dst[r];
        c.generation = gen;
    }
    *maps = c.maps;
    return true;
}

// Geometry from the plan, then the launch of the chosen copy kernel.  p.src / p.dst / pairs / status / layer range /
// reshape are set by the caller.
static amoeba_status launch_kv(const amoeba_plan* plan, KvParams& p, cudaStream_t stream) {
    kv_fill_geometry(plan, p);
    const KvGeom& g = plan->kv;
    const KvBoxGeom& bx = plan->kvbox;

    const DeviceInfo dev = cached_device_info();
    if (dev.sms <= 0) return AMOEBA_ERR_CUDA;
    cudaError_t e;
    const KernelOpts& opt = plan->opt.kv;
    const int path = opt.copy_path ? opt.copy_path : kKvDefaults.copy_path;
    const bool token_side = p.src_token_major || p.dst_token_major;
    const bool boxes = path != 1 && token_side && bx.usable && opt.tensor_maps != 1;
    const int64_t items_per_pair = boxes ? (int64_t)p.runs_per_block * bx.sub_runs * bx.tok_groups
                                         : (int64_t)g.planes * p.moving_units * g.row_groups * g.col_chunks;
    const int64_t max_items = (int64_t)p.pairs_cap * p.n_layers * items_per_pair;
    if (max_items == 0) return AMOEBA_OK;
    if (path == 1) {
        const int per_sm = opt.ctas_per_sm ? opt.ctas_per_sm : kLdstCtasPerSm;
        const int grid = (int)std::min<int64_t>((max_items + 7) / 8, grid_cap(opt, (int64_t)dev.sms * per_sm));
        if (per_sm <= 2) kv_reshard_ldst<8, 2><<<grid, 256, 0, stream>>>(p);
        else if (per_sm == 3) kv_reshard_ldst<6, 3><<<grid, 256, 0, stream>>>(p);
        else kv_reshard_ldst<4, 4><<<grid, 256, 0, stream>>>(p);
        e = cudaGetLastError();
    } else if (boxes) {
        KvMaps maps;
        if (!pool_maps(plan, p, &maps)) return AMOEBA_ERR_CUDA;
        const int stage_bytes = (int)((bx.item_bytes + 127) / 128 * 128);  // tiled copies want 128-byte aligned stages
        const BulkShape bs = bulk_shape(dev, opt, kKvDefaults, path, stage_bytes);
        const int grid = (int)std::min<int64_t>((max_items + bs.rings - 1) / bs.rings, grid_cap(opt, (int64_t)dev.sms * bs.ctas_per_sm));
        auto kernel = path == 3 ? kv_reshard_pair_box : kv_reshard_bulk_box;
        e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)bs.smem);
        if (e == cudaSuccess) {
            kernel<<<grid, bs.threads, bs.smem, stream>>>(p, maps, bs.ring);
            e = cudaGetLastError();
        }
    } else {
        const BulkShape bs = bulk_shape(dev, opt, kKvDefaults, path, (int)g.item_bytes);
        const int grid = (int)std::min<int64_t>((max_items + bs.rings - 1) / bs.rings, grid_cap(opt, (int64_t)dev.sms * bs.ctas_per_sm));
        auto kernel = path == 3 ? kv_reshard_pair : kv_reshard_bulk;
        e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)bs.smem);
        if (e == cudaSuccess) {
            kernel<<<grid, bs.threads, bs.smem, stream>>>(p, bs.ring);
            e = cudaGetLastError();
        }
    }
    if (e != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    return AMOEBA_OK;
}

}  // namespace amoeba

extern "C" amoeba_status amoeba_reshard_kv(const amoeba_plan* plan, const void* const* src_pools,
                                           void* const* dst_pools, const int32_t* d_pairs, const int32_t* d_num_pairs,
                                           int32_t pairs_cap, int32_t layer_begin, int32_t layer_end, int32_t* d_status,
                                           void* cuda_stream) {
    if (!plan || !src_pools || !dst_pools || !d_pairs || !d_num_pairs || !d_status || pairs_cap < 0)
        return AMOEBA_ERR_INVALID_ARG;
    const amoeba_model& m = plan->src.model;
    if (layer_begin < 0 || layer_end > m.num_layers || layer_begin > layer_end) return AMOEBA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_pairs) % 8) return AMOEBA_ERR_ALIGNMENT;
    KvParams p{};
    const amoeba_status pools_ok = kv_set_pools(plan, src_pools, dst_pools, p);
    if (pools_ok != AMOEBA_OK) return pools_ok;
    if (pairs_cap == 0 || layer_begin == layer_end) return AMOEBA_OK;
    p.pairs = d_pairs;
    p.num_pairs = d_num_pairs;
    p.status = d_status;
    p.pairs_cap = pairs_cap;
    p.layer_begin = layer_begin;
    p.n_layers = layer_end - layer_begin;
    return launch_kv(plan, p, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" amoeba_status amoeba_reshape_kv_inplace(const amoeba_plan* plan, void* const* pools, const int32_t* d_pairs,
                                                   const int32_t* d_num_pairs, int32_t pairs_cap, int32_t layer_begin,
                                                   int32_t layer_end, int32_t* d_status, void* cuda_stream) {
    if (!plan || !pools || !d_pairs || !d_num_pairs || !d_status || pairs_cap < 0) return AMOEBA_ERR_INVALID_ARG;
    const int f = reshape_factor(plan);
    if (!f) return AMOEBA_ERR_UNSUPPORTED;
    const int n = f > 0 ? f : -f;
    const amoeba_model& m = plan->src.model;
    if (layer_begin < 0 || layer_end > m.num_layers || layer_begin > layer_end) return AMOEBA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_pairs) % 8) return AMOEBA_ERR_ALIGNMENT;
    const int fine = std::max(plan->src.tp, plan->dst.tp);
    KvParams p{};
    for (int w = 0; w < fine; ++w) {
        if (!pools[w]) return AMOEBA_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(pools[w]) % 16) return AMOEBA_ERR_ALIGNMENT;
        for (int v = 0; v < w; ++v)
            if (pools[v] == pools[w]) return AMOEBA_ERR_INVALID_ARG;  // every worker has its own memory
    }
    // the finer side indexes pools directly; worker r of the coarser side lives in pools[r * N]
    for (int r = 0; r < plan->src.tp; ++r) p.src[r] = static_cast<const char*>(pools[f > 0 ? r * n : r]);
    for (int r = 0; r < plan->dst.tp; ++r) p.dst[r] = static_cast<char*>(pools[f > 0 ? r : r * n]);
    if (pairs_cap == 0 || layer_begin == layer_end) return AMOEBA_OK;
    p.pairs = d_pairs;
    p.num_pairs = d_num_pairs;
    p.status = d_status;
    p.pairs_cap = pairs_cap;
    p.layer_begin = layer_begin;
    p.n_layers = layer_end - layer_begin;
    p.reshape = f;
    return launch_kv(plan, p, static_cast<cudaStream_t>(cuda_stream));
}

static amoeba_status merge_or_split_kv(bool split, const amoeba_plan* plan, void* const* pools, const uint8_t* d_live,
                                       int32_t layer_begin, int32_t layer_end, int32_t* d_status, void* cuda_stream) {
    if (!plan || !pools || !d_live || !d_status) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_model& m = plan->src.model;
    if (layer_begin < 0 || layer_end > m.num_layers || layer_begin > layer_end) return AMOEBA_ERR_INVALID_ARG;
    const int n = merge_instances(plan);
    if (!n) return AMOEBA_ERR_UNSUPPORTED;
    const int a = plan->src.tp;
    MergeParams p{};
    for (int w = 0; w < n * a; ++w) {
        if (!pools[w]) return AMOEBA_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(pools[w]) % 16) return AMOEBA_ERR_ALIGNMENT;
        for (int v = 0; v < w; ++v)
            if (pools[v] == pools[w]) return AMOEBA_ERR_INVALID_ARG;  // every worker has its own memory
        p.pools[w] = static_cast<char*>(pools[w]);
    }
    if (layer_begin == layer_end) return AMOEBA_OK;
    const KernelOpts& opt = plan->opt.kv;
    const int64_t cap = std::max<int64_t>(16, (opt.chunk_bytes > 0 ? opt.chunk_bytes : kDefaultKvChunk) / 2);
    p.live = d_live;
    p.layer_stride = plan->src_layer_stride;
    p.block_bytes = plan->src_block_bytes;
    p.seg_bytes = plan->dst_block_bytes;  // one new block = one segment of an old block
    p.chunk_bytes = p.seg_bytes;          // largest divisor of the segment that is a multiple of 16 and <= cap
    for (int64_t parts = std::max<int64_t>(1, (p.seg_bytes + cap - 1) / cap); parts <= p.seg_bytes / 16; ++parts)
        if (p.seg_bytes % parts == 0 && (p.seg_bytes / parts) % 16 == 0) {
            p.chunk_bytes = p.seg_bytes / parts;
            break;
        }
    if (p.chunk_bytes > 65536) return AMOEBA_ERR_UNSUPPORTED;
    p.chunks_per_seg = (int32_t)(p.seg_bytes / p.chunk_bytes);
    p.n_inst = n;
    p.a = a;
    p.nb = plan->src.num_blocks;
    p.layer_begin = layer_begin;
    p.n_layers = layer_end - layer_begin;
    p.n_pairs = n * (n - 1) / 2;
    p.split = split ? 1 : 0;
    p.status = d_status;
    p.span = (int64_t)layer_end * p.layer_stride;

    const DeviceInfo dev = cached_device_info();
    if (dev.sms <= 0) return AMOEBA_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int path = opt.copy_path == 2 ? 2 : 3;  // a swap needs a staged copy: the rings only
    const BulkShape bs = bulk_shape(dev, opt, kMergeDefaults, path, (int)(2 * p.chunk_bytes));
    const int64_t n_items = (int64_t)p.n_layers * p.nb * p.a * p.n_pairs * p.chunks_per_seg;
    const int grid = (int)std::min<int64_t>((n_items + bs.rings - 1) / bs.rings, grid_cap(opt, (int64_t)dev.sms * bs.ctas_per_sm));
    auto kernel = path == 3 ? kv_merge_pair : kv_merge_bulk;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)bs.smem);
    if (e == cudaSuccess) {
        kernel<<<grid, bs.threads, bs.smem, stream>>>(p, bs.ring, d_status);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    return AMOEBA_OK;
}

extern "C" amoeba_status amoeba_merge_kv_inplace(const amoeba_plan* plan, void* const* pools, const uint8_t* d_live,
                                                 int32_t layer_begin, int32_t layer_end, int32_t* d_status,
                                                 void* cuda_stream) {
    return merge_or_split_kv(false, plan, pools, d_live, layer_begin, layer_end, d_status, cuda_stream);
}

extern "C" amoeba_status amoeba_split_kv_inplace(const amoeba_plan* plan, void* const* pools, const uint8_t* d_live,
                                                 int32_t layer_begin, int32_t layer_end, int32_t* d_status,
                                                 void* cuda_stream) {
    return merge_or_split_kv(true, plan, pools, d_live, layer_begin, layer_end, d_status, cuda_stream);
}
