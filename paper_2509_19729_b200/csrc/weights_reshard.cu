// Model weight transformation (Sec. 3.2): the copy that re-partitions one instance's projection weights from
// TP = a shards to TP = b shards.  Which rows / columns a worker holds is Eq. 1's partition (storage [out,in]):
// q/k/v/gate/up by output rows - contiguous runs; o_proj/down_proj by input columns - `hidden` strided runs per
// (source worker, destination worker) pair.  The planner has reduced all of it to a short per-layer list of 2-D copy
// descriptors; this kernel cuts them into work items and deals the items of all requested layers to a persistent grid.
#include <cuda_runtime.h>

#include "copy_engine.cuh"
#include "launch.hpp"
#include "plan.hpp"
#include "w_items.cuh"

namespace amoeba {

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
    const PairRing r = pair_ring_setup(smem, rs);
    const WItems items{p};
    const bool ok = pair_bulk_ring(r.role, items, items.count(), (int64_t)blockIdx.x * r.nrings + r.ring,
                                   (int64_t)gridDim.x * r.nrings, r.stages, r.full, r.empty, r.abort, rs);
    if (!ok && (threadIdx.x & 31) == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_TIMEOUT);
}

// Launches the copy kernel over `descs` (per-layer descriptors in kernel form, `items_per_layer` work items) for the
// layers [layer_begin, layer_end): src is [src_tp][L], dst is [dst_tp][L] (worker-major host arrays of device pointers).
static amoeba_status launch_descs(const amoeba_plan* plan, const std::vector<WDescDev>& descs, int32_t items_per_layer,
                                  const amoeba_layer_weights* src, int src_tp, const amoeba_layer_weights* dst,
                                  int dst_tp, int L, int layer_begin, int layer_end, int32_t* d_status,
                                  cudaStream_t stream) {
    const int n_descs = (int)descs.size();
    if (layer_begin == layer_end || n_descs == 0 || items_per_layer == 0) return AMOEBA_OK;
    const DeviceInfo dev = cached_device_info();
    if (dev.sms <= 0) return AMOEBA_ERR_CUDA;
    const KernelOpts& opt = plan->opt.w;
    const int path = opt.copy_path ? opt.copy_path : kWDefaults.copy_path;
    const int stage_bytes = w_stage_bytes(descs);
    const int a = src_tp, b = dst_tp;
    const int layers_per_launch = weight_layers_per_launch(a, b);

    WParams p;  // large: filled per launch
    p.status = d_status;
    const amoeba_layout& dst_layout = src == dst ? plan->src : plan->dst;  // in place: one set of buffers, one layout
    for (int t = 0; t < kNumTensors; ++t) {
        amoeba_layout_weight_bytes(&plan->src, t, &p.src_bytes[t]);
        amoeba_layout_weight_bytes(&dst_layout, t, &p.dst_bytes[t]);
    }
    for (int l0 = layer_begin; l0 < layer_end; l0 += layers_per_launch) {
        const int nl = std::min(layers_per_launch, layer_end - l0);
        w_fill_params(p, descs, items_per_layer, src, a, dst, b, L, l0, nl);
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
            const int grid = (int)std::min<int64_t>((n_items + bs.rings - 1) / bs.rings,
                                                    grid_cap(opt, (int64_t)dev.sms * bs.ctas_per_sm));
            auto kernel = path == 3 ? w_reshard_pair : w_reshard_bulk;
            e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)bs.smem);
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

}  // namespace amoeba

using namespace amoeba;

extern "C" amoeba_status amoeba_reshard_weights(const amoeba_plan* plan, const amoeba_layer_weights* src,
                                                const amoeba_layer_weights* dst, int32_t layer_begin,
                                                int32_t layer_end, int32_t* d_status, void* cuda_stream) {
    static_assert(sizeof(amoeba_layer_weights) == kNumTensors * sizeof(void*), "slot view of the weight struct");
    if (!plan || !src || !dst || !d_status) return AMOEBA_ERR_INVALID_ARG;
    const int L = plan->src.model.num_layers, a = plan->src.tp, b = plan->dst.tp;
    if (layer_begin < 0 || layer_end > L || layer_begin > layer_end) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_status ptrs_ok = w_check_ptrs(plan, src, dst, layer_begin, layer_end);
    if (ptrs_ok != AMOEBA_OK) return ptrs_ok;
    return launch_descs(plan, plan->wdev, plan->items_per_layer, src, a, dst, b, L, layer_begin, layer_end, d_status,
                        static_cast<cudaStream_t>(cuda_stream));
}

// ------------------------------------------------------------------------------------------------------------
// Partial swap (Sec. 3.2, base solution): a worker of TP = a that becomes a worker of TP = N*a keeps one N-th of
// every shard and moves it to the front of the buffer it is in, so that the rest can be released.  In place, hence
// ordered: a phase only writes bytes whose old content an earlier phase has already moved (or that are not kept).
//   rows (q, k, v, gate, up): one contiguous move per member; inside a fused buffer q moves first, then k, then v
//     (the new k section may lie where the kept q rows were);
//   columns (o_proj, down_proj): row j of the kept column range moves from j*w + keep*w/N to j*w/N; rows are done in
//     waves [0,1), [1,N), [N,N^2), ...: the destination of wave [m, N*m) ends at byte m*w, where its sources begin.
// The leading waves of a column tensor are tiny (1, N-1, N^2-N ... rows): one CTA per buffer runs them back to back
// in a single launch of w_compact_lead, a CTA-wide barrier between waves (every wave only depends on earlier waves
// of the same buffer, and nothing a wave writes is read again).  The remaining waves and the row moves are separate
// launches of the copy kernel on the stream; within a launch all copies are disjoint.
namespace amoeba {

constexpr int kMaxLeadBufs = 1024;          // buffers (layer, worker, column tensor) per launch of the lead kernel
constexpr int64_t kLeadBytes = 1 << 20;     // kept bytes one CTA moves for its buffer before the waves go grid-wide

struct LeadParams {
    char* bufs[kMaxLeadBufs];
    uint8_t cls[kMaxLeadBufs];   // 0 = o_proj, 1 = down_proj
    uint8_t keep[kMaxLeadBufs];  // which N-th of the columns the buffer's worker keeps
    int64_t w_old[2], w_new[2];  // bytes of a row before / after
    int32_t rows[2];             // rows [0, rows[c]) are moved here
    int32_t n;                   // N
};

constexpr int kLeadThreads = 1024;
constexpr int kLeadUnroll = 8;  // 16-byte loads in flight per thread: 128 KiB per CTA

__global__ void __launch_bounds__(kLeadThreads, 1) w_compact_lead(const __grid_constant__ LeadParams p) {
    const int b = blockIdx.x, c = p.cls[b];
    char* base = p.bufs[b];
    const int64_t w_old = p.w_old[c], w_new = p.w_new[c], keep_off = p.keep[b] * w_new;
    const int vpr = (int)(w_new >> 4);  // 16-byte vectors per row
    int64_t lo = 0, hi = 1;
    while (lo < p.rows[c]) {
        if (hi > p.rows[c]) hi = p.rows[c];
        // the wave's rows as one flat list of vectors, dealt to all threads; every load of a batch before its stores
        const int first = (lo == 0 && keep_off == 0) ? vpr : 0;  // row 0 of the first column range is in place
        const int n = (int)(hi - lo) * vpr;
        for (int i0 = first + threadIdx.x; i0 < n; i0 += kLeadThreads * kLeadUnroll) {
            uint4 v[kLeadUnroll];
#pragma unroll
            for (int u = 0; u < kLeadUnroll; ++u) {
                const int i = i0 + u * kLeadThreads;
                if (i < n) {
                    const int r = i / vpr, col = i - r * vpr;
                    v[u] = ld_stream(reinterpret_cast<const uint4*>(base + (lo + r) * w_old + keep_off) + col);
                }
            }
#pragma unroll
            for (int u = 0; u < kLeadUnroll; ++u) {
                const int i = i0 + u * kLeadThreads;
                if (i < n) {
                    const int r = i / vpr, col = i - r * vpr;
                    st_stream(reinterpret_cast<uint4*>(base + (lo + r) * w_new) + col, v[u]);
                }
            }
        }
        __syncthreads();  // every load of this wave has returned (its stores were issued after them)
        lo = hi;
        hi *= p.n;
    }
}

struct CompactSchedule {
    std::vector<std::vector<amoeba_weight_desc>> phases;  // copy-kernel launches, in order
    int32_t lead_rows[2] = {0, 0};                        // rows of o_proj / down_proj the lead kernel moves
    int64_t w_old[2] = {0, 0}, w_new[2] = {0, 0};
    int64_t bytes_per_layer = 0;                          // bytes read (= written) per layer, all workers
};

enum { Q, K, V, O, GATE, UP, DOWN };

// What moves where for plan->src (TP = a) -> plan->dst (TP = N*a) with worker r keeping sub-shard keep[r].
static void compact_schedule(const amoeba_plan* plan, const int32_t* keep, CompactSchedule* out) {
    const amoeba_layout &sl = plan->src, &dl = plan->dst;
    const amoeba_model& m = sl.model;
    const int a = sl.tp, b = dl.tp, N = b / a;
    const int64_t e = m.elem_bytes, hid = m.hidden, rb = hid * e;
    const int64_t rows_of[kNumTensors] = {(int64_t)m.num_q_heads * m.head_dim, (int64_t)m.num_kv_heads * m.head_dim,
                                          (int64_t)m.num_kv_heads * m.head_dim, 0, m.intermediate, m.intermediate, 0};
    // buffer and section offset (in rows of the old / the new shard) of every row-split member
    int buffer_of[kNumTensors] = {Q, K, V, O, GATE, UP, DOWN};
    int64_t sec_old[kNumTensors] = {0}, sec_new[kNumTensors] = {0};
    if (sl.fused_qkv) {
        buffer_of[K] = buffer_of[V] = Q;
        sec_old[K] = rows_of[Q] / a, sec_old[V] = (rows_of[Q] + rows_of[K]) / a;
        sec_new[K] = rows_of[Q] / b, sec_new[V] = (rows_of[Q] + rows_of[K]) / b;
    }
    if (sl.fused_gate_up) {
        buffer_of[UP] = GATE;
        sec_old[UP] = rows_of[GATE] / a, sec_new[UP] = rows_of[GATE] / b;
    }
    auto& phases = out->phases;
    auto phase = [&](size_t i) -> std::vector<amoeba_weight_desc>& {
        if (phases.size() <= i) phases.resize(i + 1);
        return phases[i];
    };
    // Inside a fused [q;k;v] buffer v may move together with k when its new place ends before the rows k is read
    // from (for every worker): (Rq + 2 Rk)/b <= Rq/a + keep*Rk/b.  Separate buffers never wait for one another.
    bool v_with_k = true;
    if (sl.fused_qkv)
        for (int r = 0; r < a; ++r)
            v_with_k = v_with_k && (rows_of[Q] + 2 * rows_of[K]) / b <= rows_of[Q] / a + keep[r] * (rows_of[K] / b);
    const int chains[2][3] = {{Q, K, V}, {GATE, UP, -1}};
    for (const auto& chain : chains)
        for (int pos = 0; pos < 3 && chain[pos] >= 0; ++pos) {
            const int t = chain[pos];
            int step = pos;
            if (!sl.fused_qkv && (t == K || t == V)) step = 0;        // buffers of their own
            else if (t == V && v_with_k) step = 1;
            if (!sl.fused_gate_up && t == UP) step = 0;
            for (int r = 0; r < a; ++r) {
                amoeba_weight_desc d{};
                d.src_rank = d.dst_rank = r;
                d.src_tensor = d.dst_tensor = buffer_of[t];
                d.row_bytes = rows_of[t] / b * rb;
                d.src_off = (sec_old[t] + keep[r] * (rows_of[t] / b)) * rb;
                d.dst_off = sec_new[t] * rb;
                d.n_rows = 1;
                d.src_pitch = d.dst_pitch = d.row_bytes;
                if (d.src_off != d.dst_off) {
                    phase(step).push_back(d);
                    out->bytes_per_layer += d.row_bytes;
                }
            }
        }
    const int col_tensors[2] = {O, DOWN};
    const int64_t cols_of[2] = {(int64_t)m.num_q_heads * m.head_dim, m.intermediate};
    for (int c = 0; c < 2; ++c) {
        const int64_t w_old = cols_of[c] / a * e, w_new = cols_of[c] / b * e;
        out->w_old[c] = w_old;
        out->w_new[c] = w_new;
        // the lead kernel takes rows [0, N^k): the largest such range of at most kLeadBytes kept bytes
        int64_t lead = 1;
        while (lead < hid && lead * N * w_new <= kLeadBytes) lead *= N;
        lead = std::min(lead, hid);
        out->lead_rows[c] = (int32_t)lead;
        for (int r = 0; r < a; ++r) out->bytes_per_layer += (lead - (keep[r] == 0 ? 1 : 0)) * w_new;
        int64_t lo = lead, hi = lead * N;
        for (size_t wave = 0; lo < hid; ++wave) {
            for (int r = 0; r < a; ++r) {
                amoeba_weight_desc d{};
                d.src_rank = d.dst_rank = r;
                d.src_tensor = d.dst_tensor = col_tensors[c];
                d.row_bytes = w_new;
                d.n_rows = (int32_t)(std::min(hi, hid) - lo);
                d.src_off = lo * w_old + keep[r] * w_new;
                d.dst_off = lo * w_new;
                d.src_pitch = w_old;
                d.dst_pitch = w_new;
                phase(wave).push_back(d);
                out->bytes_per_layer += d.row_bytes * d.n_rows;
            }
            lo = hi;
            hi *= N;
        }
    }
}

static amoeba_status compact_check(const amoeba_plan* plan, const int32_t* keep) {
    if (!plan || !keep) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_layout &sl = plan->src, &dl = plan->dst;
    if (dl.tp % sl.tp || sl.weight_pad_parts || dl.weight_pad_parts || sl.fused_qkv != dl.fused_qkv ||
        sl.fused_gate_up != dl.fused_gate_up)
        return AMOEBA_ERR_UNSUPPORTED;
    for (int r = 0; r < sl.tp; ++r)
        if (keep[r] < 0 || keep[r] >= dl.tp / sl.tp) return AMOEBA_ERR_INVALID_ARG;
    return AMOEBA_OK;
}

}  // namespace amoeba

static amoeba_status compact_weights_inplace(const amoeba_plan* plan, const amoeba_layer_weights* bufs,
                                             const int32_t* keep, int32_t layer_begin, int32_t layer_end,
                                             int32_t* d_status, void* cuda_stream) {
    if (!bufs || !d_status) return AMOEBA_ERR_INVALID_ARG;
    amoeba_status st = compact_check(plan, keep);
    if (st != AMOEBA_OK) return st;
    const amoeba_layout& sl = plan->src;
    const int L = sl.model.num_layers, a = sl.tp, N = plan->dst.tp / a;
    if (layer_begin < 0 || layer_end > L || layer_begin > layer_end) return AMOEBA_ERR_INVALID_ARG;
    if (N == 1 || layer_begin == layer_end) return AMOEBA_OK;
    // every buffer that is touched must be there and aligned
    int buffer_of[kNumTensors] = {Q, K, V, O, GATE, UP, DOWN};
    if (sl.fused_qkv) buffer_of[K] = buffer_of[V] = Q;
    if (sl.fused_gate_up) buffer_of[UP] = GATE;
    for (int l = layer_begin; l < layer_end; ++l)
        for (int r = 0; r < a; ++r)
            for (int t = 0; t < kNumTensors; ++t) {
                const void* ptr = slots(&bufs[(size_t)r * L + l])[buffer_of[t]];
                if (!ptr) return AMOEBA_ERR_INVALID_ARG;
                if (reinterpret_cast<uintptr_t>(ptr) % 16) return AMOEBA_ERR_ALIGNMENT;
            }
    CompactSchedule sch;
    compact_schedule(plan, keep, &sch);
    for (int c = 0; c < 2; ++c)
        if (sch.w_old[c] % 16 || sch.w_new[c] % 16) return AMOEBA_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // ---- leading waves of the column tensors: one CTA per (layer, worker, tensor) buffer
    {
        LeadParams lp;
        lp.n = N;
        for (int c = 0; c < 2; ++c) {
            lp.w_old[c] = sch.w_old[c];
            lp.w_new[c] = sch.w_new[c];
            lp.rows[c] = sch.lead_rows[c];
        }
        const int col_tensors[2] = {O, DOWN};
        int n = 0;
        auto flush = [&]() -> amoeba_status {
            if (n == 0) return AMOEBA_OK;
            w_compact_lead<<<n, kLeadThreads, 0, stream>>>(lp);
            if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
            count_launch();
            n = 0;
            return AMOEBA_OK;
        };
        for (int l = layer_begin; l < layer_end; ++l)
            for (int r = 0; r < a; ++r)
                for (int c = 0; c < 2; ++c) {
                    lp.bufs[n] = static_cast<char*>(slots(&bufs[(size_t)r * L + l])[col_tensors[c]]);
                    lp.cls[n] = (uint8_t)c;
                    lp.keep[n] = (uint8_t)keep[r];
                    if (++n == kMaxLeadBufs && (st = flush()) != AMOEBA_OK) return st;
                }
        if ((st = flush()) != AMOEBA_OK) return st;
    }

    // ---- the remaining waves and the row moves
    const int64_t cap = plan->opt.w.chunk_bytes > 0 ? plan->opt.w.chunk_bytes : kDefaultWChunk;
    for (const auto& ph : sch.phases) {
        std::vector<WDescDev> descs;
        int64_t items = 0;
        for (const amoeba_weight_desc& d : ph) {
            if (d.row_bytes % 16 || d.src_off % 16 || d.dst_off % 16 || d.src_pitch % 16 || d.dst_pitch % 16)
                return AMOEBA_ERR_ALIGNMENT;
            descs.push_back(chunk_desc(d, cap, &items));
            if (items > INT32_MAX || (int)descs.size() > kMaxWeightDescs) return AMOEBA_ERR_UNSUPPORTED;
        }
        st = launch_descs(plan, descs, (int32_t)items, bufs, a, bufs, a, L, layer_begin, layer_end, d_status, stream);
        if (st != AMOEBA_OK) return st;
    }
    return AMOEBA_OK;
}

extern "C" amoeba_status amoeba_compact_bytes(const amoeba_plan* plan, const int32_t* keep, int64_t* bytes_rw) {
    if (!bytes_rw) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_status st = compact_check(plan, keep);
    if (st != AMOEBA_OK) return st;
    try {
        CompactSchedule sch;
        if (plan->dst.tp != plan->src.tp) compact_schedule(plan, keep, &sch);
        *bytes_rw = 2 * sch.bytes_per_layer * plan->src.model.num_layers;
    } catch (...) {
        return AMOEBA_ERR_NO_MEMORY;
    }
    return AMOEBA_OK;
}

// The phase lists are host containers: an allocation failure becomes a status, no exception leaves the library.
extern "C" amoeba_status amoeba_compact_weights_inplace(const amoeba_plan* plan, const amoeba_layer_weights* bufs,
                                                        const int32_t* keep, int32_t layer_begin, int32_t layer_end,
                                                        int32_t* d_status, void* cuda_stream) {
    try {
        return compact_weights_inplace(plan, bufs, keep, layer_begin, layer_end, d_status, cuda_stream);
    } catch (...) {
        return AMOEBA_ERR_NO_MEMORY;
    }
}
