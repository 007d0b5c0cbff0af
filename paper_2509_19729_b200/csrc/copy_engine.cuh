// Device-side copy machinery shared by the KV and weight re-layout kernels (sm_100a).
//
// A work item is a small 2-D copy: n_rows runs of row_bytes bytes, run i read at src + i*src_pitch and written at
// dst + i*dst_pitch (n_rows == 1 is a plain contiguous chunk).  All addresses, pitches and row_bytes are
// multiples of 16 bytes.  Two ways to move an item:
//   * cta_copy_item:    every thread of the CTA moves 16-byte vectors, all loads of an unrolled batch issued
//                       before the first store, streaming cache hints;
//   * WarpBulkRing:     one warp drives a ring of shared-memory stages with the bulk-copy engine (TMA, 1-D
//                       cp.async.bulk, no multicast): global -> shared completes on an mbarrier, shared -> global is
//                       tracked by the issuing thread's bulk groups.  Every wait is bounded.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace amoeba {

struct Item {
    const char* src;
    char* dst;
    int64_t src_pitch, dst_pitch;
    int32_t n_rows, row_bytes;
};

// ------------------------------------------------------------------ vector load/store path
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

template <int UNROLL>
__device__ __forceinline__ void copy_vecs(const uint4* __restrict__ s, uint4* __restrict__ d, int n, int tid,
                                          int nthreads) {
    for (int base = 0; base < n; base += nthreads * UNROLL) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int i = base + u * nthreads + tid;
            if (i < n) v[u] = ld_stream(s + i);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int i = base + u * nthreads + tid;
            if (i < n) st_stream(d + i, v[u]);
        }
    }
}

// All threads of the CTA call this with the same item.
template <int UNROLL>
__device__ __forceinline__ void cta_copy_item(const Item& it) {
    if (it.n_rows == 1) {
        copy_vecs<UNROLL>(reinterpret_cast<const uint4*>(it.src), reinterpret_cast<uint4*>(it.dst), it.row_bytes >> 4,
                          threadIdx.x, blockDim.x);
    } else {  // one warp per row, lanes along the row
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
        for (int r = warp; r < it.n_rows; r += nwarps)
            copy_vecs<UNROLL>(reinterpret_cast<const uint4*>(it.src + r * it.src_pitch),
                              reinterpret_cast<uint4*>(it.dst + r * it.dst_pitch), it.row_bytes >> 4, lane, 32);
    }
}

// ------------------------------------------------------------------ bulk-copy (TMA) path
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the try budget.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t max_tries = (1u << 22)) {
    for (uint32_t i = 0; i < max_tries; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// One warp's ring of NS shared-memory stages.  Loads run LAG items ahead of stores, so up to LAG loads and
// NS - LAG stores are in flight per warp.  `item_of(w)` must return the same Item in every lane.
// Returns false if a bounded wait ran out (the caller records AMOEBA_ERR_TIMEOUT).
template <int NS, int LAG, class ItemFn>
__device__ __forceinline__ bool warp_bulk_ring(ItemFn item_of, int64_t n_items, int64_t first, int64_t stride,
                                               char* stages, int stage_bytes, uint64_t* bars) {
    static_assert(LAG >= 1 && LAG < NS, "loads must lead stores by 1..NS-1 stages");
    const int lane = threadIdx.x & 31;
    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(&bars[s], 1);
        fence_async_smem();
    }
    __syncwarp();
    const int64_t n_local = n_items > first ? (n_items - first + stride - 1) / stride : 0;
    bool ok = true;
    int64_t loads_issued = 0, loads_waited = 0;
    for (int64_t k = 0; k < n_local + LAG && ok; ++k) {
        if (k < n_local) {
            const int s = (int)(k % NS);
            if (k >= NS) bulk_wait_read<NS - LAG - 1>();  // this lane's stores out of stage s have read it
            __syncwarp();                                 // ... and so have every other lane's
            const Item it = item_of(first + k * stride);
            if (lane == 0) mbar_arrive_expect_tx(&bars[s], (uint32_t)it.n_rows * (uint32_t)it.row_bytes);
            __syncwarp();
            char* st = stages + (int64_t)s * stage_bytes;
            for (int r = lane; r < it.n_rows; r += 32)
                bulk_g2s(st + (int64_t)r * it.row_bytes, it.src + r * it.src_pitch, it.row_bytes, &bars[s]);
            ++loads_issued;
        }
        const int64_t j = k - LAG;
        if (j >= 0) {
            const int s = (int)(j % NS);
            ok = mbar_wait_bounded(&bars[s], (uint32_t)((j / NS) & 1));
            ok = __all_sync(0xffffffffu, ok);
            ++loads_waited;
            if (ok) {
                const Item it = item_of(first + j * stride);
                const char* st = stages + (int64_t)s * stage_bytes;
                for (int r = lane; r < it.n_rows; r += 32)
                    bulk_s2g(it.dst + r * it.dst_pitch, st + (int64_t)r * it.row_bytes, it.row_bytes);
            }
            bulk_commit();
        }
    }
    bulk_wait_all();  // this lane's stores are complete and visible
    if (!ok) {        // give the loads still in flight a bounded chance to land before the CTA's smem goes away
        for (int64_t j = loads_waited; j < loads_issued; ++j)
            mbar_wait_bounded(&bars[j % NS], (uint32_t)((j / NS) & 1), 1u << 16);
    }
    __syncwarp();
    return ok;
}

}  // namespace amoeba
