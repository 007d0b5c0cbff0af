// Device-side copy machinery shared by the KV and weight re-layout kernels (sm_100a).
//
// A work item is a small 2-D copy: n_rows runs of row_bytes bytes, run i read at src + i*src_pitch and written at
// dst + i*dst_pitch (n_rows == 1 is a plain contiguous chunk).  All addresses, pitches and row_bytes are
// multiples of 16 bytes.  Three ways to move items:
//   * warp_copy_item     a warp moves an item with 16-byte vector loads / stores, all loads of an unrolled batch
//                        issued before the first store, streaming cache hints;
//   * warp_bulk_ring     each warp drives its own ring of shared-memory stages with the bulk-copy engine (TMA, 1-D
//                        cp.async.bulk, one CTA, no cluster): global -> shared completes on an mbarrier, shared -> global is
//                        tracked by the issuing thread's bulk groups; loads lead stores by a fixed lag;
//   * pair_bulk_ring     a producer warp and a consumer warp share one ring: the producer only issues loads (waits
//                        on "empty" barriers), the consumer only issues stores (waits on "full" barriers), so the
//                        split of the ring between loads and stores in flight adapts by itself.
// In the ring kernels a side of an item may also be one box of a tensor map (tiled TMA), which gathers or scatters
// many short rows with a single copy instruction.
// Every wait on an mbarrier is bounded; bulk-group waits only wait for the thread's own stores.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace amoeba {

struct Item {
    const char* src;
    char* dst;
    int64_t src_pitch, dst_pitch;
    int32_t n_rows, row_bytes;
    // Bulk-copy rings only: when non-null, that side of the item is one box of a 5-D tensor map instead of rows
    // (coordinates {0, tok, 0, head, layer}); the box holds exactly n_rows * row_bytes bytes and arrives in / leaves
    // shared memory in the same dense order as the packed rows.
    const void* src_map;
    const void* dst_map;
    int32_t src_tok, src_head, dst_tok, dst_head, layer;
};

// Shape of the bulk rings (runtime, chosen by the launcher).
struct RingShape {
    int32_t stages;       // stages per ring
    int32_t lag;          // warp ring: loads lead stores by this many items; pair ring: stores kept in flight
    int32_t stage_bytes;  // bytes per stage
    int32_t hint;         // bit 0: loads evict-first in L2, bit 1: stores evict-first in L2
    int32_t max_polls;    // 0: default wait budget; v > 0: every mbarrier wait gives up after v - 1 non-blocking polls
};

// Checked build (-DAMOEBA_CHECK_ITEMS): every work item is tested against the extent of the buffers it addresses
// before it is moved; an item that would reach outside sets AMOEBA_ERR_INTERNAL in the status word and is skipped.
// True if n_rows rows of row_bytes, the first at byte `off` of a buffer and consecutive ones `pitch` apart, lie inside
// [0, size).
__device__ __forceinline__ bool rows_inside(int64_t off, int64_t pitch, int32_t n_rows, int32_t row_bytes, int64_t size) {
    if (n_rows <= 0) return true;
    const int64_t last = off + (int64_t)(n_rows - 1) * pitch;
    const int64_t lo = pitch >= 0 ? off : last, hi = (pitch >= 0 ? last : off) + row_bytes;
    return lo >= 0 && hi <= size;
}

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

// All lanes of a warp call this with the same item: the warp alone moves it, UNROLL 16-byte loads in flight per lane
// before the first store.  Rows that are not adjacent in memory are dealt to the lanes vector by vector across rows.
template <int UNROLL>
__device__ __forceinline__ void warp_copy_rows(const char* __restrict__ src, char* __restrict__ dst, int64_t src_pitch,
                                               int64_t dst_pitch, int n_rows, int row_bytes) {
    const int lane = threadIdx.x & 31;
    if (n_rows == 1 || (src_pitch == row_bytes && dst_pitch == row_bytes)) {
        copy_vecs<UNROLL>(reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), (n_rows * row_bytes) >> 4,
                          lane, 32);
        return;
    }
    const int vpr = row_bytes >> 4, n = n_rows * vpr;
    for (int base = 0; base < n; base += 32 * UNROLL) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int i = base + u * 32 + lane;
            if (i < n) {
                const int r = i / vpr, c = i - r * vpr;
                v[u] = ld_stream(reinterpret_cast<const uint4*>(src + r * src_pitch) + c);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int i = base + u * 32 + lane;
            if (i < n) {
                const int r = i / vpr, c = i - r * vpr;
                st_stream(reinterpret_cast<uint4*>(dst + r * dst_pitch) + c, v[u]);
            }
        }
    }
}
template <int UNROLL>
__device__ __forceinline__ void warp_copy_item(const Item& it) {
    warp_copy_rows<UNROLL>(it.src, it.dst, it.src_pitch, it.dst_pitch, it.n_rows, it.row_bytes);
}

// ------------------------------------------------------------------ bulk-copy (TMA) primitives
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
constexpr uint32_t kDefaultWaitTries = 1u << 22;
constexpr uint32_t kDrainWaitTries = 1u << 16;
// Bounded wait: false if the phase did not complete within the budget, or if *abort became non-zero meanwhile (the
// other warp of the ring gave up).  max_polls == 0: the default budget of potentially-suspending try_wait calls;
// max_polls = v > 0: a caller-chosen, short limit of v - 1 non-blocking polls (v = 1: give up at once, which makes
// the give-up path run on healthy copies, deterministically).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t max_polls = 0,
                                                  const volatile int32_t* abort = nullptr) {
    if (max_polls) {
        for (uint32_t i = 1; i < max_polls; ++i)
            if (mbar_test_wait(bar, parity)) return true;
        return false;
    }
    for (uint32_t i = 0; i < kDefaultWaitTries; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (abort && (i & 15) == 15 && *abort) return false;
    }
    return false;
}
// Give copies that are still in flight a bounded chance to land: waits for the phase, never reports.
__device__ __forceinline__ void mbar_drain(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kDrainWaitTries; ++i)
        if (mbar_try_wait(bar, parity)) return;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar, bool hint,
                                         uint64_t policy) {
    if (hint)
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                smem_u32(smem_dst)),
            "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
            : "memory");
    else
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         smem_u32(smem_dst)),
                     "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                     : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* gdst, const void* smem_src, uint32_t bytes, bool hint, uint64_t policy) {
    if (hint)
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(gdst),
                     "r"(smem_u32(smem_src)), "r"(bytes), "l"(policy)
                     : "memory");
    else
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                     "r"(smem_u32(smem_src)), "r"(bytes)
                     : "memory");
}
// Tiled (tensor-map) copies of one 5-D box; the innermost coordinate is always 0, so the 16-byte rule on it holds.
__device__ __forceinline__ void tensor_g2s(void* smem_dst, const void* map, int32_t c1, int32_t c3, int32_t c4,
                                           uint64_t* bar, bool hint, uint64_t policy) {
    if (hint)
        asm volatile(
            "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
            "[%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;" ::"r"(smem_u32(smem_dst)),
            "l"(map), "r"(0), "r"(c1), "r"(0), "r"(c3), "r"(c4), "r"(smem_u32(bar)), "l"(policy)
            : "memory");
    else
        asm volatile(
            "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
            "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(smem_u32(smem_dst)),
            "l"(map), "r"(0), "r"(c1), "r"(0), "r"(c3), "r"(c4), "r"(smem_u32(bar))
            : "memory");
}
__device__ __forceinline__ void tensor_s2g(const void* map, int32_t c1, int32_t c3, int32_t c4, const void* smem_src,
                                           bool hint, uint64_t policy) {
    if (hint)
        asm volatile(
            "cp.async.bulk.tensor.5d.global.shared::cta.tile.bulk_group.L2::cache_hint "
            "[%0, {%1, %2, %3, %4, %5}], [%6], %7;" ::"l"(map),
            "r"(0), "r"(c1), "r"(0), "r"(c3), "r"(c4), "r"(smem_u32(smem_src)), "l"(policy)
            : "memory");
    else
        asm volatile(
            "cp.async.bulk.tensor.5d.global.shared::cta.tile.bulk_group "
            "[%0, {%1, %2, %3, %4, %5}], [%6];" ::"l"(map),
            "r"(0), "r"(c1), "r"(0), "r"(c3), "r"(c4), "r"(smem_u32(smem_src))
            : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until at most n of this thread's bulk groups still have shared-memory reads outstanding (n in 0..15).
__device__ __forceinline__ void bulk_wait_read(int n) {
    switch (n) {
        case 0: asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.bulk.wait_group.read 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.bulk.wait_group.read 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.bulk.wait_group.read 6;" ::: "memory"); break;
        case 7: asm volatile("cp.async.bulk.wait_group.read 7;" ::: "memory"); break;
        case 8: asm volatile("cp.async.bulk.wait_group.read 8;" ::: "memory"); break;
        case 9: asm volatile("cp.async.bulk.wait_group.read 9;" ::: "memory"); break;
        case 10: asm volatile("cp.async.bulk.wait_group.read 10;" ::: "memory"); break;
        case 11: asm volatile("cp.async.bulk.wait_group.read 11;" ::: "memory"); break;
        case 12: asm volatile("cp.async.bulk.wait_group.read 12;" ::: "memory"); break;
        case 13: asm volatile("cp.async.bulk.wait_group.read 13;" ::: "memory"); break;
        case 14: asm volatile("cp.async.bulk.wait_group.read 14;" ::: "memory"); break;
        default: asm volatile("cp.async.bulk.wait_group.read 15;" ::: "memory"); break;
    }
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

constexpr int kMaxStages = 16;
// Head of a ring kernel's dynamic shared memory: mbarriers, then one abort word per producer/consumer ring.
constexpr int kBarrierBytes = 1024;
constexpr int kBarrierSlots = 112;                 // 8-byte mbarriers
constexpr int kAbortOffset = kBarrierSlots * 8;    // 32 int32 abort words behind them

// One item between global memory and a shared-memory stage (rows packed densely in the stage).  A side whose rows
// are adjacent in global memory (pitch == row_bytes, or a single row) moves as ONE bulk copy issued by lane 0;
// otherwise lane r moves row r, r + 32, ...  All lanes of the warp call these with the same item.
__device__ __forceinline__ void item_load(const Item& it, char* stage, uint64_t* bar, bool hint, uint64_t policy) {
    const int lane = threadIdx.x & 31;
    if (it.n_rows == 0) return;  // skipped item: the barrier phase completes with 0 bytes expected
    if (it.src_map) {
        if (lane == 0) tensor_g2s(stage, it.src_map, it.src_tok, it.src_head, it.layer, bar, hint, policy);
    } else if (it.n_rows == 1 || it.src_pitch == it.row_bytes) {
        if (lane == 0) bulk_g2s(stage, it.src, (uint32_t)it.n_rows * (uint32_t)it.row_bytes, bar, hint, policy);
    } else {
        for (int r = lane; r < it.n_rows; r += 32)
            bulk_g2s(stage + (int64_t)r * it.row_bytes, it.src + r * it.src_pitch, it.row_bytes, bar, hint, policy);
    }
}
__device__ __forceinline__ void item_store(const Item& it, const char* stage, bool hint, uint64_t policy) {
    const int lane = threadIdx.x & 31;
    if (it.n_rows == 0) return;
    if (it.dst_map) {
        if (lane == 0) tensor_s2g(it.dst_map, it.dst_tok, it.dst_head, it.layer, stage, hint, policy);
    } else if (it.n_rows == 1 || it.dst_pitch == it.row_bytes) {
        if (lane == 0) bulk_s2g(it.dst, stage, (uint32_t)it.n_rows * (uint32_t)it.row_bytes, hint, policy);
    } else {
        for (int r = lane; r < it.n_rows; r += 32)
            bulk_s2g(it.dst + r * it.dst_pitch, stage + (int64_t)r * it.row_bytes, it.row_bytes, hint, policy);
    }
}

// ------------------------------------------------------------------ one ring per warp
// Loads run `lag` items ahead of stores, so up to `lag` loads and `stages - lag` stores are in flight per warp.
// `item_of(w)` must return the same Item in every lane.  bars: `stages` mbarriers of this warp.
// Returns false if a bounded wait ran out (the caller records AMOEBA_ERR_TIMEOUT).
template <class ItemFn>
__device__ __forceinline__ bool warp_bulk_ring(ItemFn item_of, int64_t n_items, int64_t first, int64_t stride,
                                               char* stages, uint64_t* bars, const RingShape rs) {
    const int lane = threadIdx.x & 31;
    const int NS = rs.stages, LAG = rs.lag;
    const bool hl = rs.hint & 1, hs = rs.hint & 2;
    const uint64_t policy = policy_evict_first();
    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(&bars[s], 1);
        fence_async_smem();
    }
    __syncwarp();
    const int64_t n_local = n_items > first ? (n_items - first + stride - 1) / stride : 0;
    bool ok = true;
    int64_t loads_issued = 0, loads_waited = 0;
    int s_load = 0, s_store = 0;       // ring slots of the next load / next store
    uint32_t store_parity = 0;         // phase parity of the slot the next store waits on
    for (int64_t k = 0; k < n_local + LAG && ok; ++k) {
        if (k < n_local) {
            if (k >= NS) bulk_wait_read(NS - LAG - 1);  // this lane's stores out of this slot have read it
            __syncwarp();                               // ... and so have every other lane's
            const Item it = item_of(first + k * stride);
            if (lane == 0) mbar_arrive_expect_tx(&bars[s_load], (uint32_t)it.n_rows * (uint32_t)it.row_bytes);
            __syncwarp();
            item_load(it, stages + (int64_t)s_load * rs.stage_bytes, &bars[s_load], hl, policy);
            ++loads_issued;
            if (++s_load == NS) s_load = 0;
        }
        if (k >= LAG) {
            ok = mbar_wait_bounded(&bars[s_store], store_parity, (uint32_t)rs.max_polls);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                ++loads_waited;
                const Item it = item_of(first + (k - LAG) * stride);
                item_store(it, stages + (int64_t)s_store * rs.stage_bytes, hs, policy);
            }
            bulk_commit();
            if (++s_store == NS) {
                s_store = 0;
                store_parity ^= 1;
            }
        }
    }
    bulk_wait_all();  // this lane's stores are complete
    if (!ok) {        // give the loads still in flight a bounded chance to land before the CTA's smem goes away
        for (int64_t j = loads_waited; j < loads_issued; ++j) mbar_drain(&bars[j % NS], (uint32_t)((j / NS) & 1));
    }
    __syncwarp();
    return ok;
}

// ------------------------------------------------------------------ producer warp + consumer warp on one ring
// `role` 0 = producer (loads), 1 = consumer (stores).  full/empty: `stages` mbarriers each, and the ring's abort
// word, initialised by pair_ring_init before both warps start.  rs.lag = number of store groups the consumer keeps
// in flight before it hands a slot back.
// Giving up: a warp whose bounded wait runs out raises the ring's abort word and leaves; the other warp sees the word
// (at its next item, or while it polls) and leaves too.  Before the CTA may exit, the consumer has waited for its own
// stores, and the producer has waited - bounded again - for every load it armed, so that no copy of this ring is still
// writing into the CTA's shared memory.  Both return false.
__device__ __forceinline__ void pair_ring_init(uint64_t* full, uint64_t* empty, int32_t* abort, int stages) {
    for (int s = 0; s < stages; ++s) {
        mbar_init(&full[s], 1);
        mbar_init(&empty[s], 1);
    }
    *abort = 0;
    fence_async_smem();
}

template <class ItemFn>
__device__ __forceinline__ bool pair_bulk_ring(int role, ItemFn item_of, int64_t n_items, int64_t first,
                                               int64_t stride, char* stages, uint64_t* full, uint64_t* empty,
                                               int32_t* abort_word, const RingShape rs) {
    const int lane = threadIdx.x & 31;
    const int NS = rs.stages, D = rs.lag;
    const uint32_t polls = (uint32_t)rs.max_polls;
    volatile int32_t* abort = abort_word;
    const uint64_t policy = policy_evict_first();
    const int64_t n_local = n_items > first ? (n_items - first + stride - 1) / stride : 0;
    bool ok = true;
    int slot = 0;
    uint32_t parity = 0;
    if (role == 0) {
        const bool hl = rs.hint & 1;
        int64_t armed = 0;  // "full" phases armed so far
        for (int64_t k = 0; k < n_local; ++k) {
            if (*abort) ok = false;
            if (ok && k >= NS)  // wait until the consumer has handed this slot back (its previous use)
                ok = mbar_wait_bounded(&empty[slot], parity ^ 1, polls, abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const Item it = item_of(first + k * stride);
            if (lane == 0) mbar_arrive_expect_tx(&full[slot], (uint32_t)it.n_rows * (uint32_t)it.row_bytes);
            __syncwarp();
            item_load(it, stages + (int64_t)slot * rs.stage_bytes, &full[slot], hl, policy);
            ++armed;
            if (++slot == NS) {
                slot = 0;
                parity ^= 1;
            }
        }
        if (!ok) {
            if (lane == 0) *abort = 1;
            // the last min(NS, armed) uses of the ring may still have loads in flight
            for (int64_t j = armed > NS ? armed - NS : 0; j < armed; ++j)
                mbar_drain(&full[j % NS], (uint32_t)((j / NS) & 1));
        }
    } else {
        const bool hs = rs.hint & 2;
        int release = 0;  // slot of the oldest store not yet handed back
        for (int64_t k = 0; k < n_local; ++k) {
            if (*abort) ok = false;
            if (ok) ok = mbar_wait_bounded(&full[slot], parity, polls, abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const Item it = item_of(first + k * stride);
            item_store(it, stages + (int64_t)slot * rs.stage_bytes, hs, policy);
            bulk_commit();
            if (k >= D) {  // the store issued D items ago has read its slot: hand it back
                bulk_wait_read(D);
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[release]);
                if (++release == NS) release = 0;
            }
            if (++slot == NS) {
                slot = 0;
                parity ^= 1;
            }
        }
        if (!ok && lane == 0) *abort = 1;
        bulk_wait_all();
    }
    __syncwarp();
    return ok;
}

// The calling warp's place in a CTA of producer/consumer rings: warps 2r and 2r+1 are the producer and the consumer of
// ring r.  Initialises the ring's barriers and ends with a CTA-wide barrier: call it from every thread.
struct PairRing {
    uint64_t *full, *empty;
    int32_t* abort;
    char* stages;
    int ring, role, nrings;
};
__device__ __forceinline__ PairRing pair_ring_setup(char* smem, const RingShape& rs) {
    PairRing r;
    const int warp = threadIdx.x >> 5;
    r.ring = warp >> 1;
    r.role = warp & 1;
    r.nrings = blockDim.x >> 6;
    r.full = reinterpret_cast<uint64_t*>(smem) + r.ring * 2 * rs.stages;
    r.empty = r.full + rs.stages;
    r.abort = reinterpret_cast<int32_t*>(smem + kAbortOffset) + r.ring;
    r.stages = smem + kBarrierBytes + (int64_t)r.ring * rs.stages * rs.stage_bytes;
    if (r.role == 0 && (threadIdx.x & 31) == 0) pair_ring_init(r.full, r.empty, r.abort, rs.stages);
    __syncthreads();
    return r;
}

}  // namespace amoeba
