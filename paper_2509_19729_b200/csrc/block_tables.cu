// Destination block bookkeeping for the KV migration (Sec. 3.1: each worker prepares reserved pages for the KV it
// receives), and the block tables of the in-place block reshaping of one instance (Sec. 3.1, Improvement 1).
// No CTA ever waits on another.  Phases:
//   scan   (1 CTA)  blocks per sequence and their exclusive prefix sum; when the free blocks come as a byte mask,
//                   their compaction into an ascending id list (16 mask bytes per thread, popc + CTA prefix sum);
//                   the whole-call errors.
//   claim  (grid)   only when destination ids can repeat (a free LIST, or ids derived from the source table): the
//                   first user of every destination id in (sequence, block) order, by atomicMin.
//   rank   (1 CTA)  only for the pair list in destination order: the number of given destination ids below every id
//                   (prefix sum over the ids), i.e. where the pair of the block that was given the id goes.
//   assign (grid)   one warp per 128-entry segment of a block-table row: the k-th block overall takes the k-th free
//                   id (or the reshaped id of its source block); writes the destination table (with -1 padding) and
//                   the (source, destination) pair list; an id whose first user is another block is refused.
// Small tables run all phases in one launch of one CTA; larger ones as separate launches, each of which starts when
// the one before it has completed.
#include <cuda_runtime.h>

#include <climits>
#include <mutex>

#include "launch.hpp"
#include "plan.hpp"

namespace amoeba {

struct BtHeader {  // first 64 bytes of the workspace
    int32_t total;   // blocks assigned by this call (0 on a whole-call error)
    int32_t n_free;  // free destination blocks before the call
    int32_t err;     // whole-call error code or 0
    int32_t n_given; // destination order: blocks that were given a destination id (the others' pairs go to the tail)
    int32_t pad[12];
};

struct BtArgs {
    const int32_t* src_bt;
    const int32_t* seq_lens;
    const int32_t* free_list;  // list form, or null
    const uint8_t* free_mask;  // mask form, or null
    BtHeader* hdr;
    int32_t* seq_off;     // [num_seqs] exclusive prefix sum of the blocks per sequence
    int32_t* area;        // mask form: compacted ascending free ids; otherwise: first user of every destination id
    int32_t* rank;        // destination order (not mask form): number of given destination ids below every id
    int32_t* dst_bt;
    int2* pairs;
    int32_t* num_pairs;
    int32_t* free_count_out;
    int32_t* status;
    uint8_t* free_mask_out;  // reshaping only: 1 = free id of the destination side
    int32_t num_seqs, block_tokens, maxb, n_free_or_nb, pairs_cap, nb_src, nb_dst;
    int32_t reshape;  // 0: ids from the free list / mask; +N: destination id = source id * N; -N: source id / N
    int32_t dst_order;  // 1: pair list ascending by destination id (a mask hands ids out in that order anyway)
};

constexpr int kScanThreads = 1024;
constexpr int kSegment = 128;  // table entries one warp handles per step

// Exclusive scan of one value per thread across the CTA; returns the thread's offset, *total = CTA sum.
__device__ __forceinline__ int32_t cta_exclusive_scan(int32_t v, int32_t* warp_sums, int32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int32_t t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int32_t w = warp_sums[lane];  // kScanThreads / 32 == 32 warps
        int32_t wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int32_t t = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += t;
        }
        warp_sums[lane] = wi - w;                // exclusive warp offsets
        if (lane == 31) warp_sums[32] = wi;      // CTA total
    }
    __syncthreads();
    const int32_t off = warp_sums[warp] + incl - v;
    *total = warp_sums[32];
    __syncthreads();  // warp_sums may be reused by the caller's next round
    return off;
}

__device__ __forceinline__ int32_t blocks_needed(int32_t len, int32_t block_tokens) {
    return (int32_t)(((int64_t)len + block_tokens - 1) / block_tokens);
}

// Destination id of the k-th block overall, whose source id is `src`; -1 if there is none.
__device__ __forceinline__ int32_t dst_id_of(const BtArgs& a, int32_t k, int32_t src) {
    if (a.reshape == 0) return a.free_mask ? a.area[k] : a.free_list[k];
    if (src < 0 || src >= a.nb_src) return -1;
    if (a.reshape > 0) return (int32_t)min((int64_t)src * a.reshape, (int64_t)INT32_MAX);
    const int32_t n = -a.reshape;
    return src % n == 0 ? src / n : -1;
}

// Bit j set = byte j of the word is non-zero.
__device__ __forceinline__ uint32_t nonzero_bytes(uint32_t w) {
    return (w & 0xffu ? 1u : 0u) | (w & 0xff00u ? 2u : 0u) | (w & 0xff0000u ? 4u : 0u) | (w & 0xff000000u ? 8u : 0u);
}

// All kScanThreads threads of ONE CTA.
__device__ void scan_phase(const BtArgs& a, int32_t* warp_sums, int32_t* flags) {
    const int tid = threadIdx.x;
    if (tid == 0) flags[0] = 0;  // a negative or too long sequence was seen
    __syncthreads();

    // ---- blocks per sequence and their exclusive prefix sum
    int64_t carry = 0;
    for (int32_t base = 0; base < a.num_seqs; base += kScanThreads) {
        const int32_t s = base + tid;
        int32_t nb = 0;
        if (s < a.num_seqs) {
            const int32_t len = a.seq_lens[s];
            const int64_t need = ((int64_t)len + a.block_tokens - 1) / a.block_tokens;
            if (len < 0 || need > a.maxb) flags[0] = 1;
            else nb = (int32_t)need;
        }
        int32_t tile_total;
        const int32_t off = cta_exclusive_scan(nb, warp_sums, &tile_total);
        if (s < a.num_seqs) a.seq_off[s] = (int32_t)min(carry + off, (int64_t)INT32_MAX);
        carry += tile_total;
    }
    const int64_t total = carry;

    // ---- ordered free list from the mask: ascending ids of the non-zero bytes, 16 mask bytes per thread
    int64_t n_free = a.reshape ? a.nb_dst : a.n_free_or_nb;
    if (a.free_mask) {
        const bool vec_ok = (reinterpret_cast<uintptr_t>(a.free_mask) & 15) == 0;
        int32_t found = 0;
        for (int32_t base = 0; base < a.n_free_or_nb; base += kScanThreads * 16) {
            const int32_t i0 = base + tid * 16;
            uint32_t bits = 0;
            if (vec_ok && i0 + 16 <= a.n_free_or_nb) {
                const uint4 v = *reinterpret_cast<const uint4*>(a.free_mask + i0);
                bits = nonzero_bytes(v.x) | nonzero_bytes(v.y) << 4 | nonzero_bytes(v.z) << 8 | nonzero_bytes(v.w) << 12;
            } else {
                for (int j = 0; j < 16; ++j)
                    if (i0 + j < a.n_free_or_nb && a.free_mask[i0 + j]) bits |= 1u << j;
            }
            int32_t tile_total;
            int32_t pos = found + cta_exclusive_scan(__popc(bits), warp_sums, &tile_total);
            while (bits) {
                const int j = __ffs(bits) - 1;
                bits &= bits - 1;
                a.area[pos++] = i0 + j;
            }
            found += tile_total;
        }
        n_free = found;
    }

    __syncthreads();
    if (tid == 0) {
        int32_t err = 0;
        if (flags[0]) err = AMOEBA_ERR_INVALID_ARG;
        else if (total > a.pairs_cap) err = AMOEBA_ERR_INVALID_ARG;
        else if (!a.reshape && total > n_free) err = AMOEBA_ERR_NO_FREE_BLOCKS;
        const int32_t assigned = err ? 0 : (int32_t)total;
        a.hdr->total = assigned;
        a.hdr->n_free = (int32_t)n_free;
        a.hdr->err = err;
        a.hdr->n_given = 0;
        *a.num_pairs = assigned;
        *a.free_count_out = (int32_t)n_free - assigned;
        if (err) atomicCAS(a.status, 0, err);
    }
    __syncthreads();

    // ---- nobody holds a destination id yet (ids from a list or from the source table may repeat)
    if (!a.free_mask)
        for (int32_t q = tid; q < a.nb_dst; q += kScanThreads) a.area[q] = INT32_MAX;
}

// First user of every destination id in (sequence, block) order, by atomicMin over the k of the blocks that are
// given it.  Any number of threads; thread `t` of `n`.  Runs after scan_phase has completed.
__device__ void claim_phase(const BtArgs& a, int64_t t, int64_t n) {
    if (a.free_mask || a.hdr->err) return;
    if (a.reshape == 0) {  // the k-th block is given the k-th list entry, whatever its source id
        const int32_t total = a.hdr->total;
        for (int64_t k = t; k < total; k += n) {
            const int32_t d = a.free_list[k];
            if (d >= 0 && d < a.nb_dst) atomicMin(a.area + d, (int32_t)k);
        }
        return;
    }
    const int64_t entries = (int64_t)a.num_seqs * a.maxb;
    for (int64_t e = t; e < entries; e += n) {
        const int32_t s = (int32_t)(e / a.maxb), i = (int32_t)(e - (int64_t)s * a.maxb);
        if (i >= blocks_needed(a.seq_lens[s], a.block_tokens)) continue;
        const int32_t k = a.seq_off[s] + i;
        const int32_t d = dst_id_of(a, k, a.src_bt[e]);
        if (d >= 0 && d < a.nb_dst) atomicMin(a.area + d, k);
    }
}

// Pair list in destination order: rank[d] = number of destination ids below d that some block was given.  All
// kScanThreads threads of ONE CTA; runs after claim_phase has completed.  Each warp owns one contiguous run of ids
// (a whole number of 32-id rows): it counts the given ids of its run, the CTA scans the 32 counts, and the warp
// walks its run again (the flags are in L1/L2 by then) handing out ranks row by row.
__device__ void rank_phase(const BtArgs& a, int32_t* warp_sums) {
    if (!a.dst_order || a.free_mask) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kScanThreads / 32;
    const bool ok = a.hdr->err == 0;
    const int32_t rows = ok ? ((a.nb_dst + 31) / 32 + kWarps - 1) / kWarps : 0;  // 32-id rows per warp
    const int64_t first = (int64_t)warp * rows * 32;
    int32_t mine = 0;
#pragma unroll 8
    for (int32_t j = 0; j < rows; ++j) {
        const int64_t d = first + (int64_t)j * 32 + lane;
        mine += (d < a.nb_dst && a.area[d] != INT32_MAX) ? 1 : 0;
    }
    mine = __reduce_add_sync(0xffffffffu, mine);
    __syncthreads();  // warp_sums may still be read by the phase before
    if (lane == 0) warp_sums[warp] = mine;
    __syncthreads();
    int32_t before = 0, given = 0;
    for (int w = 0; w < kWarps; ++w) {
        const int32_t c = warp_sums[w];
        before += w < warp ? c : 0;
        given += c;
    }
    for (int32_t j = 0; j < rows; ++j) {
        const int64_t d = first + (int64_t)j * 32 + lane;
        const bool flag = d < a.nb_dst && a.area[d] != INT32_MAX;
        const unsigned row = __ballot_sync(0xffffffffu, flag);
        if (d < a.nb_dst) a.rank[d] = before + __popc(row & ((1u << lane) - 1u));
        before += __popc(row);
    }
    if (threadIdx.x == 0) a.hdr->n_given = given;
}

// Any number of warps; warp `warp` of `n_warps`.  Runs after claim_phase (and rank_phase) has completed (next launch,
// or after a __syncthreads() of the one CTA that ran it).
__device__ void assign_phase(const BtArgs& a, int64_t warp, int64_t n_warps) {
    const int lane = threadIdx.x & 31;
    const int32_t segs_per_row = (a.maxb + kSegment - 1) / kSegment;
    const bool call_failed = a.hdr->err != 0;
    const bool check_first = a.free_mask == nullptr;
    const bool by_rank = a.dst_order && check_first;  // where the pairs go: by destination id, refused blocks last
    bool bad = false;
    int32_t refused = 0;  // reshaping: blocks that keep no destination id
    for (int64_t unit = warp; unit < (int64_t)a.num_seqs * segs_per_row; unit += n_warps) {
        const int32_t s = (int32_t)(unit / segs_per_row);
        const int32_t col0 = (int32_t)(unit - (int64_t)s * segs_per_row) * kSegment;
        const int32_t nb = call_failed ? 0 : blocks_needed(a.seq_lens[s], a.block_tokens);
        const int32_t off = a.seq_off[s];
        for (int32_t i = col0 + lane; i < min(col0 + kSegment, a.maxb); i += 32) {
            int32_t out = -1;
            if (i < nb) {
                const int32_t k = off + i;
                const int32_t src = a.src_bt[(int64_t)s * a.maxb + i];
                const int32_t dst = dst_id_of(a, k, src);
                bool dst_ok = dst >= 0 && dst < a.nb_dst;
                if (dst_ok && check_first && a.area[dst] != k) dst_ok = false;  // an earlier block holds this id
                const bool src_ok = src >= 0 && src < a.nb_src;
                out = dst_ok ? dst : -1;
                const int2 pair = (dst_ok && src_ok) ? make_int2(src, dst) : make_int2(-1, -1);
                if (!by_rank) a.pairs[k] = pair;
                else if (dst_ok) a.pairs[a.rank[dst]] = pair;
                bad |= !(dst_ok && src_ok);
                refused += !dst_ok;
            }
            a.dst_bt[(int64_t)s * a.maxb + i] = out;
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicCAS(a.status, 0, (int)AMOEBA_ERR_BAD_BLOCK_ID);
    if (by_rank)  // the blocks that were given no destination id: their (-1,-1) pairs close the list
        for (int64_t k = a.hdr->n_given + warp * 32 + lane; k < a.hdr->total; k += n_warps * 32)
            a.pairs[k] = make_int2(-1, -1);
    if (a.reshape) {
        refused = __reduce_add_sync(0xffffffffu, refused);
        if (refused && lane == 0) atomicAdd(a.free_count_out, refused);
        for (int64_t q = warp * 32 + lane; q < a.nb_dst; q += n_warps * 32)
            a.free_mask_out[q] = (call_failed || a.area[q] == INT32_MAX) ? 1 : 0;
    }
}

__global__ void __launch_bounds__(kScanThreads) bt_scan(const __grid_constant__ BtArgs a) {
    __shared__ int32_t warp_sums[33];
    __shared__ int32_t flags[1];
    scan_phase(a, warp_sums, flags);
}

__global__ void __launch_bounds__(256) bt_claim(const __grid_constant__ BtArgs a) {
    claim_phase(a, (int64_t)blockIdx.x * blockDim.x + threadIdx.x, (int64_t)gridDim.x * blockDim.x);
}

__global__ void __launch_bounds__(kScanThreads) bt_rank(const __grid_constant__ BtArgs a) {
    __shared__ int32_t warp_sums[33];
    rank_phase(a, warp_sums);
}

__global__ void __launch_bounds__(256) bt_assign(const __grid_constant__ BtArgs a) {
    assign_phase(a, ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, ((int64_t)gridDim.x * blockDim.x) >> 5);
}

// All phases in one CTA: what the CTA wrote to global memory in a phase is visible to all its threads after the
// barrier that ends it.
__global__ void __launch_bounds__(kScanThreads) bt_fused(const __grid_constant__ BtArgs a) {
    __shared__ int32_t warp_sums[33];
    __shared__ int32_t flags[1];
    scan_phase(a, warp_sums, flags);
    __threadfence_block();
    __syncthreads();
    claim_phase(a, threadIdx.x, kScanThreads);
    __threadfence_block();
    __syncthreads();
    rank_phase(a, warp_sums);
    __threadfence_block();
    __syncthreads();
    assign_phase(a, threadIdx.x >> 5, kScanThreads / 32);
}

constexpr int64_t kFusedEntries = 8 * 1024;  // up to this many table entries (and destination ids): one launch

static int64_t align16(int64_t x) { return (x + 15) & ~int64_t(15); }

static int64_t ids_bytes(const amoeba_plan* plan) {
    return align16(4 * (int64_t)std::max(plan->src.num_blocks, plan->dst.num_blocks));
}

static int64_t tables_workspace_bytes(const amoeba_plan* plan, int32_t num_seqs) {
    return (int64_t)sizeof(BtHeader) + align16(4 * ((int64_t)num_seqs + 1)) + 2 * ids_bytes(plan);
}

static amoeba_status launch_tables(const amoeba_plan* plan, BtArgs a, void* d_workspace, cudaStream_t stream) {
    char* ws = static_cast<char*>(d_workspace);
    a.hdr = reinterpret_cast<BtHeader*>(ws);
    a.seq_off = reinterpret_cast<int32_t*>(ws + sizeof(BtHeader));
    a.area = reinterpret_cast<int32_t*>(ws + sizeof(BtHeader) + align16(4 * ((int64_t)a.num_seqs + 1)));
    a.rank = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(a.area) + ids_bytes(plan));
    // 0 = default: destination order, but table order when reshaping in place (measured faster there)
    a.dst_order = plan->opt.pair_order == 2 || (plan->opt.pair_order == 0 && !a.reshape);
    a.block_tokens = plan->src.block_tokens;
    a.nb_src = plan->src.num_blocks;
    a.nb_dst = plan->dst.num_blocks;
    const int64_t entries = (int64_t)a.num_seqs * a.maxb;
    if (entries <= kFusedEntries && a.nb_dst <= kFusedEntries) {
        bt_fused<<<1, kScanThreads, 0, stream>>>(a);
        if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
        count_launch();
        return AMOEBA_OK;
    }
    bt_scan<<<1, kScanThreads, 0, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    if (a.num_seqs == 0 && !a.reshape) return AMOEBA_OK;
    const int sms = cached_device_info().sms;
    if (sms <= 0) return AMOEBA_ERR_CUDA;
    if (!a.free_mask && a.num_seqs > 0) {  // ids that can repeat: who is first
        const int64_t work = a.reshape ? entries : std::min<int64_t>(a.pairs_cap, entries);
        const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((work + 255) / 256, (int64_t)sms * 8));
        bt_claim<<<grid, 256, 0, stream>>>(a);
        if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
        count_launch();
        if (a.dst_order) {
            bt_rank<<<1, kScanThreads, 0, stream>>>(a);
            if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
            count_launch();
        }
    }
    const int64_t units = std::max<int64_t>((int64_t)a.num_seqs * ((a.maxb + kSegment - 1) / kSegment),
                                            a.reshape ? (a.nb_dst + 31) / 32 : 0);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((units + 7) / 8, (int64_t)sms * 8));
    bt_assign<<<grid, 256, 0, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    return AMOEBA_OK;
}

}  // namespace amoeba

using namespace amoeba;

extern "C" amoeba_status amoeba_rewrite_workspace_bytes(const amoeba_plan* plan, int32_t num_seqs,
                                                        int32_t n_free_or_nb, int64_t* bytes) {
    if (!plan || !bytes || num_seqs < 0 || n_free_or_nb < 0) return AMOEBA_ERR_INVALID_ARG;
    *bytes = tables_workspace_bytes(plan, num_seqs);
    return AMOEBA_OK;
}

extern "C" amoeba_status amoeba_rewrite_block_tables(const amoeba_plan* plan, const int32_t* d_src_bt,
                                                     const int32_t* d_seq_lens, int32_t num_seqs,
                                                     int32_t max_blocks_per_seq, const int32_t* d_dst_free_list,
                                                     const uint8_t* d_dst_free_mask, int32_t n_free_or_nb,
                                                     int32_t* d_dst_bt, int32_t* d_pairs, int32_t pairs_cap,
                                                     int32_t* d_num_pairs, int32_t* d_dst_free_count_out,
                                                     int32_t* d_status, void* d_workspace, int64_t workspace_bytes,
                                                     void* cuda_stream) {
    if (!plan || num_seqs < 0 || max_blocks_per_seq <= 0 || n_free_or_nb < 0 || pairs_cap < 0)
        return AMOEBA_ERR_INVALID_ARG;
    if ((d_dst_free_list != nullptr) == (d_dst_free_mask != nullptr)) return AMOEBA_ERR_INVALID_ARG;
    if (!d_num_pairs || !d_dst_free_count_out || !d_status || !d_workspace) return AMOEBA_ERR_INVALID_ARG;
    if (num_seqs > 0 && (!d_src_bt || !d_seq_lens || !d_dst_bt)) return AMOEBA_ERR_INVALID_ARG;
    if (pairs_cap > 0 && !d_pairs) return AMOEBA_ERR_INVALID_ARG;
    if (d_dst_free_mask && n_free_or_nb != plan->dst.num_blocks) return AMOEBA_ERR_INVALID_ARG;
    if (workspace_bytes < tables_workspace_bytes(plan, num_seqs)) return AMOEBA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_workspace) % 16 || reinterpret_cast<uintptr_t>(d_pairs) % 8)
        return AMOEBA_ERR_ALIGNMENT;
    BtArgs a{};
    a.src_bt = d_src_bt;
    a.seq_lens = d_seq_lens;
    a.free_list = d_dst_free_list;
    a.free_mask = d_dst_free_mask;
    a.dst_bt = d_dst_bt;
    a.pairs = reinterpret_cast<int2*>(d_pairs);
    a.num_pairs = d_num_pairs;
    a.free_count_out = d_dst_free_count_out;
    a.status = d_status;
    a.num_seqs = num_seqs;
    a.maxb = max_blocks_per_seq;
    a.n_free_or_nb = n_free_or_nb;
    a.pairs_cap = pairs_cap;
    return launch_tables(plan, a, d_workspace, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" amoeba_status amoeba_reshape_block_tables(const amoeba_plan* plan, const int32_t* d_src_bt,
                                                     const int32_t* d_seq_lens, int32_t num_seqs,
                                                     int32_t max_blocks_per_seq, int32_t* d_dst_bt, int32_t* d_pairs,
                                                     int32_t pairs_cap, int32_t* d_num_pairs,
                                                     uint8_t* d_dst_free_mask_out, int32_t* d_dst_free_count_out,
                                                     int32_t* d_status, void* d_workspace, int64_t workspace_bytes,
                                                     void* cuda_stream) {
    if (!plan || num_seqs < 0 || max_blocks_per_seq <= 0 || pairs_cap < 0) return AMOEBA_ERR_INVALID_ARG;
    const int n = reshape_factor(plan);
    if (!n) return AMOEBA_ERR_UNSUPPORTED;
    if (!d_num_pairs || !d_dst_free_count_out || !d_dst_free_mask_out || !d_status || !d_workspace)
        return AMOEBA_ERR_INVALID_ARG;
    if (num_seqs > 0 && (!d_src_bt || !d_seq_lens || !d_dst_bt)) return AMOEBA_ERR_INVALID_ARG;
    if (pairs_cap > 0 && !d_pairs) return AMOEBA_ERR_INVALID_ARG;
    if (workspace_bytes < tables_workspace_bytes(plan, num_seqs)) return AMOEBA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_workspace) % 16 || reinterpret_cast<uintptr_t>(d_pairs) % 8)
        return AMOEBA_ERR_ALIGNMENT;
    BtArgs a{};
    a.src_bt = d_src_bt;
    a.seq_lens = d_seq_lens;
    a.dst_bt = d_dst_bt;
    a.pairs = reinterpret_cast<int2*>(d_pairs);
    a.num_pairs = d_num_pairs;
    a.free_count_out = d_dst_free_count_out;
    a.free_mask_out = d_dst_free_mask_out;
    a.status = d_status;
    a.num_seqs = num_seqs;
    a.maxb = max_blocks_per_seq;
    a.n_free_or_nb = plan->dst.num_blocks;
    a.pairs_cap = pairs_cap;
    a.reshape = n;
    return launch_tables(plan, a, d_workspace, static_cast<cudaStream_t>(cuda_stream));
}

// ------------------------------------------------------------------------------------------------------------
// Block tables of the in-place merge of N instances (Sec. 3.1, Improvement 1): block p of instance i becomes block
// p*N+i of the merged instance, and the blocks each instance's table names are marked live for the KV kernel.
// One launch; no CTA waits on another: every CTA decides the whole-call error by scanning all sequence lengths itself
// (a few KB), the live bytes are zeroed by a memset that precedes the launch on the stream.
namespace amoeba {

// split == false: instance tables -> merged table (p -> p*N+i).  split == true: the way back, merged table rows of
// the requests that go to instance i -> that instance's table (q -> q/N; q must be = i mod N).
template <bool split>
__global__ void __launch_bounds__(256) merge_tables(const int32_t* __restrict__ src_bt,
                                                    const int32_t* __restrict__ seq_lens, int32_t n_inst,
                                                    int32_t num_seqs, int32_t block_tokens,
                                                    int32_t max_blocks_per_seq, int32_t nb, int32_t* __restrict__ dst_bt,
                                                    uint32_t* live_words, int32_t* status) {
    const int64_t rows = (int64_t)n_inst * num_seqs;
    int bad_len = 0;
    for (int64_t k = threadIdx.x; k < rows; k += blockDim.x) {
        const int32_t len = seq_lens[k];
        bad_len |= len < 0 || ((int64_t)len + block_tokens - 1) / block_tokens > max_blocks_per_seq;
    }
    const bool call_failed = __syncthreads_or(bad_len) != 0;
    if (call_failed && blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_INVALID_ARG);

    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int32_t segs_per_row = (max_blocks_per_seq + kSegment - 1) / kSegment;
    bool bad = false;
    for (int64_t unit = warp; unit < rows * segs_per_row; unit += n_warps) {
        const int64_t row = unit / segs_per_row;  // instance * num_seqs + sequence
        const int32_t inst = (int32_t)(row / num_seqs);
        const int32_t col0 = (int32_t)(unit - row * segs_per_row) * kSegment;
        const int32_t nblk = call_failed ? 0 : (int32_t)(((int64_t)seq_lens[row] + block_tokens - 1) / block_tokens);
        for (int32_t i = col0 + lane; i < min(col0 + kSegment, max_blocks_per_seq); i += 32) {
            int32_t out = -1;
            if (i < nblk) {
                const int32_t id = src_bt[row * max_blocks_per_seq + i];
                const bool ok = split ? (id >= 0 && id < (int64_t)nb * n_inst && id % n_inst == inst)
                                      : (id >= 0 && id < nb);
                if (ok) {
                    const int32_t p = split ? id / n_inst : id;  // block of the instance's own pool
                    out = split ? p : p * n_inst + inst;
                    const int64_t idx = (int64_t)inst * nb + p;  // byte of the live array
                    const uint32_t bit = 1u << (8 * (idx & 3));
                    if (atomicOr(live_words + (idx >> 2), bit) & bit) bad = true;  // named twice by this instance
                } else {
                    bad = true;
                }
            }
            dst_bt[row * max_blocks_per_seq + i] = out;
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_BAD_BLOCK_ID);
}

}  // namespace amoeba

static amoeba_status merge_or_split_tables(bool split, const amoeba_plan* plan, const int32_t* d_src_bt,
                                           const int32_t* d_seq_lens, int32_t num_seqs, int32_t max_blocks_per_seq,
                                           int32_t* d_dst_bt, uint8_t* d_live, int32_t* d_status, void* cuda_stream) {
    if (!plan || num_seqs < 0 || max_blocks_per_seq <= 0 || !d_live || !d_status) return AMOEBA_ERR_INVALID_ARG;
    if (num_seqs > 0 && (!d_src_bt || !d_seq_lens || !d_dst_bt)) return AMOEBA_ERR_INVALID_ARG;
    const int n = merge_instances(plan);
    if (!n) return AMOEBA_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(d_live) % 16) return AMOEBA_ERR_ALIGNMENT;
    int64_t live_bytes = 0;
    amoeba_merge_live_bytes(plan, &live_bytes);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(d_live, 0, (size_t)live_bytes, stream) != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    if (num_seqs == 0) return AMOEBA_OK;
    const DeviceInfo dev = cached_device_info();
    if (dev.sms <= 0) return AMOEBA_ERR_CUDA;
    const int64_t units = (int64_t)n * num_seqs * ((max_blocks_per_seq + kSegment - 1) / kSegment);
    const int grid = (int)std::min<int64_t>((units + 7) / 8, (int64_t)dev.sms * 4);
    auto kernel = split ? merge_tables<true> : merge_tables<false>;
    kernel<<<grid, 256, 0, stream>>>(d_src_bt, d_seq_lens, n, num_seqs, plan->src.block_tokens, max_blocks_per_seq,
                                     plan->src.num_blocks, d_dst_bt, reinterpret_cast<uint32_t*>(d_live), d_status);
    if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    return AMOEBA_OK;
}

extern "C" amoeba_status amoeba_merge_block_tables(const amoeba_plan* plan, const int32_t* d_src_bt,
                                                   const int32_t* d_seq_lens, int32_t num_seqs,
                                                   int32_t max_blocks_per_seq, int32_t* d_dst_bt, uint8_t* d_live,
                                                   int32_t* d_status, void* cuda_stream) {
    return merge_or_split_tables(false, plan, d_src_bt, d_seq_lens, num_seqs, max_blocks_per_seq, d_dst_bt, d_live,
                                 d_status, cuda_stream);
}

extern "C" amoeba_status amoeba_split_block_tables(const amoeba_plan* plan, const int32_t* d_merged_bt,
                                                   const int32_t* d_seq_lens, int32_t num_seqs,
                                                   int32_t max_blocks_per_seq, int32_t* d_inst_bt, uint8_t* d_live,
                                                   int32_t* d_status, void* cuda_stream) {
    return merge_or_split_tables(true, plan, d_merged_bt, d_seq_lens, num_seqs, max_blocks_per_seq, d_inst_bt, d_live,
                                 d_status, cuda_stream);
}

// ------------------------------------------------------------------------------------------------------------
// Variant for callers that cannot allocate device memory: the scratch is an array in the library's device image.
namespace amoeba {

// One copy per GPU that loads this library, alive until the process exits.
static __device__ __align__(256) unsigned char g_builtin_scratch[AMOEBA_BUILTIN_SCRATCH_BYTES];

// In host code `g_builtin_scratch` is only a handle for the runtime, not an address a kernel could use; the
// device-side address is asked for once per device and remembered here (index = device ordinal).  The remembered
// address belongs to the device's primary context as it was at that first call: it does not survive a
// cudaDeviceReset of that device.
static void* g_builtin_scratch_addr[kMaxDevices];
static std::mutex g_builtin_scratch_mutex;

}  // namespace amoeba

extern "C" amoeba_status amoeba_rewrite_block_tables_builtin_scratch(
    const amoeba_plan* plan, const int32_t* d_src_bt, const int32_t* d_seq_lens, int32_t num_seqs,
    int32_t max_blocks_per_seq, const int32_t* d_dst_free_list, const uint8_t* d_dst_free_mask, int32_t n_free_or_nb,
    int32_t* d_dst_bt, int32_t* d_pairs, int32_t pairs_cap, int32_t* d_num_pairs, int32_t* d_dst_free_count_out,
    int32_t* d_status, void* cuda_stream) {
    if (!plan || num_seqs < 0 || n_free_or_nb < 0) return AMOEBA_ERR_INVALID_ARG;
    if (tables_workspace_bytes(plan, num_seqs) > (int64_t)AMOEBA_BUILTIN_SCRATCH_BYTES) return AMOEBA_ERR_TOO_LARGE;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) {
        (void)cudaGetLastError();  // do not leave the runtime's error state set for a later, unrelated check
        return AMOEBA_ERR_CUDA;
    }
    if (dev >= kMaxDevices) return AMOEBA_ERR_UNSUPPORTED;  // more device ordinals than this table remembers
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_builtin_scratch_mutex);
        if (!g_builtin_scratch_addr[dev]) {  // first use with this device current
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_builtin_scratch) != cudaSuccess || !p) {
                (void)cudaGetLastError();
                return AMOEBA_ERR_CUDA;
            }
            g_builtin_scratch_addr[dev] = p;
        }
        scratch = g_builtin_scratch_addr[dev];
    }
    return amoeba_rewrite_block_tables(plan, d_src_bt, d_seq_lens, num_seqs, max_blocks_per_seq, d_dst_free_list,
                                       d_dst_free_mask, n_free_or_nb, d_dst_bt, d_pairs, pairs_cap, d_num_pairs,
                                       d_dst_free_count_out, d_status, scratch, AMOEBA_BUILTIN_SCRATCH_BYTES,
                                       cuda_stream);
}
