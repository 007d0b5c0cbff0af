// Destination block bookkeeping for the KV migration (Sec. 3.1: each worker prepares reserved pages for the KV it
// receives).  Two launches, no CTA ever waits on another:
//   bt_scan   (1 CTA)   blocks per sequence, exclusive prefix sum over the sequences, and - when the free blocks
//                       come as a byte mask - their compaction into an ascending id list (ballot + popc prefix
//                       sums, one warp-wide ballot per 32 mask bytes); decides the whole-call errors.
//   bt_assign (grid)    one warp per 128-entry segment of a block-table row: k-th block overall takes the k-th free
//                       id; writes the destination table (with -1 padding) and the (source, destination) pair list.
#include <cuda_runtime.h>

#include <mutex>

#include "launch.hpp"
#include "plan.hpp"

namespace amoeba {

struct BtHeader {  // first 64 bytes of the workspace
    int32_t total;   // blocks assigned by this call (0 on a whole-call error)
    int32_t n_free;  // free destination blocks before the call
    int32_t err;     // whole-call error code or 0
    int32_t pad[13];
};

constexpr int kScanThreads = 1024;

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

__global__ void __launch_bounds__(kScanThreads) bt_scan(const int32_t* __restrict__ seq_lens, int32_t num_seqs,
                                                        int32_t block_tokens, int32_t max_blocks_per_seq,
                                                        const uint8_t* __restrict__ free_mask, int32_t n_free_or_nb,
                                                        int32_t pairs_cap, BtHeader* hdr, int32_t* __restrict__ seq_off,
                                                        int32_t* __restrict__ free_ids, int32_t* num_pairs,
                                                        int32_t* free_count_out, int32_t* status) {
    __shared__ int32_t warp_sums[33];
    __shared__ int32_t bad_len;
    if (threadIdx.x == 0) bad_len = 0;
    __syncthreads();

    // ---- blocks per sequence and their exclusive prefix sum
    int64_t carry = 0;
    for (int32_t base = 0; base < num_seqs; base += kScanThreads) {
        const int32_t s = base + threadIdx.x;
        int32_t nb = 0;
        if (s < num_seqs) {
            const int32_t len = seq_lens[s];
            const int64_t need = ((int64_t)len + block_tokens - 1) / block_tokens;
            if (len < 0 || need > max_blocks_per_seq) bad_len = 1;
            else nb = (int32_t)need;
        }
        int32_t tile_total;
        const int32_t off = cta_exclusive_scan(nb, warp_sums, &tile_total);
        if (s < num_seqs) seq_off[s] = (int32_t)min(carry + off, (int64_t)INT32_MAX);
        carry += tile_total;
    }
    const int64_t total = carry;

    // ---- ordered free list from the mask: ascending ids of the non-zero bytes
    int64_t n_free = n_free_or_nb;
    if (free_mask) {
        const int lane = threadIdx.x & 31;
        int32_t found = 0;
        for (int32_t base = 0; base < n_free_or_nb; base += kScanThreads) {
            const int32_t id = base + threadIdx.x;
            const bool is_free = id < n_free_or_nb && free_mask[id] != 0;
            const uint32_t ballot = __ballot_sync(0xffffffffu, is_free);
            int32_t tile_total;
            const int32_t warp_off = cta_exclusive_scan(lane == 0 ? __popc(ballot) : 0, warp_sums, &tile_total);
            const int32_t my_warp_off = __shfl_sync(0xffffffffu, warp_off, 0);
            if (is_free) free_ids[found + my_warp_off + __popc(ballot & ((1u << lane) - 1u))] = id;
            found += tile_total;
        }
        n_free = found;
    }

    __syncthreads();
    if (threadIdx.x == 0) {
        int32_t err = 0;
        if (bad_len) err = AMOEBA_ERR_INVALID_ARG;
        else if (total > pairs_cap) err = AMOEBA_ERR_INVALID_ARG;
        else if (total > n_free) err = AMOEBA_ERR_NO_FREE_BLOCKS;
        const int32_t assigned = err ? 0 : (int32_t)total;
        hdr->total = assigned;
        hdr->n_free = (int32_t)n_free;
        hdr->err = err;
        *num_pairs = assigned;
        *free_count_out = (int32_t)n_free - assigned;
        if (err) atomicCAS(status, 0, err);
    }
}

constexpr int kSegment = 128;  // table entries one warp handles per step

__global__ void __launch_bounds__(256) bt_assign(const int32_t* __restrict__ src_bt,
                                                 const int32_t* __restrict__ seq_lens, int32_t num_seqs,
                                                 int32_t block_tokens, int32_t max_blocks_per_seq,
                                                 const int32_t* __restrict__ free_ids, const BtHeader* hdr,
                                                 const int32_t* __restrict__ seq_off, int32_t nb_src, int32_t nb_dst,
                                                 int32_t* __restrict__ dst_bt, int2* __restrict__ pairs,
                                                 int32_t* status) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int32_t segs_per_row = (max_blocks_per_seq + kSegment - 1) / kSegment;
    const bool call_failed = hdr->err != 0;
    bool bad = false;
    for (int64_t unit = warp; unit < (int64_t)num_seqs * segs_per_row; unit += n_warps) {
        const int32_t s = (int32_t)(unit / segs_per_row);
        const int32_t col0 = (int32_t)(unit - (int64_t)s * segs_per_row) * kSegment;
        const int32_t nb = call_failed ? 0 : (int32_t)(((int64_t)seq_lens[s] + block_tokens - 1) / block_tokens);
        const int32_t off = seq_off[s];
        for (int32_t i = col0 + lane; i < min(col0 + kSegment, max_blocks_per_seq); i += 32) {
            int32_t out = -1;
            if (i < nb) {
                const int32_t k = off + i;
                const int32_t dst = free_ids[k];
                const int32_t src = src_bt[(int64_t)s * max_blocks_per_seq + i];
                const bool dst_ok = dst >= 0 && dst < nb_dst, src_ok = src >= 0 && src < nb_src;
                out = dst_ok ? dst : -1;
                pairs[k] = (dst_ok && src_ok) ? make_int2(src, dst) : make_int2(-1, -1);
                bad |= !(dst_ok && src_ok);
            }
            dst_bt[(int64_t)s * max_blocks_per_seq + i] = out;
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicCAS(status, 0, (int)AMOEBA_ERR_BAD_BLOCK_ID);
}

static int64_t align16(int64_t x) { return (x + 15) & ~int64_t(15); }

}  // namespace amoeba

using namespace amoeba;

extern "C" amoeba_status amoeba_rewrite_workspace_bytes(const amoeba_plan* plan, int32_t num_seqs,
                                                        int32_t n_free_or_nb, int64_t* bytes) {
    if (!plan || !bytes || num_seqs < 0 || n_free_or_nb < 0) return AMOEBA_ERR_INVALID_ARG;
    *bytes = (int64_t)sizeof(BtHeader) + align16(4 * ((int64_t)num_seqs + 1)) + align16(4 * (int64_t)n_free_or_nb);
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
    int64_t need = 0;
    amoeba_rewrite_workspace_bytes(plan, num_seqs, n_free_or_nb, &need);
    if (workspace_bytes < need) return AMOEBA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_workspace) % 16 || reinterpret_cast<uintptr_t>(d_pairs) % 8)
        return AMOEBA_ERR_ALIGNMENT;

    char* ws = static_cast<char*>(d_workspace);
    BtHeader* hdr = reinterpret_cast<BtHeader*>(ws);
    int32_t* seq_off = reinterpret_cast<int32_t*>(ws + sizeof(BtHeader));
    int32_t* compact = reinterpret_cast<int32_t*>(ws + sizeof(BtHeader) + align16(4 * ((int64_t)num_seqs + 1)));
    const int32_t* free_ids = d_dst_free_mask ? compact : d_dst_free_list;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    bt_scan<<<1, kScanThreads, 0, stream>>>(d_seq_lens, num_seqs, plan->src.block_tokens, max_blocks_per_seq,
                                            d_dst_free_mask, n_free_or_nb, pairs_cap, hdr, seq_off, compact,
                                            d_num_pairs, d_dst_free_count_out, d_status);
    if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    if (num_seqs == 0) return AMOEBA_OK;

    DeviceInfo dev;
    if (!device_info(&dev)) return AMOEBA_ERR_CUDA;
    const int64_t units = (int64_t)num_seqs * ((max_blocks_per_seq + kSegment - 1) / kSegment);
    const int grid = (int)std::min<int64_t>((units + 7) / 8, (int64_t)dev.sms * 8);
    bt_assign<<<grid, 256, 0, stream>>>(d_src_bt, d_seq_lens, num_seqs, plan->src.block_tokens, max_blocks_per_seq,
                                        free_ids, hdr, seq_off, plan->src.num_blocks, plan->dst.num_blocks, d_dst_bt,
                                        reinterpret_cast<int2*>(d_pairs), d_status);
    if (cudaGetLastError() != cudaSuccess) return AMOEBA_ERR_CUDA;
    count_launch();
    return AMOEBA_OK;
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
    DeviceInfo dev;
    if (!device_info(&dev)) return AMOEBA_ERR_CUDA;
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
// device-side address is asked for once per device and remembered here (index = device ordinal).
constexpr int kMaxDevices = 64;
static void* g_builtin_scratch_addr[kMaxDevices];
static std::mutex g_builtin_scratch_mutex;

}  // namespace amoeba

extern "C" amoeba_status amoeba_rewrite_block_tables_builtin_scratch(
    const amoeba_plan* plan, const int32_t* d_src_bt, const int32_t* d_seq_lens, int32_t num_seqs,
    int32_t max_blocks_per_seq, const int32_t* d_dst_free_list, const uint8_t* d_dst_free_mask, int32_t n_free_or_nb,
    int32_t* d_dst_bt, int32_t* d_pairs, int32_t pairs_cap, int32_t* d_num_pairs, int32_t* d_dst_free_count_out,
    int32_t* d_status, void* cuda_stream) {
    int64_t need = 0;
    const amoeba_status st = amoeba_rewrite_workspace_bytes(plan, num_seqs, n_free_or_nb, &need);
    if (st != AMOEBA_OK) return st;
    if (need > (int64_t)AMOEBA_BUILTIN_SCRATCH_BYTES) return AMOEBA_ERR_TOO_LARGE;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AMOEBA_ERR_CUDA;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_builtin_scratch_mutex);
        if (!g_builtin_scratch_addr[dev]) {  // first use with this device current
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_builtin_scratch) != cudaSuccess || !p) return AMOEBA_ERR_CUDA;
            g_builtin_scratch_addr[dev] = p;
        }
        scratch = g_builtin_scratch_addr[dev];
    }
    return amoeba_rewrite_block_tables(plan, d_src_bt, d_seq_lens, num_seqs, max_blocks_per_seq, d_dst_free_list,
                                       d_dst_free_mask, n_free_or_nb, d_dst_bt, d_pairs, pairs_cap, d_num_pairs,
                                       d_dst_free_count_out, d_status, scratch, AMOEBA_BUILTIN_SCRATCH_BYTES,
                                       cuda_stream);
}
