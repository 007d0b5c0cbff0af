// Internal definitions shared by the host planner and the kernel launchers of the re-layout library.
#pragma once
#include <atomic>
#include <cstdint>
#include <vector>

#include "amoeba.h"

namespace amoeba {

constexpr int kNumTensors = 7;  // q,k,v,o,gate,up,down
constexpr int kMaxWeightDescs = 256;
constexpr int kMaxWeightPtrs = 1536;  // per launch: layers * (a + b) * kNumTensors pointers
// (descriptors and pointers travel in kernel parameter space: 256 * 72 + 1536 * 8 bytes, under the 32 KiB limit)
constexpr int64_t kDefaultKvChunk = 8192;   // upper bound of one KV copy work item
constexpr int64_t kDefaultWChunk = 8192;    // upper bound of one weight copy work item

// One weight copy descriptor as the kernels see it (per layer, relative to that layer's buffers).
struct WDescDev {
    int64_t src_off, dst_off;      // bytes into the source / destination buffer
    int64_t src_pitch, dst_pitch;  // bytes between consecutive rows
    int64_t row_bytes;             // bytes per row
    int32_t n_rows;
    int32_t src_slot, dst_slot;    // rank * kNumTensors + tensor
    int32_t rows_per_item;         // rows one work item covers (1 when a row is split into column chunks)
    int32_t col_chunks;            // work items per row group along the row
    int32_t chunk_bytes;           // bytes per column chunk (last one may be shorter)
    int32_t item_begin;            // first work item of this descriptor within a layer
    int32_t pad;
};

// Box geometry of the KV copy when a side is token-first and the bulk-copy kernels address it through a tensor map
// (tiled TMA): a work item is `heads` consecutive headers x K and V x `tokens` consecutive tokens of one block.  On a
// token-first side that is one 5-D box {dim, token, K/V, header, layer} of the worker's pool; on a header-centric
// side it is 2*heads rows of tokens*vec_bytes, consecutive rows block_tokens*vec_bytes apart.  In shared memory
// both are the same dense [header][K/V][token][dim] tile, so one load and one store move the item.
struct KvBoxGeom {
    int32_t usable;      // 0: shape outside the tensor-map limits, row copies are used instead
    int32_t heads;       // headers per item (divides the run length)
    int32_t tokens;      // tokens per item (divides block_tokens)
    int32_t sub_runs;    // items along a run of headers
    int32_t tok_groups;  // items along the tokens of a block
    int64_t item_bytes;
};

// Tuning knobs of one copy kernel; 0 = use the kernel's default.
struct KernelOpts {
    int copy_path = 0;    // 1 vector ld/st, 2 bulk-copy ring per warp, 3 bulk-copy producer/consumer ring
    int ctas_per_sm = 0;
    int64_t chunk_bytes = 0;
    int stages = 0;       // ring depth
    int lag = 0;          // loads ahead of stores (path 2) / stores kept in flight (path 3)
    int warps = 0;        // rings per CTA
    int hint = 0;         // 1 + bit mask: bit 0 loads evict-first, bit 1 stores evict-first (0 = default)
    int max_ctas = 0;     // cap on the persistent grid (0 = none): leaves SMs free for kernels that run beside the copy
    int tensor_maps = 0;  // KV only: 1 = row copies on token-first sides, 2 = tensor-map boxes (0 = default)
    int l2_promotion = 0; // KV only: 1 + CUtensorMapL2promotion of the token-first pools' tensor maps (0 = default)
    int wait_tries = 0;   // polls of one bounded mbarrier wait before the kernel gives up (0 = default)
};

struct Options {
    KernelOpts kv, w;
    int pair_order = 0;  // pair list of the table calls: 0 / 2 ascending by destination id, 1 in table order
};

// How the KV copy of one (block pair, layer) is cut into 2-D work items.  A "unit" is the largest piece that is a
// regular 2-D copy on both sides: `rows` rows of `row_bytes`, consecutive rows `src_row_pitch` / `dst_row_pitch`
// apart.  It covers `heads_per_unit` consecutive headers and either both of K and V (planes == 1) or one of them.
//   both sides header-centric : unit = one run of headers, K and V together, one contiguous row
//   both sides token-first    : unit = one run of headers of K or of V; one row per token
//   mixed orders              : unit = one header of K or of V; one row per token (head_dim elements)
struct KvGeom {
    int32_t planes;          // 1: a unit spans K and V; 2: K and V are separate units
    int32_t heads_per_unit;  // consecutive headers per unit
    int32_t head_units;      // num_kv_heads / heads_per_unit
    int32_t rows;            // rows per unit (1 or block_tokens)
    int64_t row_bytes;
    int64_t src_row_pitch, dst_row_pitch;
    int32_t rows_per_item;   // rows one work item covers (1 when a row is split into column chunks)
    int32_t row_groups;      // ceil(rows / rows_per_item)
    int32_t col_chunks;      // work items along a row
    int32_t chunk_bytes;     // bytes per column chunk (divides row_bytes)
    int64_t item_bytes;      // largest work item
};

}  // namespace amoeba

struct amoeba_plan {
    amoeba_layout src, dst;
    // KV
    int32_t heads_src, heads_dst;  // K/V headers per source / destination worker
    int32_t heads_per_run, runs_per_block;
    int64_t unit_bytes;  // one (block, header): 2 * T * D * e
    int64_t run_bytes, chunk_bytes;  // chunk_bytes: largest KV work item
    int64_t vec_bytes;   // one (token, header): D * e
    amoeba::KvGeom kv;
    amoeba::KvBoxGeom kvbox;
    int64_t src_block_bytes, dst_block_bytes, src_layer_stride, dst_layer_stride;
    // weights
    std::vector<amoeba_weight_desc> wdescs;  // public form
    std::vector<amoeba::WDescDev> wdev;      // kernel form (chunked with the current options)
    int32_t items_per_layer;
    int64_t weight_bytes_per_layer;  // one copy (read side)
    amoeba::Options opt;
    // Bumped whenever the options change: anything a launcher has cached for this plan (encoded tensor maps) is
    // re-derived when its generation differs.
    std::atomic<uint64_t> generation{1};
    void bump_generation() { generation.fetch_add(1, std::memory_order_relaxed); }
    struct LaunchCache* cache = nullptr;  // owned; created on first use by the KV launcher
    ~amoeba_plan();
};

namespace amoeba {
// Number of instances N if the plan describes an in-place merge of N instances (see amoeba.h), else 0.
int merge_instances(const amoeba_plan* p);
// In-place block reshaping of one instance: +N if the destination has N times the source's TP degree and blocks,
// -N if the source has N times the destination's, 0 if the plan describes neither.
int reshape_factor(const amoeba_plan* p);
// One public weight descriptor in kernel form; *item is the running count of work items.
WDescDev chunk_desc(const amoeba_weight_desc& d, int64_t cap, int64_t* item);
// Re-derives chunk sizes and the per-descriptor work-item split from plan->opt.
amoeba_status finalize_chunks(amoeba_plan* p);
void count_launch(int n = 1);
}  // namespace amoeba
