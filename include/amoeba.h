/*
 * amoeba.h - C ABI of the on-GPU TP a->b re-layout library (sm_100a).
 *
 * The library re-lays-out the state of one running LLM instance from a tensor-parallel partition of degree a to
 * one of degree b without recomputing anything (the transformation the Amoeba paper introduces in its Sec. 1 and
 * designs in Sec. 3.1 - 3.2).  The state is
 *   - the paged, head-sharded KV cache, by default in the header-centric layout of Sec. 3.1 ("Improvement 1"):
 *       pool of worker r:  [layer][block][header of r][K/V][token][head_dim]
 *     (the token-first order [layer][K/V][block][token][header of r][head_dim] is accepted on either side, so a
 *     transformation can also convert between the two), where worker r (0-indexed here; W_{r+1} in the paper) owns the K/V headers r*Hkv/tp ... (r+1)*Hkv/tp - 1
 *     (Sec. 3.1 "Base solution", 1-indexed there), and
 *   - the projection weights, stored [out,in] row-major and partitioned as in Sec. 3.2, Eq. 1:
 *     q/k/v/gate/up by output rows (the paper's column-wise split of U), o_proj/down_proj by input columns (the
 *     paper's row-wise split of D).
 * All shards of all workers live on the one GPU; nothing crosses GPUs.
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer unless its name starts with h_ or the comment says "host array".
 *     The caller owns every buffer and the stream; the library owns only the plan object.
 *   - Data calls are asynchronous on the given stream (a cudaStream_t passed as void*; NULL = default stream),
 *     never synchronise and never allocate device memory.  amoeba_reshard_kv and amoeba_reshard_weights are out of
 *     place: a destination buffer that is also a source buffer is refused (INVALID_ARG), and partial overlaps are
 *     the caller's to avoid.  The calls whose names end in _inplace work on the buffers they are given.
 *   - Errors the host can see return a code and launch nothing.  Errors only the device can see (bad block ids,
 *     not enough free blocks) are written to *d_status: an int32 the caller zeroes beforehand; the first non-zero
 *     code sticks, offending items are skipped, the kernel never traps.
 *   - Only destination blocks named in the pair list, and destination weight bytes covered by the layout, are
 *     written.  Every other destination byte keeps its value.
 *   - Block ids are int32; byte offsets are 64-bit.  Pointers, run lengths and pitches must be multiples of 16 B
 *     (checked: AMOEBA_ERR_ALIGNMENT).
 *   - Thread-compatible.  Process-wide state is limited to an atomic launch counter and a few lock-protected
 *     look-up caches (device attributes, the shared-memory opt-in of each kernel, the driver's tensor-map encoder,
 *     the built-in scratch address per device); a plan also caches the tensor maps it encoded for the last set of
 *     pool addresses.  The per-device caches assume that a device's primary context lives as long as the process: after a
 *     cudaDeviceReset of a device the library must not be used on that device any more.  A plan may be used from
 *     several threads if its options are not changed concurrently.
 *     No C++ exception crosses this boundary (a failed host allocation is AMOEBA_ERR_NO_MEMORY).
 *   - AMOEBA_ERR_TIMEOUT: every on-device wait of a kernel on one of its own bulk copies is bounded.  A kernel whose
 *     wait runs out records the code in *d_status, waits (bounded again) for the copies it still has in flight and
 *     returns; the CUDA context stays usable, the destination holds a mix of copied and untouched items, and the
 *     call can simply be issued again.
 */
#ifndef AMOEBA_H_
#define AMOEBA_H_

#include <stdint.h>

#define AMOEBA_API __attribute__((visibility("default")))

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AMOEBA_OK = 0,
    AMOEBA_ERR_INVALID_ARG = 1,    /* null pointer, negative size, inconsistent layouts, bad sequence length */
    AMOEBA_ERR_UNSUPPORTED = 2,    /* e.g. head count not divisible by tp, unknown kv_order */
    AMOEBA_ERR_ALIGNMENT = 3,      /* a pointer, run or pitch is not a multiple of 16 bytes */
    AMOEBA_ERR_NO_FREE_BLOCKS = 4, /* destination has fewer free blocks than the sequences need */
    AMOEBA_ERR_BAD_BLOCK_ID = 5,   /* a block id outside its pool (or -1 inside a sequence) */
    AMOEBA_ERR_CUDA = 6,           /* a CUDA runtime call failed (launch error, no device) */
    AMOEBA_ERR_TIMEOUT = 7,        /* a bounded on-device wait on the kernel's own bulk copy ran out */
    AMOEBA_ERR_TOO_LARGE = 8,      /* the problem needs more scratch than the library's built-in scratch array holds */
    AMOEBA_ERR_NO_MEMORY = 9,      /* a host allocation inside the library failed */
    AMOEBA_ERR_INTERNAL = 10       /* checked build only: a work item would have reached outside its buffer (skipped) */
} amoeba_status;

/* Storage order of one layer of a worker's KV pool (Sec. 3.1).  HEAD_MAJOR is the paper's header-centric layout
 * ("Improvement 1"); TOKEN_MAJOR is the token-first layout of mainstream engines that the paper starts from: K and V
 * are two contiguous regions of the layer and a token's headers are stored together. */
enum {
    AMOEBA_KV_HEAD_MAJOR = 0, /* [block][header][K/V][token][dim] */
    AMOEBA_KV_TOKEN_MAJOR = 1 /* [K/V][block][token][header][dim] */
};
enum { AMOEBA_MAX_TP = 32 }; /* and at most 36 intersecting (source worker, destination worker) pairs: 256 weight
                                descriptors per layer; nested degrees up to 32 -> 1 and 1 -> 32 fit */

/* Transformer shape.  elem_bytes is the size of one weight / KV element: 2 (fp16, bf16 - the paper's types), 1 (8-bit
 * formats) or 4; the elements are moved, never interpreted.  Every contiguous run must still be a multiple of 16 bytes. */
typedef struct {
    int32_t num_layers, hidden, num_q_heads, num_kv_heads, head_dim, intermediate, elem_bytes;
} amoeba_model;

/* How one instance's state is laid out at one TP degree. */
typedef struct {
    amoeba_model model;
    int32_t tp;            /* number of workers; must divide num_q_heads, num_kv_heads and intermediate */
    int32_t block_tokens;  /* tokens per KV block */
    int32_t num_blocks;    /* capacity of every worker's pool, in blocks, per layer */
    int32_t kv_order;      /* AMOEBA_KV_HEAD_MAJOR or AMOEBA_KV_TOKEN_MAJOR; source and destination may differ */
    int32_t fused_qkv;     /* 1: worker buffer [q_r; k_r; v_r] (pointer in .q, .k/.v unused); 0: three buffers */
    int32_t fused_gate_up; /* 1: worker buffer [gate_r; up_r] (pointer in .gate, .up unused); 0: two buffers */
    int64_t kv_layer_stride_bytes; /* distance between layers inside a worker's pool; 0 = dense */
    /* Weight padding (Sec. 3.2, "Improvement 1").  weight_pad_parts = P > 0: every weight buffer of a worker is P/tp
     * partitions (P = the largest TP degree the instance may take; tp must divide P, P must divide the head counts
     * and the FFN width), partition j starting at j * pitch, pitch = the partition's bytes rounded up to a multiple
     * of weight_page_bytes (0 = 2 MiB, the allocation granularity the paper pads to).  A partition of q/k/v/gate/up
     * is its rows; a partition of o_proj/down_proj is its own dense [hidden, columns/P] matrix (the paper's D_i); a
     * fused buffer pads after each partition's [q;k;v] or [gate;up].  Pad bytes are never read or written.
     * weight_pad_parts = 0: dense shards, no padding. */
    int32_t weight_pad_parts;
    int32_t reserved;
    int64_t weight_page_bytes;
} amoeba_layout;

/* Padding arithmetic of one weight buffer of a layout (Sec. 3.2, Table 2 counts `pages` per tensor). */
typedef struct {
    int32_t partitions_per_worker; /* P/tp, or 1 without padding */
    int32_t reserved;
    int64_t partition_bytes;       /* bytes of one partition of this buffer */
    int64_t pitch_bytes;           /* partition_bytes rounded up to whole pages (= partition_bytes without padding) */
    int64_t page_bytes;
    double pages;                  /* partition_bytes / page_bytes: fractional = the partition boundary is unaligned */
} amoeba_pad_info;

/* One worker's weight buffers for one layer (device pointers; unused slots NULL). */
typedef struct {
    void *q, *k, *v, *o, *gate, *up, *down;
} amoeba_layer_weights;

/* Buffer sizes implied by a layout: one worker's KV pool over all layers, and one worker's buffer of one layer for
 * `tensor` (0..6 = q,k,v,o,gate,up,down; a fused buffer is asked for by its first member, its other members give 0).
 * Errors: INVALID_ARG, UNSUPPORTED (same checks as amoeba_plan_create). */
AMOEBA_API amoeba_status amoeba_layout_kv_pool_bytes(const amoeba_layout* layout, int64_t* bytes);
AMOEBA_API amoeba_status amoeba_layout_weight_bytes(const amoeba_layout* layout, int32_t tensor, int64_t* bytes);
/* Partition size, pitch and page count of buffer `tensor` (same numbering; a member of a fused buffer other than its
 * first gives zeros).  Errors as above. */
AMOEBA_API amoeba_status amoeba_layout_pad_info(const amoeba_layout* layout, int32_t tensor, amoeba_pad_info* out);

typedef struct amoeba_plan amoeba_plan; /* opaque, host memory only */

/*
 * amoeba_plan_create  (the planning step, "amoeba_plan(src_layout, dst_layout)")
 * Validates the two layouts (same model, same block_tokens; tp divides the head counts and the FFN width) and
 * derives, from the partition rules of Sec. 3.1 / Eq. 1, which byte ranges of which source worker go to which
 * destination worker: the K/V header run shared by one source and one destination worker, and one copy descriptor
 * per intersecting (source worker, destination worker, tensor).  Needs no GPU.  *out is owned by the caller until
 * amoeba_plan_destroy.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT.
 */
AMOEBA_API amoeba_status amoeba_plan_create(const amoeba_layout* src, const amoeba_layout* dst, amoeba_plan** out);
AMOEBA_API void amoeba_plan_destroy(amoeba_plan* plan);

/* Algorithmic bytes (read + written) of re-laying-out n_blocks live KV blocks over all layers, and of all layers'
 * weights: what the roofline figures are computed from.  Either output may be NULL. */
AMOEBA_API amoeba_status amoeba_plan_bytes(const amoeba_plan* plan, int64_t n_blocks, int64_t* kv_bytes_rw, int64_t* w_bytes_rw);

/* What the planner derived, for inspection and host-side tests. */
typedef struct {
    int32_t heads_per_run;   /* consecutive K/V headers that share one source and one destination worker */
    int32_t runs_per_block;  /* num_kv_heads / heads_per_run */
    int64_t run_bytes;       /* heads_per_run * 2 * block_tokens * head_dim * elem_bytes */
    int64_t chunk_bytes;     /* largest copy work item in bytes (both sides header-centric: it divides run_bytes) */
    int64_t src_block_bytes, dst_block_bytes;   /* one block in a source / destination worker's pool */
    int64_t src_layer_stride, dst_layer_stride; /* bytes between layers in a pool */
} amoeba_kv_info;
AMOEBA_API amoeba_status amoeba_plan_kv_info(const amoeba_plan* plan, amoeba_kv_info* out);

/* One weight copy descriptor, relative to the buffers of one layer: n_rows runs of row_bytes each, run i read at
 * src_off + i*src_pitch of source worker src_rank's buffer `src_tensor` (0..6 = q,k,v,o,gate,up,down; a fused
 * buffer is named by its first member) and written at dst_off + i*dst_pitch of the destination's. */
typedef struct {
    int32_t src_rank, src_tensor, dst_rank, dst_tensor;
    int64_t src_off, dst_off, row_bytes, src_pitch, dst_pitch;
    int32_t n_rows, reserved;
} amoeba_weight_desc;
AMOEBA_API int32_t amoeba_plan_num_weight_descs(const amoeba_plan* plan);
AMOEBA_API amoeba_status amoeba_plan_weight_desc(const amoeba_plan* plan, int32_t index, amoeba_weight_desc* out);

/* Tuning knobs (defaults are chosen from measurements; the tests and the benchmark sweep them).  An option id
 * sets both copy kernels; id + AMOEBA_OPT_WEIGHTS_ONLY sets the weight kernel only, id + AMOEBA_OPT_KV_ONLY the KV
 * kernel only.  Value 0 = the kernel's default. */
enum {
    AMOEBA_OPT_COPY_PATH = 0,   /* 1 = 16-byte vector loads/stores, 2 = bulk-copy (TMA) ring per warp,
                                   3 = bulk-copy ring shared by a producer warp and a consumer warp */
    AMOEBA_OPT_CTAS_PER_SM = 1, /* persistent grid = this * SM count */
    AMOEBA_OPT_CHUNK_BYTES = 2, /* upper bound of one copy work item, multiple of 16, <= 65536 */
    AMOEBA_OPT_STAGES = 3,      /* bulk-copy ring depth (2..16) */
    AMOEBA_OPT_LAG = 4,         /* path 2: loads issued ahead of stores; path 3: stores kept in flight (< stages) */
    AMOEBA_OPT_WARPS = 5,       /* bulk-copy rings per CTA */
    AMOEBA_OPT_L2_HINT = 6,     /* 1 = none, 2 = loads evict-first, 3 = stores evict-first, 4 = both */
    AMOEBA_OPT_TENSOR_MAPS = 7, /* KV, bulk-copy paths, token-first sides: 1 = one bulk copy per token row,
                                   2 = one tiled (tensor-map) copy per work item */
    AMOEBA_OPT_MAX_CTAS = 8,    /* cap on the persistent grid of the copy kernels (0 = none).  One CTA occupies one SM,
                                   so a cap below the SM count leaves SMs to kernels running on other streams - the
                                   paper starts its migration on a side stream once enough SMs are free (Sec. 3.1,
                                   Improvement 2) */
    AMOEBA_OPT_WAIT_TRIES = 9,  /* bulk-copy paths: value v > 0 makes every wait of a kernel on one of its own copies give
                                   up after v - 1 non-blocking polls and report AMOEBA_ERR_TIMEOUT (0 = the default,
                                   generous budget).  For tests of the give-up path: v = 1 gives up at once, so healthy
                                   copies time out, every time. */
    AMOEBA_OPT_L2_PROMOTION = 10, /* tensor-map copies of token-first pools: L2 promotion of the maps, 1 = none, 2 = 64 B,
                                   3 = 128 B, 4 = 256 B */
    AMOEBA_OPT_PAIR_ORDER = 11, /* order of the pair list the table calls write: 1 = table order (entry k = the k-th
                                   block), 2 = ascending by destination id (the out-of-place KV copy then writes every
                                   destination pool front to back, which DRAM rewards with 1 - 2 %; the in-place reshape
                                   measured 2 % slower with it), 0 = default: 2 for amoeba_rewrite_block_tables, 1 for
                                   amoeba_reshape_block_tables */
    AMOEBA_OPT_WEIGHTS_ONLY = 16,
    AMOEBA_OPT_KV_ONLY = 32
};
AMOEBA_API amoeba_status amoeba_plan_set_option(amoeba_plan* plan, int32_t option, int64_t value);

/*
 * amoeba_rewrite_block_tables  (destination block bookkeeping: Sec. 3.1, the reserved pages each worker prepares
 * for the KV it receives; the paper gives no order, the one used is stated below)
 *
 * Sequence s needs nblk[s] = ceil(seq_lens[s] / block_tokens) blocks.  Walking sequences in index order and their
 * blocks in logical order, the k-th block overall gets the k-th id of the ordered destination free list - the list
 * d_dst_free_list[n_free_or_nb] as given, or, if that is NULL, the ascending ids whose byte in
 * d_dst_free_mask[n_free_or_nb] is non-zero (the mask covers the whole destination pool).  Exactly one of the two
 * is non-NULL.
 *
 * in  d_src_bt   int32 [num_seqs][max_blocks_per_seq], entries past a sequence's blocks are -1
 *     d_seq_lens int32 [num_seqs]
 * out d_dst_bt   int32 [num_seqs][max_blocks_per_seq], fully written, -1 past each sequence's blocks
 *     d_pairs    int32 [pairs_cap][2]: one (source block, destination block) entry per block, a work list for
 *                amoeba_reshard_kv.  By default the entries are ascending by destination id, and the entries of
 *                blocks that were given no destination id - (-1,-1) - close the list; with AMOEBA_OPT_PAIR_ORDER = 1
 *                entry k belongs to the k-th block in (sequence, block) order.  A block with a destination but a
 *                bad source id has (-1,-1) in its place in either order.
 *     d_num_pairs, d_dst_free_count_out  int32 scalars: number of pairs, free blocks left
 *     d_status   int32 scalar, sticky (see conventions)
 * d_workspace: scratch of at least amoeba_rewrite_workspace_bytes(...) bytes, 16-byte aligned, contents irrelevant
 *     before and after; calls that overlap on the GPU need separate workspaces.  Its size depends on num_seqs and on
 *     the plan's block counts (n_free_or_nb is only range-checked).
 *
 * Device-detected errors.  Whole call (d_dst_bt all -1, 0 pairs, free count unchanged): a negative length or a
 * sequence needing more than max_blocks_per_seq blocks, or more blocks than pairs_cap -> INVALID_ARG; more blocks
 * than free blocks -> NO_FREE_BLOCKS.  Per block -> BAD_BLOCK_ID: a free id outside [0, dst num_blocks), or one that
 * an earlier block (in sequence, block order) of this call was already given - a free list that names an id twice -
 * gives table entry -1 and pair (-1,-1); a source id outside [0, src num_blocks) keeps the table entry, pair (-1,-1).
 * Host-detected: INVALID_ARG (null pointers, negative sizes, both or neither free form), ALIGNMENT, CUDA.
 */
AMOEBA_API amoeba_status amoeba_rewrite_workspace_bytes(const amoeba_plan* plan, int32_t num_seqs, int32_t n_free_or_nb,
                                             int64_t* bytes);
AMOEBA_API amoeba_status amoeba_rewrite_block_tables(const amoeba_plan* plan, const int32_t* d_src_bt, const int32_t* d_seq_lens,
                                          int32_t num_seqs, int32_t max_blocks_per_seq,
                                          const int32_t* d_dst_free_list, const uint8_t* d_dst_free_mask,
                                          int32_t n_free_or_nb, int32_t* d_dst_bt, int32_t* d_pairs,
                                          int32_t pairs_cap, int32_t* d_num_pairs, int32_t* d_dst_free_count_out,
                                          int32_t* d_status, void* d_workspace, int64_t workspace_bytes,
                                          void* cuda_stream);

/*
 * amoeba_rewrite_block_tables_builtin_scratch  (no counterpart in the paper: a packaging variant of the call above)
 *
 * Same computation, same arguments and same outputs as amoeba_rewrite_block_tables, minus the workspace: the scratch
 * the two kernels need lives in an array that is part of the library's device image instead of being supplied by the
 * caller.  It exists for callers that must not, or cannot, allocate device memory at the point where a
 * transformation is triggered: a serving process whose memory pool has already claimed the whole GPU for weights and
 * KV blocks (so a cudaMalloc would fail or fragment the pool), code running inside a region where allocation is
 * forbidden by the host framework, or a plug-in that is handed buffers and a stream but no allocator.  This call
 * performs no cudaMalloc / cudaFree and calls no allocating routine of any library.
 *
 * Limit: the scratch array is AMOEBA_BUILTIN_SCRATCH_BYTES (1 MiB) per GPU, held by every GPU that loads the library
 * until the process exits.  It must cover amoeba_rewrite_workspace_bytes(...), i.e. roughly num_seqs + twice the larger
 * of the plan's two block counts <= 262 000 entries, in either free-block form; larger problems are refused with
 * AMOEBA_ERR_TOO_LARGE and nothing is launched - use amoeba_rewrite_block_tables with your own workspace for those.
 *
 * First use on a device: the first call made while a given device is current looks up that device's address of the
 * array (one cudaGetSymbolAddress, checked; AMOEBA_ERR_CUDA if it fails, with the runtime's error state cleared) and
 * remembers it per device ordinal (up to 64 ordinals; beyond that AMOEBA_ERR_UNSUPPORTED).  Make that first call
 * during start-up, outside any stream capture; later calls on the device only launch the kernels.  The remembered
 * address is the one of the device's primary context at that time: after a cudaDeviceReset of the device it is
 * stale, so a process that resets a device must not use this entry point on it afterwards.
 *
 * Sharing: all calls on one GPU use the same array, and it keeps whatever the previous call left in it.  Nothing in
 * it has to start at zero (the kernels write every word before reading it), so no clearing is needed; but two calls
 * whose kernels can overlap on the GPU (different streams without an ordering between them, or different threads or
 * processes' worth of streams on one context) race on it and produce garbage.  Order such calls on one stream, or
 * with events, or give the concurrent ones their own workspace through amoeba_rewrite_block_tables.
 */
enum { AMOEBA_BUILTIN_SCRATCH_BYTES = 1 << 20 };
AMOEBA_API amoeba_status amoeba_rewrite_block_tables_builtin_scratch(
    const amoeba_plan* plan, const int32_t* d_src_bt, const int32_t* d_seq_lens, int32_t num_seqs,
    int32_t max_blocks_per_seq, const int32_t* d_dst_free_list, const uint8_t* d_dst_free_mask, int32_t n_free_or_nb,
    int32_t* d_dst_bt, int32_t* d_pairs, int32_t pairs_cap, int32_t* d_num_pairs, int32_t* d_dst_free_count_out,
    int32_t* d_status, void* cuda_stream);

/*
 * amoeba_reshard_kv  (KV cache migration in the head dimension, Sec. 3.1: every header of every live block moves
 * from the source worker that holds it to the destination worker that keeps it; here as an on-GPU gather/scatter)
 *
 * For every pair k < min(*d_num_pairs, pairs_cap) with both ids >= 0, every layer in [layer_begin, layer_end) and
 * every K/V header h: the 2*block_tokens*head_dim elements of (block, header) are copied from
 * src_pools[h / (Hkv/a)] to dst_pools[h / (Hkv/b)], read at the addresses of the source layout's kv_order and
 * written at those of the destination layout's kv_order.
 * src_pools / dst_pools are HOST arrays of a / b device pointers (read during the call only).
 * A pair with an id outside its pool is skipped and sets BAD_BLOCK_ID in *d_status.  The list may be in any order -
 * the result is the same - provided no destination id appears twice (amoeba_rewrite_block_tables never lists one
 * twice); the order only decides in which order DRAM is visited (see AMOEBA_OPT_PAIR_ORDER).
 */
AMOEBA_API amoeba_status amoeba_reshard_kv(const amoeba_plan* plan, const void* const* src_pools, void* const* dst_pools,
                                const int32_t* d_pairs, const int32_t* d_num_pairs, int32_t pairs_cap,
                                int32_t layer_begin, int32_t layer_end, int32_t* d_status, void* cuda_stream);

/*
 * In-place block reshaping of ONE instance  (Sec. 3.1, "Improvement 1": a worker retains the headers the new TP degree
 * gives it where they are; the room the migrated headers leave inside a block is reused by reshaping the block)
 *
 * Split: the plan's source layout is the instance at TP = a with NB blocks, the destination layout the same instance
 * at TP = N*a with NB*N blocks; merge back: the other way round (source TP = N*a with NB*N blocks, destination TP = a
 * with NB).  Both header-centric, same layer stride; anything else is UNSUPPORTED.  The header ranges are contiguous,
 * so worker r of TP = a holds the headers of workers r*N .. r*N+N-1 of TP = N*a; the paper names no numbering and
 * this one is used: worker r becomes worker r*N, and block p becomes block p*N on every worker (the block table stays
 * shared).  In worker r's memory, read as NB*N blocks of Hkv/(N*a) headers, block p*N is exactly the retained N-th
 * of old block p: it does not move.  The other N-1 header groups go to block p*N of workers r*N+1 .. r*N+N-1, whose
 * pools have the same capacity and are otherwise untouched.  Afterwards every id that is not p*N for a live p is
 * free - the ids p*N+1 .. p*N+N-1 are the segments the migrated headers left.  (N-1)/N of the live bytes move and
 * the retained workers need no second pool.  The merge back brings the groups home: only blocks whose id is a
 * multiple of N can be reshaped (the caller first renumbers other blocks with amoeba_rewrite_block_tables /
 * amoeba_reshard_kv inside the TP = N*a pools, using free ids q = 0 mod N whose followers q+1 .. q+N-1 are free too).
 *
 * amoeba_reshape_block_tables: same inputs as amoeba_rewrite_block_tables without a free list.  Writes d_dst_bt
 * (p -> p*N, or q -> q/N; -1 past each sequence's blocks), the pair list (old id, new id) - entry k = the k-th block in
 * (sequence, block) order unless AMOEBA_OPT_PAIR_ORDER = 2 asks for destination order as described above -,
 * d_dst_free_mask_out: uint8 [destination num_blocks], 1 = free afterwards, and the free count.  Workspace as for
 * amoeba_rewrite_block_tables.  Device-detected errors: whole call as there (no NO_FREE_BLOCKS); per block ->
 * BAD_BLOCK_ID, table entry -1, pair (-1,-1), block not moved: an id outside the source pool, -1 inside a sequence,
 * an id an earlier block already named, and for the merge an id that is not a multiple of N.
 *
 * amoeba_reshape_kv_inplace: pools is a HOST array of N*a device pointers, pools[w] = worker w of the TP = N*a side;
 * worker r of the TP = a side is pools[r*N].  All distinct.  For every pair (both ids >= 0), layer and header group
 * k = 1 .. N-1 the group's bytes are copied between pools[r*N] and pools[r*N+k]; nothing is written into a pool
 * that the same call reads (split: the old workers are only read; merge: they are only written), so no ordering
 * between work items is needed.  A pair whose ids are not (p, p*N) resp. (q, q/N) is skipped with BAD_BLOCK_ID.
 * All three copy paths apply.  amoeba_reshape_bytes: bytes read + written for n_live_blocks blocks over all layers.
 */
AMOEBA_API amoeba_status amoeba_reshape_block_tables(const amoeba_plan* plan, const int32_t* d_src_bt,
                                          const int32_t* d_seq_lens, int32_t num_seqs, int32_t max_blocks_per_seq,
                                          int32_t* d_dst_bt, int32_t* d_pairs, int32_t pairs_cap, int32_t* d_num_pairs,
                                          uint8_t* d_dst_free_mask_out, int32_t* d_dst_free_count_out,
                                          int32_t* d_status, void* d_workspace, int64_t workspace_bytes,
                                          void* cuda_stream);
AMOEBA_API amoeba_status amoeba_reshape_kv_inplace(const amoeba_plan* plan, void* const* pools, const int32_t* d_pairs,
                                        const int32_t* d_num_pairs, int32_t pairs_cap, int32_t layer_begin,
                                        int32_t layer_end, int32_t* d_status, void* cuda_stream);
AMOEBA_API amoeba_status amoeba_reshape_bytes(const amoeba_plan* plan, int64_t n_live_blocks, int64_t* kv_bytes_rw);

/*
 * In-place merge of N instances of TP = a into one instance of TP = N*a  (Sec. 3.1, "Improvement 1": in-place
 * migration with the header-centric layout; the freed parts of a block are reused through block reshaping)
 *
 * The plan's source layout describes every one of the N instances (tp = a, num_blocks = NB); its destination layout
 * describes the merged instance: tp = N*a, num_blocks = NB*N, same model, block_tokens and layer stride; both
 * header-centric (with the token-first order the retained headers of a block are not one segment: UNSUPPORTED, as
 * the paper argues).  Every worker keeps its memory: pools[i*a + r], before the call the pool of worker r of instance
 * i with NB blocks of Hkv/a headers, is after the call the pool of worker r*N+i of the merged instance with NB*N
 * blocks of Hkv/(N*a) headers.  Block p of instance i becomes block p*N+i of the merged instance; on the worker that
 * retains its headers that is the same memory, so those bytes do not move.  The paper gives no numbering; this one
 * keeps the block table shared by all workers and needs no free list.
 *
 * amoeba_merge_block_tables: d_src_bt int32 [N][num_seqs][max_blocks_per_seq] and d_seq_lens int32 [N][num_seqs] are
 * the N instances' tables (an instance with fewer sequences pads with length 0).  Writes d_dst_bt (same shape:
 * entry p -> p*N+i, -1 past each sequence's blocks) and d_live: uint8 [N][NB] rounded up to a multiple of 16 bytes
 * (amoeba_merge_live_bytes), 1 for every block an instance's table names, which amoeba_merge_kv_inplace reads.
 * Device-detected errors: a negative length or a sequence needing more than max_blocks_per_seq blocks -> whole call
 * INVALID_ARG (d_dst_bt all -1, d_live all 0, so nothing moves); an id outside [0, NB) or -1 inside a sequence ->
 * BAD_BLOCK_ID, table entry -1, block not moved; an id named twice by one instance -> BAD_BLOCK_ID, moved once.
 *
 * amoeba_merge_kv_inplace: pools is a HOST array of N*a device pointers.  For every layer in [layer_begin, layer_end),
 * every old block id p and every two instances i != k, the headers of block p that instance i's worker r holds for
 * merged worker r*N+k move to that worker's memory (pools[k*a + r]), into the place of the headers it gives up for
 * worker r*N+i; where both blocks are live the two segments are exchanged through shared memory (both are read
 * completely before either is written), where one is live it is copied, where neither is nothing happens.  Bytes of
 * blocks no table names, and vacated segments nothing is received into, keep their values.  Moves (N-1)/N of the live
 * bytes and needs no second pool.  The vector load/store copy path does not apply; the bulk-copy rings are used.
 */
AMOEBA_API amoeba_status amoeba_merge_live_bytes(const amoeba_plan* plan, int64_t* bytes);
AMOEBA_API amoeba_status amoeba_merge_block_tables(const amoeba_plan* plan, const int32_t* d_src_bt, const int32_t* d_seq_lens,
                                        int32_t num_seqs, int32_t max_blocks_per_seq, int32_t* d_dst_bt,
                                        uint8_t* d_live, int32_t* d_status, void* cuda_stream);
AMOEBA_API amoeba_status amoeba_merge_kv_inplace(const amoeba_plan* plan, void* const* pools, const uint8_t* d_live,
                                      int32_t layer_begin, int32_t layer_end, int32_t* d_status, void* cuda_stream);
/*
 * amoeba_split_block_tables  (the way back: Sec. 3.3's scale-down, where the KV cache is transformed first so that
 * every new instance holds all headers of its own requests; in place, with the same plan as the merge)
 *
 * One instance of TP = N*a becomes N instances of TP = a on the same memory.  d_merged_bt int32
 * [N][num_seqs][max_blocks_per_seq], d_seq_lens int32 [N][num_seqs]: row block i = the merged instance's table rows
 * of the requests that go to instance i.  A block with merged id q = p*N+i can only go to instance i and becomes its
 * block p; blocks with other ids are first renumbered by the caller with amoeba_rewrite_block_tables /
 * amoeba_reshard_kv inside the merged pools, using a free list of ids = i (mod N).  Writes d_inst_bt (q -> q/N, -1
 * past each sequence's blocks) and d_live as amoeba_merge_block_tables does; an id outside [0, NB*N) or with q mod N
 * != i is BAD_BLOCK_ID (entry -1, block not moved).
 *
 * amoeba_split_kv_inplace: same arguments as amoeba_merge_kv_inplace, with the live marks of
 * amoeba_split_block_tables; pools[i*a + r] is merged worker r*N+i before and worker r of instance i after.  Where
 * both blocks of a pair are live the two segments are exchanged exactly as in the merge; where one is live the
 * direction is the opposite one: the live block of instance i fetches its headers from the other worker.
 */
AMOEBA_API amoeba_status amoeba_split_block_tables(const amoeba_plan* plan, const int32_t* d_merged_bt, const int32_t* d_seq_lens,
                                        int32_t num_seqs, int32_t max_blocks_per_seq, int32_t* d_inst_bt,
                                        uint8_t* d_live, int32_t* d_status, void* cuda_stream);
AMOEBA_API amoeba_status amoeba_split_kv_inplace(const amoeba_plan* plan, void* const* pools, const uint8_t* d_live,
                                      int32_t layer_begin, int32_t layer_end, int32_t* d_status, void* cuda_stream);
/* Bytes read + written by amoeba_merge_kv_inplace when n_live_blocks old blocks (summed over the instances) are
 * live, over all layers: 2 * (N-1)/N of their size. */
AMOEBA_API amoeba_status amoeba_merge_bytes(const amoeba_plan* plan, int64_t n_live_blocks, int64_t* kv_bytes_rw);

/*
 * amoeba_reshard_weights  (model weight transformation, Sec. 3.2: the copy that re-partitions the weights; Eq. 1
 * fixes which rows / columns each worker holds)
 *
 * src is a HOST array [a][num_layers] (worker-major) of device pointers, dst likewise [b][num_layers]; only layers
 * in [layer_begin, layer_end) are read.  Either side may be padded (weight_pad_parts): padded -> padded moves whole
 * partitions, dense <-> padded changes the pitch; pad bytes of the destination keep their values (zero them once at
 * load time if a GEMM is to run over a whole padded buffer, Eq. 2).  A destination worker whose seven pointers are all
 * NULL in a layer is left out: its shard is not produced (a worker that only needs its own new shard, as each worker
 * of a merge does, passes the others as NULL).  Any other NULL pointer a descriptor needs is INVALID_ARG.  A caller transforming a few layers per inference step (Sec. 3.3's
 * layer-by-layer order) passes successive ranges.
 */
AMOEBA_API amoeba_status amoeba_reshard_weights(const amoeba_plan* plan, const amoeba_layer_weights* src,
                                     const amoeba_layer_weights* dst, int32_t layer_begin, int32_t layer_end,
                                     int32_t* d_status, void* cuda_stream);

/*
 * amoeba_compact_weights_inplace  (Sec. 3.2, base solution "partial swap": the part of a shard a worker keeps is moved
 * to the start of the layer's weight space so that the rest can be released; the paper does it with a blocking copy)
 *
 * The plan's source layout is the instance before (TP = a), its destination layout the instance after (TP = N*a);
 * both dense (no padding), same fused flags.  bufs is a HOST array [a][num_layers] of the a workers' buffers;
 * keep[r] in [0, N) (host array) says which N-th of its shards worker r keeps: it becomes worker r*N + keep[r] of the
 * new partition.  After the call the first bytes of every buffer hold exactly that worker's dense TP = N*a shard
 * (the same bytes amoeba_reshard_weights writes for that worker); the bytes behind it are unspecified leftovers.
 * No second buffer is used; about 1/N of the weights is read and written (what already sits where it belongs - with
 * keep[r] = 0 the first section of every buffer and row 0 of o_proj / down_proj - is not touched).  The moves are
 * ordered on the stream so that no byte is overwritten before it has been moved: one small launch for the first rows
 * of o_proj / down_proj, then log_N(hidden) - 2 or so launches of the copy kernel (4 for N = 4, 7 for N = 2 at
 * hidden = 4096).  Errors: INVALID_ARG (null pointers, keep out of range, layers), UNSUPPORTED (padded layouts,
 * different fused flags, TP not a multiple), ALIGNMENT, CUDA, NO_MEMORY.
 * amoeba_compact_bytes: the bytes the call reads + writes over all layers for the given keep[] (host arithmetic).
 */
AMOEBA_API amoeba_status amoeba_compact_weights_inplace(const amoeba_plan* plan, const amoeba_layer_weights* bufs,
                                             const int32_t* keep, int32_t layer_begin, int32_t layer_end,
                                             int32_t* d_status, void* cuda_stream);
AMOEBA_API amoeba_status amoeba_compact_bytes(const amoeba_plan* plan, const int32_t* keep, int64_t* bytes_rw);

/*
 * amoeba_plan_weight_alias  (Sec. 3.2, Improvement 1: with padded partitions a scale-up needs no weight copy at all)
 *
 * When both layouts are padded with the same weight_pad_parts, page size and fused flags and the destination TP is a
 * multiple of the source TP, the buffer `tensor` of destination worker dst_rank is, byte for byte (pads included),
 * the range [*src_offset, *src_offset + *bytes) of the same buffer of source worker *src_rank: the worker that keeps
 * those pages can use them where they are and release the others, instead of calling amoeba_reshard_weights.
 * Host arithmetic only.  Errors: INVALID_ARG; UNSUPPORTED when the layouts do not allow it (a copy is needed).
 */
AMOEBA_API amoeba_status amoeba_plan_weight_alias(const amoeba_plan* plan, int32_t dst_rank, int32_t tensor,
                                       int32_t* src_rank, int64_t* src_offset, int64_t* bytes);

/* Number of kernels the library has launched in this process (for launch accounting in benchmarks). */
AMOEBA_API int64_t amoeba_launch_count(void);

AMOEBA_API const char* amoeba_status_string(amoeba_status s);

#ifdef __cplusplus
}
#endif
#endif /* AMOEBA_H_ */
