// Host planner of the TP a->b re-layout: validates the two layouts and derives, from the partition rules
// (K/V headers per worker: Sec. 3.1 "Base solution"; weight rows / columns per worker: Sec. 3.2, Eq. 1),
// which byte ranges go from which source worker to which destination worker.  No CUDA in this file.
#include <algorithm>
#include <atomic>
#include <new>
#include <numeric>

#include "plan.hpp"

namespace amoeba {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static bool same_model(const amoeba_model& x, const amoeba_model& y) {
    return x.num_layers == y.num_layers && x.hidden == y.hidden && x.num_q_heads == y.num_q_heads &&
           x.num_kv_heads == y.num_kv_heads && x.head_dim == y.head_dim && x.intermediate == y.intermediate &&
           x.elem_bytes == y.elem_bytes;
}

static amoeba_status check_layout(const amoeba_layout& l) {
    const amoeba_model& m = l.model;
    if (m.num_layers <= 0 || m.hidden <= 0 || m.num_q_heads <= 0 || m.num_kv_heads <= 0 || m.head_dim <= 0 ||
        m.intermediate <= 0 || l.tp <= 0 || l.block_tokens <= 0 || l.num_blocks <= 0 || l.kv_layer_stride_bytes < 0)
        return AMOEBA_ERR_INVALID_ARG;
    if (m.elem_bytes != 1 && m.elem_bytes != 2 && m.elem_bytes != 4) return AMOEBA_ERR_UNSUPPORTED;
    if (l.kv_order != AMOEBA_KV_HEAD_MAJOR && l.kv_order != AMOEBA_KV_TOKEN_MAJOR) return AMOEBA_ERR_UNSUPPORTED;
    if (l.tp > AMOEBA_MAX_TP) return AMOEBA_ERR_UNSUPPORTED;
    // Even partition of the headers and of the FFN width over the workers; K/V header replication for
    // tp > num_kv_heads is not a re-layout of existing state and is not handled.
    if (m.num_q_heads % l.tp || m.num_kv_heads % l.tp || m.intermediate % l.tp) return AMOEBA_ERR_UNSUPPORTED;
    if (m.num_q_heads % m.num_kv_heads) return AMOEBA_ERR_UNSUPPORTED;
    if (l.weight_pad_parts < 0 || l.weight_page_bytes < 0) return AMOEBA_ERR_INVALID_ARG;
    if (l.weight_pad_parts > 0) {
        const int P = l.weight_pad_parts;
        if (P > 4 * AMOEBA_MAX_TP || P % l.tp || m.num_q_heads % P || m.num_kv_heads % P || m.intermediate % P)
            return AMOEBA_ERR_UNSUPPORTED;
        if (l.weight_page_bytes % 16) return AMOEBA_ERR_ALIGNMENT;
    }
    return AMOEBA_OK;
}

// ---- how one layout stores the weights: every buffer is `parts` partitions, `per_worker` of them per worker, each
// `block` bytes at a pitch of `pitch` bytes (dense shards: one partition per worker, parts = tp).
constexpr int64_t kDefaultPageBytes = 2 << 20;
enum { Q, K, V, O, GATE, UP, DOWN };

struct WeightForm {
    int parts, per_worker;
    int64_t page;
    int64_t block[kNumTensors], pitch[kNumTensors];  // per buffer (0 for a member folded into a fused buffer)
    int buffer_of[kNumTensors];                      // buffer that holds the member
    int64_t member_off[kNumTensors];                 // byte offset of the member inside a partition of its buffer
};

static WeightForm weight_form(const amoeba_layout& l) {
    const amoeba_model& m = l.model;
    WeightForm f{};
    const bool padded = l.weight_pad_parts > 0;
    f.parts = padded ? l.weight_pad_parts : l.tp;
    f.per_worker = f.parts / l.tp;
    f.page = padded ? (l.weight_page_bytes ? l.weight_page_bytes : kDefaultPageBytes) : 1;
    const int64_t e = m.elem_bytes, hid = m.hidden;
    const int64_t q = (int64_t)m.num_q_heads * m.head_dim / f.parts * hid * e;
    const int64_t kv = (int64_t)m.num_kv_heads * m.head_dim / f.parts * hid * e;
    const int64_t ffn = (int64_t)m.intermediate / f.parts * hid * e;
    for (int t = 0; t < kNumTensors; ++t) f.buffer_of[t] = t;
    f.block[Q] = q, f.block[K] = f.block[V] = kv, f.block[O] = q, f.block[GATE] = f.block[UP] = f.block[DOWN] = ffn;
    if (l.fused_qkv) {
        f.block[Q] = q + 2 * kv, f.block[K] = f.block[V] = 0;
        f.buffer_of[K] = f.buffer_of[V] = Q;
        f.member_off[K] = q, f.member_off[V] = q + kv;
    }
    if (l.fused_gate_up) {
        f.block[GATE] = 2 * ffn, f.block[UP] = 0;
        f.buffer_of[UP] = GATE;
        f.member_off[UP] = ffn;
    }
    for (int t = 0; t < kNumTensors; ++t) f.pitch[t] = (f.block[t] + f.page - 1) / f.page * f.page;
    return f;
}

// Largest divisor d of `total` with d <= cap and d % 16 == 0 (total % 16 == 0 is a precondition).
static int64_t chunk_of(int64_t total, int64_t cap) {
    for (int64_t n = std::max<int64_t>(1, (total + cap - 1) / cap); n <= total / 16; ++n)
        if (total % n == 0 && (total / n) % 16 == 0) return total / n;
    return 16;
}

// One public descriptor in kernel form: long rows are cut into column chunks of at most `cap` bytes, short rows are
// grouped so that a work item is at most `cap` bytes.  *item counts the work items so far.
WDescDev chunk_desc(const amoeba_weight_desc& d, int64_t cap, int64_t* item) {
    WDescDev w{};
    w.src_off = d.src_off;
    w.dst_off = d.dst_off;
    w.src_pitch = d.src_pitch;
    w.dst_pitch = d.dst_pitch;
    w.row_bytes = d.row_bytes;
    w.n_rows = d.n_rows;
    w.src_slot = d.src_rank * kNumTensors + d.src_tensor;
    w.dst_slot = d.dst_rank * kNumTensors + d.dst_tensor;
    if (d.row_bytes > cap) {  // cut a long row into the fewest chunks of (nearly) equal size
        w.rows_per_item = 1;
        w.col_chunks = (int32_t)((d.row_bytes + cap - 1) / cap);
        w.chunk_bytes = (int32_t)(((d.row_bytes + w.col_chunks - 1) / w.col_chunks + 15) / 16 * 16);
    } else {
        w.rows_per_item = (int32_t)std::min<int64_t>(std::max<int64_t>(1, cap / d.row_bytes), d.n_rows);
        w.col_chunks = 1;
        w.chunk_bytes = (int32_t)d.row_bytes;
    }
    w.item_begin = (int32_t)*item;
    *item += (int64_t)((d.n_rows + w.rows_per_item - 1) / w.rows_per_item) * w.col_chunks;
    return w;
}

amoeba_status finalize_chunks(amoeba_plan* p) {
    const int64_t kv_cap = p->opt.kv.chunk_bytes > 0 ? p->opt.kv.chunk_bytes : kDefaultKvChunk;
    const int64_t cap = p->opt.w.chunk_bytes > 0 ? p->opt.w.chunk_bytes : kDefaultWChunk;
    if (cap < 16 || cap % 16 || kv_cap < 16 || kv_cap % 16) return AMOEBA_ERR_INVALID_ARG;
    // KV work items: cut a unit's rows into column chunks (long rows) or group whole rows (short rows).
    KvGeom& g = p->kv;
    const bool src_tok = p->src.kv_order == AMOEBA_KV_TOKEN_MAJOR, dst_tok = p->dst.kv_order == AMOEBA_KV_TOKEN_MAJOR;
    const int32_t T = p->src.block_tokens;
    if (!src_tok && !dst_tok) {  // a run of headers with K and V is contiguous on both sides
        g.planes = 1;
        g.heads_per_unit = p->heads_per_run;
        g.rows = 1;
        g.row_bytes = p->run_bytes;
        g.src_row_pitch = g.dst_row_pitch = p->run_bytes;
    } else {
        g.planes = 2;
        g.heads_per_unit = (src_tok && dst_tok) ? p->heads_per_run : 1;
        g.rows = T;
        g.row_bytes = g.heads_per_unit * p->vec_bytes;
        g.src_row_pitch = src_tok ? p->heads_src * p->vec_bytes : p->vec_bytes;
        g.dst_row_pitch = dst_tok ? p->heads_dst * p->vec_bytes : p->vec_bytes;
    }
    g.head_units = p->src.model.num_kv_heads / g.heads_per_unit;
    if (g.row_bytes > kv_cap) {
        g.rows_per_item = 1;
        g.chunk_bytes = (int32_t)chunk_of(g.row_bytes, kv_cap);
        g.col_chunks = (int32_t)(g.row_bytes / g.chunk_bytes);
    } else {
        g.rows_per_item = (int32_t)std::min<int64_t>(g.rows, std::max<int64_t>(1, kv_cap / g.row_bytes));
        g.chunk_bytes = (int32_t)g.row_bytes;
        g.col_chunks = 1;
    }
    g.row_groups = (g.rows + g.rows_per_item - 1) / g.rows_per_item;
    g.item_bytes = (int64_t)g.rows_per_item * g.chunk_bytes;
    p->chunk_bytes = g.item_bytes;

    // Box items for the tensor-map path (only meaningful when a side is token-first).
    KvBoxGeom& bx = p->kvbox;
    bx = KvBoxGeom{};
    const int32_t D = p->src.model.head_dim;
    if ((src_tok || dst_tok) && D <= 256 && p->vec_bytes % 16 == 0) {
        bx.usable = 1;
        auto largest_divisor = [](int64_t n, int64_t limit) {
            int64_t best = 1;
            for (int64_t d = 1; d <= n && d <= limit; ++d)
                if (n % d == 0) best = d;
            return best;
        };
        if (p->unit_bytes <= kv_cap) {
            bx.tokens = T;
            bx.heads = (int32_t)largest_divisor(p->heads_per_run, std::min<int64_t>(128, kv_cap / p->unit_bytes));
        } else {
            bx.heads = 1;
            bx.tokens = (int32_t)largest_divisor(T, std::min<int64_t>(256, std::max<int64_t>(1, kv_cap / (2 * p->vec_bytes))));
        }
        if (T > 256 && bx.tokens == T) bx.tokens = (int32_t)largest_divisor(T, 256);
        bx.sub_runs = p->heads_per_run / bx.heads;
        bx.tok_groups = T / bx.tokens;
        bx.item_bytes = 2 * (int64_t)bx.heads * bx.tokens * p->vec_bytes;
    }
    p->wdev.clear();
    int64_t item = 0;
    for (const amoeba_weight_desc& d : p->wdescs) {
        p->wdev.push_back(chunk_desc(d, cap, &item));
        if (item > INT32_MAX) return AMOEBA_ERR_UNSUPPORTED;
    }
    p->items_per_layer = (int32_t)item;
    return AMOEBA_OK;
}

int merge_instances(const amoeba_plan* p) {
    const amoeba_layout &s = p->src, &d = p->dst;
    if (s.kv_order != AMOEBA_KV_HEAD_MAJOR || d.kv_order != AMOEBA_KV_HEAD_MAJOR) return 0;
    if (d.tp % s.tp) return 0;
    const int64_t n = d.tp / s.tp;
    if (n < 2 || (int64_t)d.num_blocks != (int64_t)s.num_blocks * n) return 0;
    if (p->src_layer_stride != p->dst_layer_stride) return 0;
    return (int)n;
}

int reshape_factor(const amoeba_plan* p) {
    const amoeba_layout &s = p->src, &d = p->dst;
    if (s.kv_order != AMOEBA_KV_HEAD_MAJOR || d.kv_order != AMOEBA_KV_HEAD_MAJOR) return 0;
    if (p->src_layer_stride != p->dst_layer_stride) return 0;
    if (d.tp > s.tp && d.tp % s.tp == 0 && (int64_t)d.num_blocks == (int64_t)s.num_blocks * (d.tp / s.tp))
        return d.tp / s.tp;
    if (s.tp > d.tp && s.tp % d.tp == 0 && (int64_t)s.num_blocks == (int64_t)d.num_blocks * (s.tp / d.tp))
        return -(s.tp / d.tp);
    return 0;
}

struct Range {
    int64_t lo, hi;
};
static Range part(int64_t total, int tp, int r) { return {total / tp * r, total / tp * (r + 1)}; }

// Descriptors of one weight member between two forms.  The member has `units` rows (split_rows) or columns along
// its partition axis; partition p of a form covers units [p*units/parts, (p+1)*units/parts) and lives in worker
// p / per_worker at byte (p % per_worker) * pitch + member_off of the member's buffer.  Every intersection of a source
// partition with a destination partition is one copy: contiguous for a row split (unit_bytes = bytes of one row),
// `rows` strided runs for a column split (unit_bytes = bytes of one element), contiguous again when the common range
// is a whole partition on both sides.
static void add_member(std::vector<amoeba_weight_desc>& out, const WeightForm& fs, const WeightForm& fd, int member,
                       int64_t units, int64_t unit_bytes, bool split_rows, int64_t rows) {
    const int bs = fs.buffer_of[member], bd = fd.buffer_of[member];
    for (int ps = 0; ps < fs.parts; ++ps)
        for (int pd = 0; pd < fd.parts; ++pd) {
            const Range s = part(units, fs.parts, ps), d = part(units, fd.parts, pd);
            const int64_t lo = std::max(s.lo, d.lo), hi = std::min(s.hi, d.hi);
            if (lo >= hi) continue;
            amoeba_weight_desc w{};
            w.src_rank = ps / fs.per_worker;
            w.dst_rank = pd / fd.per_worker;
            w.src_tensor = bs;
            w.dst_tensor = bd;
            const int64_t sbase = (ps % fs.per_worker) * fs.pitch[bs] + fs.member_off[member];
            const int64_t dbase = (pd % fd.per_worker) * fd.pitch[bd] + fd.member_off[member];
            w.src_off = sbase + (lo - s.lo) * unit_bytes;
            w.dst_off = dbase + (lo - d.lo) * unit_bytes;
            w.row_bytes = (hi - lo) * unit_bytes;
            if (split_rows) {  // consecutive rows are one contiguous run
                w.n_rows = 1;
                w.src_pitch = w.dst_pitch = w.row_bytes;
            } else {
                w.n_rows = (int32_t)rows;
                w.src_pitch = (s.hi - s.lo) * unit_bytes;
                w.dst_pitch = (d.hi - d.lo) * unit_bytes;
                if (w.src_pitch == w.row_bytes && w.dst_pitch == w.row_bytes) {  // whole partition on both sides
                    w.row_bytes *= rows;
                    w.n_rows = 1;
                    w.src_pitch = w.dst_pitch = w.row_bytes;
                }
            }
            // Fold an arithmetic progression of equal contiguous runs (partition after partition between the same
            // two workers) into one 2-D descriptor.
            if (!out.empty() && w.n_rows == 1) {
                amoeba_weight_desc& p = out.back();
                const bool same = p.src_rank == w.src_rank && p.dst_rank == w.dst_rank && p.src_tensor == w.src_tensor &&
                                  p.dst_tensor == w.dst_tensor && p.row_bytes == w.row_bytes &&
                                  (p.reserved & 255) == member + 1;
                const bool foldable = (p.reserved & 256) != 0;
                if (same && p.n_rows == 1 && w.src_off > p.src_off && w.dst_off > p.dst_off) {
                    p.src_pitch = w.src_off - p.src_off;
                    p.dst_pitch = w.dst_off - p.dst_off;
                    p.n_rows = 2;
                    continue;
                }
                if (same && p.n_rows > 1 && foldable && w.src_off == p.src_off + p.n_rows * p.src_pitch &&
                    w.dst_off == p.dst_off + p.n_rows * p.dst_pitch) {
                    ++p.n_rows;
                    continue;
                }
            }
            w.reserved = (member + 1) | (w.n_rows == 1 ? 256 : 0);  // building notes, cleared by the caller
            out.push_back(w);
        }
}

}  // namespace amoeba

using namespace amoeba;

extern "C" {

static amoeba_status plan_create(const amoeba_layout* src, const amoeba_layout* dst, amoeba_plan** out) {
    amoeba_status st = check_layout(*src);
    if (st != AMOEBA_OK) return st;
    st = check_layout(*dst);
    if (st != AMOEBA_OK) return st;
    if (!same_model(src->model, dst->model) || src->block_tokens != dst->block_tokens) return AMOEBA_ERR_INVALID_ARG;

    amoeba_plan* p = new (std::nothrow) amoeba_plan();
    if (!p) return AMOEBA_ERR_INVALID_ARG;
    p->src = *src;
    p->dst = *dst;
    const amoeba_model& m = src->model;
    const int a = src->tp, b = dst->tp;
    const int64_t e = m.elem_bytes;

    // ---- KV: headers h .. h+g-1 with g = gcd(Hkv/a, Hkv/b) never straddle a worker boundary on either side,
    // so each such group is one contiguous run in the source block and in the destination block.
    p->heads_src = m.num_kv_heads / a;
    p->heads_dst = m.num_kv_heads / b;
    p->heads_per_run = std::gcd(p->heads_src, p->heads_dst);
    p->runs_per_block = m.num_kv_heads / p->heads_per_run;
    p->vec_bytes = (int64_t)m.head_dim * e;
    p->unit_bytes = 2 * (int64_t)src->block_tokens * m.head_dim * e;
    p->run_bytes = p->heads_per_run * p->unit_bytes;
    p->src_block_bytes = p->heads_src * p->unit_bytes;
    p->dst_block_bytes = p->heads_dst * p->unit_bytes;
    const int64_t src_dense = p->src_block_bytes * src->num_blocks, dst_dense = p->dst_block_bytes * dst->num_blocks;
    p->src_layer_stride = src->kv_layer_stride_bytes ? src->kv_layer_stride_bytes : src_dense;
    p->dst_layer_stride = dst->kv_layer_stride_bytes ? dst->kv_layer_stride_bytes : dst_dense;
    if (p->src_layer_stride < src_dense || p->dst_layer_stride < dst_dense) {
        delete p;
        return AMOEBA_ERR_INVALID_ARG;
    }
    const bool any_token_major = src->kv_order == AMOEBA_KV_TOKEN_MAJOR || dst->kv_order == AMOEBA_KV_TOKEN_MAJOR;
    if (p->unit_bytes % 16 || p->src_layer_stride % 16 || p->dst_layer_stride % 16 ||
        (any_token_major && p->vec_bytes % 16)) {
        delete p;
        return AMOEBA_ERR_ALIGNMENT;
    }

    // ---- weights
    const int64_t hid = m.hidden, qrows = (int64_t)m.num_q_heads * m.head_dim,
                  kvrows = (int64_t)m.num_kv_heads * m.head_dim, I = m.intermediate;
    const int64_t rb = hid * e;  // bytes of one [*, hidden] row
    auto& w = p->wdescs;
    const WeightForm fs = weight_form(*src), fd = weight_form(*dst);
    add_member(w, fs, fd, Q, qrows, rb, true, 0);
    add_member(w, fs, fd, K, kvrows, rb, true, 0);
    add_member(w, fs, fd, V, kvrows, rb, true, 0);
    add_member(w, fs, fd, O, qrows, e, false, hid);
    add_member(w, fs, fd, GATE, I, rb, true, 0);
    add_member(w, fs, fd, UP, I, rb, true, 0);
    add_member(w, fs, fd, DOWN, I, e, false, hid);
    for (auto& d : w) d.reserved = 0;
    if ((int)w.size() > kMaxWeightDescs) {
        delete p;
        return AMOEBA_ERR_UNSUPPORTED;
    }
    p->weight_bytes_per_layer = 0;
    for (const auto& d : w) {
        if (d.row_bytes % 16 || d.src_off % 16 || d.dst_off % 16 || d.src_pitch % 16 || d.dst_pitch % 16) {
            delete p;
            return AMOEBA_ERR_ALIGNMENT;
        }
        p->weight_bytes_per_layer += d.row_bytes * d.n_rows;
    }

    st = finalize_chunks(p);
    if (st != AMOEBA_OK) {
        delete p;
        return st;
    }
    *out = p;
    return AMOEBA_OK;
}

// The containers of a plan allocate; an allocation failure is reported as a status, never thrown across the C ABI.
amoeba_status amoeba_plan_create(const amoeba_layout* src, const amoeba_layout* dst, amoeba_plan** out) {
    if (!src || !dst || !out) return AMOEBA_ERR_INVALID_ARG;
    *out = nullptr;
    try {
        return plan_create(src, dst, out);
    } catch (...) {
        return AMOEBA_ERR_NO_MEMORY;
    }
}

void amoeba_plan_destroy(amoeba_plan* plan) { delete plan; }

amoeba_status amoeba_layout_kv_pool_bytes(const amoeba_layout* l, int64_t* bytes) {
    if (!l || !bytes) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_status st = check_layout(*l);
    if (st != AMOEBA_OK) return st;
    const amoeba_model& m = l->model;
    const int64_t dense = (int64_t)l->num_blocks * (m.num_kv_heads / l->tp) * 2 * l->block_tokens * m.head_dim * m.elem_bytes;
    if (l->kv_layer_stride_bytes && l->kv_layer_stride_bytes < dense) return AMOEBA_ERR_INVALID_ARG;
    *bytes = (l->kv_layer_stride_bytes ? l->kv_layer_stride_bytes : dense) * m.num_layers;
    return AMOEBA_OK;
}

amoeba_status amoeba_layout_weight_bytes(const amoeba_layout* l, int32_t tensor, int64_t* bytes) {
    if (!l || !bytes || tensor < 0 || tensor >= kNumTensors) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_status st = check_layout(*l);
    if (st != AMOEBA_OK) return st;
    const WeightForm f = weight_form(*l);
    // dense shards: the one partition; padded: per_worker partitions at the padded pitch
    *bytes = f.block[tensor] ? (l->weight_pad_parts > 0 ? f.per_worker * f.pitch[tensor] : f.block[tensor]) : 0;
    return AMOEBA_OK;
}

amoeba_status amoeba_layout_pad_info(const amoeba_layout* l, int32_t tensor, amoeba_pad_info* out) {
    if (!l || !out || tensor < 0 || tensor >= kNumTensors) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_status st = check_layout(*l);
    if (st != AMOEBA_OK) return st;
    const WeightForm f = weight_form(*l);
    const int64_t page = l->weight_pad_parts > 0 ? f.page : (l->weight_page_bytes ? l->weight_page_bytes : kDefaultPageBytes);
    *out = amoeba_pad_info{};
    out->partitions_per_worker = f.block[tensor] ? f.per_worker : 0;
    out->partition_bytes = f.block[tensor];
    out->pitch_bytes = f.pitch[tensor];
    out->page_bytes = page;
    out->pages = (double)f.block[tensor] / (double)page;
    return AMOEBA_OK;
}

amoeba_status amoeba_plan_bytes(const amoeba_plan* plan, int64_t n_blocks, int64_t* kv_bytes_rw, int64_t* w_bytes_rw) {
    if (!plan || n_blocks < 0) return AMOEBA_ERR_INVALID_ARG;
    const amoeba_model& m = plan->src.model;
    if (kv_bytes_rw) *kv_bytes_rw = 2 * n_blocks * m.num_layers * m.num_kv_heads * plan->unit_bytes;
    if (w_bytes_rw) *w_bytes_rw = 2 * plan->weight_bytes_per_layer * m.num_layers;
    return AMOEBA_OK;
}

amoeba_status amoeba_plan_kv_info(const amoeba_plan* plan, amoeba_kv_info* out) {
    if (!plan || !out) return AMOEBA_ERR_INVALID_ARG;
    out->heads_per_run = plan->heads_per_run;
    out->runs_per_block = plan->runs_per_block;
    out->run_bytes = plan->run_bytes;
    out->chunk_bytes = plan->chunk_bytes;
    out->src_block_bytes = plan->src_block_bytes;
    out->dst_block_bytes = plan->dst_block_bytes;
    out->src_layer_stride = plan->src_layer_stride;
    out->dst_layer_stride = plan->dst_layer_stride;
    return AMOEBA_OK;
}

int32_t amoeba_plan_num_weight_descs(const amoeba_plan* plan) { return plan ? (int32_t)plan->wdescs.size() : 0; }

amoeba_status amoeba_plan_weight_desc(const amoeba_plan* plan, int32_t index, amoeba_weight_desc* out) {
    if (!plan || !out || index < 0 || index >= (int32_t)plan->wdescs.size()) return AMOEBA_ERR_INVALID_ARG;
    *out = plan->wdescs[index];
    return AMOEBA_OK;
}

amoeba_status amoeba_plan_set_option(amoeba_plan* plan, int32_t option, int64_t value) {
    if (!plan || value < 0 || option < 0) return AMOEBA_ERR_INVALID_ARG;
    const Options old = plan->opt;
    const int which = option / AMOEBA_OPT_WEIGHTS_ONLY;  // 0 both kernels, 1 weights only, 2 KV only
    const int id = option % AMOEBA_OPT_WEIGHTS_ONLY;
    if (which > 2) return AMOEBA_ERR_INVALID_ARG;
    if (option == AMOEBA_OPT_PAIR_ORDER) {  // a property of the table calls, not of a copy kernel
        if (value > 2) return AMOEBA_ERR_INVALID_ARG;
        plan->opt.pair_order = (int)value;
        return AMOEBA_OK;
    }
    KernelOpts* targets[2] = {which != 1 ? &plan->opt.kv : nullptr, which != 2 ? &plan->opt.w : nullptr};
    for (KernelOpts* k : targets) {
        if (!k) continue;
        switch (id) {
            case AMOEBA_OPT_COPY_PATH:
                if (value > 3) return AMOEBA_ERR_INVALID_ARG;
                k->copy_path = (int)value;
                break;
            case AMOEBA_OPT_CTAS_PER_SM:
                if (value > 32) return AMOEBA_ERR_INVALID_ARG;
                k->ctas_per_sm = (int)value;
                break;
            case AMOEBA_OPT_CHUNK_BYTES:
                if (value > 65536) return AMOEBA_ERR_INVALID_ARG;
                k->chunk_bytes = value;
                break;
            case AMOEBA_OPT_STAGES:
                if (value > 16) return AMOEBA_ERR_INVALID_ARG;
                k->stages = (int)value;
                break;
            case AMOEBA_OPT_LAG:
                if (value > 15) return AMOEBA_ERR_INVALID_ARG;
                k->lag = (int)value;
                break;
            case AMOEBA_OPT_WARPS:
                if (value > 16) return AMOEBA_ERR_INVALID_ARG;
                k->warps = (int)value;
                break;
            case AMOEBA_OPT_L2_HINT:
                if (value > 4) return AMOEBA_ERR_INVALID_ARG;
                k->hint = (int)value;
                break;
            case AMOEBA_OPT_MAX_CTAS:
                if (value > (1 << 20)) return AMOEBA_ERR_INVALID_ARG;
                k->max_ctas = (int)value;
                break;
            case AMOEBA_OPT_TENSOR_MAPS:
                if (value > 2) return AMOEBA_ERR_INVALID_ARG;
                k->tensor_maps = (int)value;
                break;
            case AMOEBA_OPT_L2_PROMOTION:
                if (value > 4) return AMOEBA_ERR_INVALID_ARG;
                k->l2_promotion = (int)value;
                break;
            case AMOEBA_OPT_WAIT_TRIES:
                if (value > (int64_t(1) << 30)) return AMOEBA_ERR_INVALID_ARG;
                k->wait_tries = (int)value;
                break;
            default:
                return AMOEBA_ERR_INVALID_ARG;
        }
    }
    amoeba_status st;
    try {
        st = finalize_chunks(plan);
        if (st != AMOEBA_OK) {
            plan->opt = old;
            finalize_chunks(plan);
        }
    } catch (...) {
        plan->opt = old;
        return AMOEBA_ERR_NO_MEMORY;
    }
    plan->bump_generation();
    return st;
}

amoeba_status amoeba_merge_live_bytes(const amoeba_plan* plan, int64_t* bytes) {
    if (!plan || !bytes) return AMOEBA_ERR_INVALID_ARG;
    const int n = merge_instances(plan);
    if (!n) return AMOEBA_ERR_UNSUPPORTED;
    *bytes = ((int64_t)n * plan->src.num_blocks + 15) / 16 * 16;
    return AMOEBA_OK;
}

amoeba_status amoeba_merge_bytes(const amoeba_plan* plan, int64_t n_live_blocks, int64_t* kv_bytes_rw) {
    if (!plan || !kv_bytes_rw || n_live_blocks < 0) return AMOEBA_ERR_INVALID_ARG;
    const int n = merge_instances(plan);
    if (!n) return AMOEBA_ERR_UNSUPPORTED;
    const amoeba_model& m = plan->src.model;
    // one old block on all a workers of its instance: Hkv headers; (n-1)/n of them move, read once and written once
    *kv_bytes_rw = 2 * n_live_blocks * m.num_layers * (m.num_kv_heads / n) * (n - 1) * plan->unit_bytes;
    return AMOEBA_OK;
}

amoeba_status amoeba_reshape_bytes(const amoeba_plan* plan, int64_t n_live_blocks, int64_t* kv_bytes_rw) {
    if (!plan || !kv_bytes_rw || n_live_blocks < 0) return AMOEBA_ERR_INVALID_ARG;
    const int f = reshape_factor(plan);
    if (!f) return AMOEBA_ERR_UNSUPPORTED;
    const int n = f > 0 ? f : -f;
    const amoeba_model& m = plan->src.model;
    // of the N header groups of a block one stays where it is; the others are read once and written once
    *kv_bytes_rw = 2 * n_live_blocks * m.num_layers * (m.num_kv_heads / n) * (n - 1) * plan->unit_bytes;
    return AMOEBA_OK;
}

amoeba_status amoeba_plan_weight_alias(const amoeba_plan* plan, int32_t dst_rank, int32_t tensor, int32_t* src_rank,
                                       int64_t* src_offset, int64_t* bytes) {
    if (!plan || !src_rank || !src_offset || !bytes || tensor < 0 || tensor >= kNumTensors || dst_rank < 0 ||
        dst_rank >= plan->dst.tp)
        return AMOEBA_ERR_INVALID_ARG;
    const amoeba_layout &s = plan->src, &d = plan->dst;
    if (s.weight_pad_parts <= 0 || s.weight_pad_parts != d.weight_pad_parts || s.fused_qkv != d.fused_qkv ||
        s.fused_gate_up != d.fused_gate_up || d.tp % s.tp)
        return AMOEBA_ERR_UNSUPPORTED;
    const WeightForm fs = weight_form(s), fd = weight_form(d);
    if (fs.page != fd.page) return AMOEBA_ERR_UNSUPPORTED;
    const int first = dst_rank * fd.per_worker;  // first partition the destination worker holds
    *src_rank = first / fs.per_worker;
    *src_offset = (int64_t)(first % fs.per_worker) * fs.pitch[tensor];
    *bytes = fd.block[tensor] ? (int64_t)fd.per_worker * fd.pitch[tensor] : 0;
    return AMOEBA_OK;
}

int64_t amoeba_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* amoeba_status_string(amoeba_status s) {
    switch (s) {
        case AMOEBA_OK: return "ok";
        case AMOEBA_ERR_INVALID_ARG: return "invalid argument";
        case AMOEBA_ERR_UNSUPPORTED: return "unsupported layout";
        case AMOEBA_ERR_ALIGNMENT: return "pointer, run or pitch not a multiple of 16 bytes";
        case AMOEBA_ERR_NO_FREE_BLOCKS: return "not enough free destination blocks";
        case AMOEBA_ERR_BAD_BLOCK_ID: return "block id out of range";
        case AMOEBA_ERR_CUDA: return "CUDA runtime error";
        case AMOEBA_ERR_TIMEOUT: return "on-device wait for a bulk copy ran out";
        case AMOEBA_ERR_TOO_LARGE: return "problem exceeds the library's built-in scratch array";
        case AMOEBA_ERR_NO_MEMORY: return "host memory allocation failed";
        case AMOEBA_ERR_INTERNAL: return "a work item outside its buffer was skipped (checked build)";
    }
    return "unknown status";
}

}  // extern "C"
