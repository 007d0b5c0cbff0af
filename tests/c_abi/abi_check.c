/*
 * A C11 caller of the library's C ABI: proves that amoeba.h is valid C, prints the size and the field offsets of
 * every struct that crosses the boundary (compared by the tests with the Python binding's mirrors), and drives the
 * host-only calls of one TP 2 -> 4 plan.  Needs no GPU.  Output: one "key value" pair per line.
 */
#include <stddef.h>
#include <stdio.h>
#include <string.h>

#include "amoeba.h"

#define SIZE(T) printf("sizeof." #T " %zu\n", sizeof(T))
#define OFF(T, f) printf("offsetof." #T "." #f " %zu\n", offsetof(T, f))

int main(void) {
    SIZE(amoeba_model);
    OFF(amoeba_model, num_layers); OFF(amoeba_model, hidden); OFF(amoeba_model, num_q_heads);
    OFF(amoeba_model, num_kv_heads); OFF(amoeba_model, head_dim); OFF(amoeba_model, intermediate);
    OFF(amoeba_model, elem_bytes);
    SIZE(amoeba_layout);
    OFF(amoeba_layout, model); OFF(amoeba_layout, tp); OFF(amoeba_layout, block_tokens); OFF(amoeba_layout, num_blocks);
    OFF(amoeba_layout, kv_order); OFF(amoeba_layout, fused_qkv); OFF(amoeba_layout, fused_gate_up);
    OFF(amoeba_layout, kv_layer_stride_bytes); OFF(amoeba_layout, weight_pad_parts); OFF(amoeba_layout, reserved);
    OFF(amoeba_layout, weight_page_bytes);
    SIZE(amoeba_pad_info);
    OFF(amoeba_pad_info, partitions_per_worker); OFF(amoeba_pad_info, reserved); OFF(amoeba_pad_info, partition_bytes);
    OFF(amoeba_pad_info, pitch_bytes); OFF(amoeba_pad_info, page_bytes); OFF(amoeba_pad_info, pages);
    SIZE(amoeba_layer_weights);
    OFF(amoeba_layer_weights, q); OFF(amoeba_layer_weights, k); OFF(amoeba_layer_weights, v);
    OFF(amoeba_layer_weights, o); OFF(amoeba_layer_weights, gate); OFF(amoeba_layer_weights, up);
    OFF(amoeba_layer_weights, down);
    SIZE(amoeba_kv_info);
    OFF(amoeba_kv_info, heads_per_run); OFF(amoeba_kv_info, runs_per_block); OFF(amoeba_kv_info, run_bytes);
    OFF(amoeba_kv_info, chunk_bytes); OFF(amoeba_kv_info, src_block_bytes); OFF(amoeba_kv_info, dst_block_bytes);
    OFF(amoeba_kv_info, src_layer_stride); OFF(amoeba_kv_info, dst_layer_stride);
    SIZE(amoeba_weight_desc);
    OFF(amoeba_weight_desc, src_rank); OFF(amoeba_weight_desc, src_tensor); OFF(amoeba_weight_desc, dst_rank);
    OFF(amoeba_weight_desc, dst_tensor); OFF(amoeba_weight_desc, src_off); OFF(amoeba_weight_desc, dst_off);
    OFF(amoeba_weight_desc, row_bytes); OFF(amoeba_weight_desc, src_pitch); OFF(amoeba_weight_desc, dst_pitch);
    OFF(amoeba_weight_desc, n_rows); OFF(amoeba_weight_desc, reserved);

    /* host-only call sequence: Llama-3-8B-shaped GQA, TP 2 -> 4 */
    amoeba_layout src, dst;
    memset(&src, 0, sizeof src);
    src.model.num_layers = 2; src.model.hidden = 512; src.model.num_q_heads = 16; src.model.num_kv_heads = 8;
    src.model.head_dim = 128; src.model.intermediate = 1792; src.model.elem_bytes = 2;
    src.tp = 2; src.block_tokens = 16; src.num_blocks = 10; src.fused_qkv = 1; src.fused_gate_up = 1;
    dst = src;
    dst.tp = 4; dst.num_blocks = 12;
    amoeba_plan* plan = NULL;
    amoeba_status st = amoeba_plan_create(&src, &dst, &plan);
    printf("plan_create %d\n", (int)st);
    if (st != AMOEBA_OK) return 1;
    amoeba_kv_info info;
    printf("kv_info %d\n", (int)amoeba_plan_kv_info(plan, &info));
    printf("heads_per_run %d\nrun_bytes %lld\nsrc_block_bytes %lld\ndst_block_bytes %lld\n", info.heads_per_run,
           (long long)info.run_bytes, (long long)info.src_block_bytes, (long long)info.dst_block_bytes);
    int64_t kv = 0, w = 0, ws = 0, pool = 0;
    printf("plan_bytes %d\n", (int)amoeba_plan_bytes(plan, 3, &kv, &w));
    printf("kv_bytes_rw %lld\nw_bytes_rw %lld\n", (long long)kv, (long long)w);
    printf("workspace %d\n", (int)amoeba_rewrite_workspace_bytes(plan, 5, 12, &ws));
    printf("workspace_bytes %lld\n", (long long)ws);
    printf("pool_bytes_status %d\n", (int)amoeba_layout_kv_pool_bytes(&dst, &pool));
    printf("dst_pool_bytes %lld\n", (long long)pool);
    printf("num_weight_descs %d\n", (int)amoeba_plan_num_weight_descs(plan));
    amoeba_weight_desc d;
    printf("weight_desc0 %d\n", (int)amoeba_plan_weight_desc(plan, 0, &d));
    printf("desc0_row_bytes %lld\n", (long long)d.row_bytes);
    printf("set_option %d\n", (int)amoeba_plan_set_option(plan, AMOEBA_OPT_CHUNK_BYTES, 4096));
    printf("bad_option %d\n", (int)amoeba_plan_set_option(plan, AMOEBA_OPT_CHUNK_BYTES, 24));
    printf("null_plan %d\n", (int)amoeba_plan_kv_info(NULL, &info));
    src.tp = 3;
    amoeba_plan* bad = NULL;
    printf("unsupported %d\n", (int)amoeba_plan_create(&src, &dst, &bad));
    printf("status_string %s\n", amoeba_status_string(AMOEBA_ERR_BAD_BLOCK_ID));
    amoeba_plan_destroy(plan);
    printf("done 1\n");
    return 0;
}
