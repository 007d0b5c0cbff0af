/*
 * A C11 program that drives one TP a -> b transformation through the library's C ABI with nothing but the CUDA
 * runtime: cudaMalloc for every buffer, host-built tables and pools read from a file, the three data calls on a
 * stream of its own, results written to a file for the test to compare with the CPU oracle.
 *
 * in : int32 header {L, hidden, Hq, Hkv, D, I, a, b, T, NB_src, NB_dst, S, maxb, n_free}; seq_lens[S]; src_bt[S][maxb];
 *      free[n_free]; a source pools; then per source worker, per layer: fused qkv, o, fused gate_up, down.
 * out: int32 {status, n_pairs, free_left}; dst_bt[S][maxb]; b destination pools; per destination worker, per layer:
 *      fused qkv, o, fused gate_up, down.
 */
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "amoeba.h"

#define CHECK_CUDA(x)                                                                  \
    do {                                                                               \
        cudaError_t e_ = (x);                                                          \
        if (e_ != cudaSuccess) {                                                       \
            fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_));                   \
            return 2;                                                                  \
        }                                                                              \
    } while (0)
#define CHECK_AMOEBA(x)                                                                \
    do {                                                                               \
        amoeba_status s_ = (x);                                                        \
        if (s_ != AMOEBA_OK) {                                                         \
            fprintf(stderr, "%s: %s\n", #x, amoeba_status_string(s_));                 \
            return 3;                                                                  \
        }                                                                              \
    } while (0)

static void* upload(FILE* f, size_t bytes) {
    void* h = malloc(bytes ? bytes : 1);
    void* d = NULL;
    if (!h || fread(h, 1, bytes, f) != bytes) exit(4);
    if (cudaMalloc(&d, bytes ? bytes : 16) != cudaSuccess) exit(5);
    if (cudaMemcpy(d, h, bytes, cudaMemcpyHostToDevice) != cudaSuccess) exit(6);
    free(h);
    return d;
}

static void* device_filled(size_t bytes, int value) {
    void* d = NULL;
    if (cudaMalloc(&d, bytes ? bytes : 16) != cudaSuccess) exit(5);
    if (cudaMemset(d, value, bytes) != cudaSuccess) exit(6);
    return d;
}

static void download(FILE* f, const void* d, size_t bytes) {
    void* h = malloc(bytes ? bytes : 1);
    if (!h || cudaMemcpy(h, d, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) exit(7);
    if (fwrite(h, 1, bytes, f) != bytes) exit(8);
    free(h);
}

int main(int argc, char** argv) {
    if (argc != 3) return 1;
    FILE* in = fopen(argv[1], "rb");
    if (!in) return 1;
    int32_t hd[14];
    if (fread(hd, sizeof(int32_t), 14, in) != 14) return 1;
    const int L = hd[0], a = hd[6], b = hd[7], S = hd[11], maxb = hd[12], n_free = hd[13];
    amoeba_layout src, dst;
    memset(&src, 0, sizeof src);
    src.model.num_layers = L; src.model.hidden = hd[1]; src.model.num_q_heads = hd[2]; src.model.num_kv_heads = hd[3];
    src.model.head_dim = hd[4]; src.model.intermediate = hd[5]; src.model.elem_bytes = 2;
    src.tp = a; src.block_tokens = hd[8]; src.num_blocks = hd[9]; src.fused_qkv = 1; src.fused_gate_up = 1;
    dst = src;
    dst.tp = b; dst.num_blocks = hd[10];
    amoeba_plan* plan = NULL;
    CHECK_AMOEBA(amoeba_plan_create(&src, &dst, &plan));

    int32_t* d_lens = upload(in, sizeof(int32_t) * (size_t)S);
    int32_t* d_src_bt = upload(in, sizeof(int32_t) * (size_t)S * maxb);
    int32_t* d_free = upload(in, sizeof(int32_t) * (size_t)n_free);
    int64_t src_pool_bytes = 0, dst_pool_bytes = 0, ws_bytes = 0;
    CHECK_AMOEBA(amoeba_layout_kv_pool_bytes(&src, &src_pool_bytes));
    CHECK_AMOEBA(amoeba_layout_kv_pool_bytes(&dst, &dst_pool_bytes));
    const void* src_pools[AMOEBA_MAX_TP];
    void* dst_pools[AMOEBA_MAX_TP];
    for (int r = 0; r < a; ++r) src_pools[r] = upload(in, (size_t)src_pool_bytes);
    for (int r = 0; r < b; ++r) dst_pools[r] = device_filled((size_t)dst_pool_bytes, 0xA5);
    const int tensors[4] = {0, 3, 4, 6}; /* q (fused qkv), o, gate (fused gate_up), down */
    amoeba_layer_weights* sw = calloc((size_t)a * L, sizeof *sw);
    amoeba_layer_weights* dw = calloc((size_t)b * L, sizeof *dw);
    int64_t sbytes[4], dbytes[4];
    for (int t = 0; t < 4; ++t) {
        CHECK_AMOEBA(amoeba_layout_weight_bytes(&src, tensors[t], &sbytes[t]));
        CHECK_AMOEBA(amoeba_layout_weight_bytes(&dst, tensors[t], &dbytes[t]));
    }
    for (int r = 0; r < a; ++r)
        for (int l = 0; l < L; ++l) {
            amoeba_layer_weights* w = &sw[(size_t)r * L + l];
            w->q = upload(in, (size_t)sbytes[0]);
            w->o = upload(in, (size_t)sbytes[1]);
            w->gate = upload(in, (size_t)sbytes[2]);
            w->down = upload(in, (size_t)sbytes[3]);
        }
    for (int r = 0; r < b; ++r)
        for (int l = 0; l < L; ++l) {
            amoeba_layer_weights* w = &dw[(size_t)r * L + l];
            w->q = device_filled((size_t)dbytes[0], 0xA5);
            w->o = device_filled((size_t)dbytes[1], 0xA5);
            w->gate = device_filled((size_t)dbytes[2], 0xA5);
            w->down = device_filled((size_t)dbytes[3], 0xA5);
        }
    fclose(in);

    CHECK_AMOEBA(amoeba_rewrite_workspace_bytes(plan, S, n_free, &ws_bytes));
    void* d_ws = device_filled((size_t)ws_bytes, 0);
    int32_t* d_dst_bt = device_filled(sizeof(int32_t) * (size_t)S * maxb, 0xEE);
    const int pairs_cap = S * maxb;
    int32_t* d_pairs = device_filled(sizeof(int32_t) * 2 * (size_t)pairs_cap, 0xEE);
    int32_t* d_scalars = device_filled(sizeof(int32_t) * 4, 0); /* n_pairs, free_left, status */

    cudaStream_t stream;
    CHECK_CUDA(cudaStreamCreate(&stream));
    CHECK_AMOEBA(amoeba_rewrite_block_tables(plan, d_src_bt, d_lens, S, maxb, d_free, NULL, n_free, d_dst_bt, d_pairs,
                                             pairs_cap, d_scalars, d_scalars + 1, d_scalars + 2, d_ws, ws_bytes,
                                             stream));
    CHECK_AMOEBA(amoeba_reshard_kv(plan, src_pools, dst_pools, d_pairs, d_scalars, pairs_cap, 0, L, d_scalars + 2,
                                   stream));
    CHECK_AMOEBA(amoeba_reshard_weights(plan, sw, dw, 0, L, d_scalars + 2, stream));
    CHECK_CUDA(cudaStreamSynchronize(stream));

    FILE* out = fopen(argv[2], "wb");
    if (!out) return 1;
    int32_t sc[3];
    CHECK_CUDA(cudaMemcpy(sc, d_scalars, sizeof sc, cudaMemcpyDeviceToHost));
    const int32_t head[3] = {sc[2], sc[0], sc[1]};
    fwrite(head, sizeof(int32_t), 3, out);
    download(out, d_dst_bt, sizeof(int32_t) * (size_t)S * maxb);
    for (int r = 0; r < b; ++r) download(out, dst_pools[r], (size_t)dst_pool_bytes);
    for (int r = 0; r < b; ++r)
        for (int l = 0; l < L; ++l) {
            const amoeba_layer_weights* w = &dw[(size_t)r * L + l];
            download(out, w->q, (size_t)dbytes[0]);
            download(out, w->o, (size_t)dbytes[1]);
            download(out, w->gate, (size_t)dbytes[2]);
            download(out, w->down, (size_t)dbytes[3]);
        }
    fclose(out);
    amoeba_plan_destroy(plan);
    CHECK_CUDA(cudaStreamDestroy(stream));
    return 0;
}
