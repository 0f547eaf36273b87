/* A plain C99 caller of the C ABI: no Python, no ctypes.  Reads one repack problem from a file,
 * runs create -> plan -> repack -> read_counts on a stream of its own, writes every output and both
 * pools to a second file.  The GPU test compiles this with gcc, runs it and compares the file with
 * the CPU oracle.
 *
 * input  : int64 header {L, NB, S, H, D, R, T, NBT, NF, thr_num, thr_den}, then
 *          bt_offsets[R+1] bt_blocks[NBT] tt_offsets[R+1] tt_slots[T] (int32), keep[T] (bytes, padded to a
 *          multiple of 4), free_blocks[NF] (int32), K pool, V pool (L*NB*S*H*D*2 bytes each)
 * output : vtoken_counts, new_bt_offsets[R+1] new_bt_blocks[NBT] new_tt_slots[T] freed_blocks[NBT]
 *          req_status[R] (int32), K pool, V pool
 * exit   : 0 ok, 2 usage or file error, 3 CUDA error, 4 library error
 */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "vtoken.h"

#define CK(call)                                                                              \
    do {                                                                                      \
        cudaError_t e_ = (call);                                                              \
        if (e_ != cudaSuccess) {                                                              \
            fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_));                       \
            return 3;                                                                         \
        }                                                                                     \
    } while (0)

#define VT(call)                                                                              \
    do {                                                                                      \
        int r_ = (call);                                                                      \
        if (r_ != VTOKEN_OK) {                                                                \
            fprintf(stderr, "%s: %s\n", #call, vtoken_strerror(r_));                          \
            return 4;                                                                         \
        }                                                                                     \
    } while (0)

static void *read_array(FILE *f, size_t bytes)
{
    void *p = malloc(bytes ? bytes : 1);
    if (p == NULL || fread(p, 1, bytes, f) != bytes) {
        fprintf(stderr, "short read (%zu bytes)\n", bytes);
        exit(2);
    }
    return p;
}

static int to_device(void **dev, const void *host, size_t bytes)
{
    CK(cudaMalloc(dev, bytes ? bytes : 16));
    if (bytes) CK(cudaMemcpy(*dev, host, bytes, cudaMemcpyHostToDevice));
    return 0;
}

static int write_device(FILE *f, const void *dev, size_t bytes)
{
    void *h = malloc(bytes ? bytes : 1);
    if (h == NULL) return 2;
    if (bytes) CK(cudaMemcpy(h, dev, bytes, cudaMemcpyDeviceToHost));
    if (fwrite(h, 1, bytes, f) != bytes) return 2;
    free(h);
    return 0;
}

int main(int argc, char **argv)
{
    if (argc != 3) {
        fprintf(stderr, "usage: %s <input file> <output file>\n", argv[0]);
        return 2;
    }
    FILE *f = fopen(argv[1], "rb");
    if (f == NULL) return 2;
    int64_t h[11];
    if (fread(h, sizeof(int64_t), 11, f) != 11) return 2;
    const int64_t L = h[0], NB = h[1], S = h[2], H = h[3], D = h[4], R = h[5], T = h[6], NBT = h[7], NF = h[8];
    const size_t pool_bytes = (size_t)(L * NB * S * H * D * 2);
    int32_t *bt_offsets = read_array(f, (size_t)(R + 1) * 4), *bt_blocks = read_array(f, (size_t)NBT * 4);
    int32_t *tt_offsets = read_array(f, (size_t)(R + 1) * 4), *tt_slots = read_array(f, (size_t)T * 4);
    uint8_t *keep = read_array(f, (size_t)((T + 3) / 4 * 4));
    int32_t *free_blocks = read_array(f, (size_t)NF * 4);
    void *k_host = read_array(f, pool_bytes), *v_host = read_array(f, pool_bytes);
    fclose(f);

    CK(cudaSetDevice(0));
    cudaStream_t stream;
    CK(cudaStreamCreate(&stream));
    void *k_pool, *v_pool, *d_bt_offsets, *d_bt_blocks, *d_tt_offsets, *d_tt_slots, *d_keep, *d_free, *d_R, *d_NF;
    const int32_t R32 = (int32_t)R, NF32 = (int32_t)NF;
    if (to_device(&k_pool, k_host, pool_bytes) || to_device(&v_pool, v_host, pool_bytes) ||
        to_device(&d_bt_offsets, bt_offsets, (size_t)(R + 1) * 4) || to_device(&d_bt_blocks, bt_blocks, (size_t)NBT * 4) ||
        to_device(&d_tt_offsets, tt_offsets, (size_t)(R + 1) * 4) || to_device(&d_tt_slots, tt_slots, (size_t)T * 4) ||
        to_device(&d_keep, keep, (size_t)T) || to_device(&d_free, free_blocks, (size_t)NF * 4) ||
        to_device(&d_R, &R32, 4) || to_device(&d_NF, &NF32, 4))
        return 3;

    vtoken_config cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.num_layers = (int32_t)L;
    cfg.num_blocks = (int32_t)NB;
    cfg.block_size = (int32_t)S;
    cfg.num_kv_heads = (int32_t)H;
    cfg.head_dim = (int32_t)D;
    cfg.elem_bytes = 2;
    cfg.k_pool = k_pool;
    cfg.v_pool = v_pool;
    cfg.layer_stride_bytes = 0;
    cfg.max_requests = (int32_t)(R > 0 ? R : 1);
    cfg.max_tokens = T > 0 ? T : 1;
    cfg.max_table_blocks = NBT > 0 ? NBT : 1;
    cfg.max_free_blocks = (int32_t)(NF > 0 ? NF : 1);
    vtoken_ctx *ctx = NULL;
    VT(vtoken_create(&cfg, &ctx));

    vtoken_plan_in in;
    memset(&in, 0, sizeof in);
    in.num_requests = d_R;
    in.bt_offsets = d_bt_offsets;
    in.bt_blocks = d_bt_blocks;
    in.tt_offsets = d_tt_offsets;
    in.tt_slots = d_tt_slots;
    in.keep = d_keep;
    in.select = NULL;
    in.thr_num = (uint32_t)h[9];
    in.thr_den = (uint32_t)h[10];
    in.free_blocks = d_free;
    in.num_free = d_NF;

    vtoken_plan_out out;
    memset(&out, 0, sizeof out);
    void *o_bt_offsets, *o_bt_blocks, *o_tt_slots, *o_freed, *o_status, *o_counts;
    CK(cudaMalloc(&o_bt_offsets, (size_t)(R + 1) * 4));
    CK(cudaMalloc(&o_bt_blocks, (size_t)cfg.max_table_blocks * 4));
    CK(cudaMalloc(&o_tt_slots, (size_t)cfg.max_tokens * 4));
    CK(cudaMalloc(&o_freed, (size_t)cfg.max_table_blocks * 4));
    CK(cudaMalloc(&o_status, (size_t)cfg.max_requests * 4));
    CK(cudaMalloc(&o_counts, sizeof(vtoken_counts)));
    CK(cudaMemset(o_bt_blocks, 0xff, (size_t)cfg.max_table_blocks * 4));
    CK(cudaMemset(o_freed, 0xff, (size_t)cfg.max_table_blocks * 4));
    out.new_bt_offsets = o_bt_offsets;
    out.new_bt_blocks = o_bt_blocks;
    out.new_tt_slots = o_tt_slots;
    out.freed_blocks = o_freed;
    out.req_status = o_status;
    out.counts = o_counts;

    VT(vtoken_plan(ctx, &in, &out, stream));
    VT(vtoken_repack(ctx, stream));
    vtoken_counts counts;
    VT(vtoken_read_counts(ctx, &counts, stream));      /* the call that synchronises */
    CK(cudaStreamSynchronize(stream));

    f = fopen(argv[2], "wb");
    if (f == NULL) return 2;
    if (fwrite(&counts, sizeof counts, 1, f) != 1) return 2;
    if (write_device(f, o_bt_offsets, (size_t)(R + 1) * 4) || write_device(f, o_bt_blocks, (size_t)NBT * 4) ||
        write_device(f, o_tt_slots, (size_t)T * 4) || write_device(f, o_freed, (size_t)NBT * 4) ||
        write_device(f, o_status, (size_t)R * 4) || write_device(f, k_pool, pool_bytes) ||
        write_device(f, v_pool, pool_bytes))
        return 3;
    fclose(f);
    vtoken_destroy(ctx);
    printf("moves %d dst_blocks %d freed %d consumed %d admitted %d deferred %d flags %u\n", counts.num_moves,
           counts.num_dst_blocks, counts.num_freed, counts.num_free_consumed, counts.num_admitted, counts.num_deferred,
           counts.error_flags);
    return 0;
}
