/* A C99 caller of the library: shows that pdkv.h is plain C and exercises the
 * host-only part of the ABI (no CUDA call is made: "dry_run" plans).  Prints
 * "key value" lines that the Python test compares with its own expectations. */
#include <stdio.h>
#include <string.h>

#include "pdkv.h"

int main(void)
{
    /* 2 layers, 2 KV heads, head_dim 16, 2-byte elements */
    pdkv_pool_desc ds = {PDKV_LAYOUT_BLOCK_MAJOR, 2, 2, 16, 2, 4, 6};
    pdkv_pool_desc dd = {PDKV_LAYOUT_LAYER_MAJOR, 2, 2, 16, 2, 8, 4};
    char *fake = (char *)0x7F0000000000; /* never dereferenced by a dry-run plan */
    pdkv_pool *ps = NULL, *pd = NULL, *none = NULL;
    pdkv_plan *plan = NULL;
    int32_t seq_len[2] = {5, 9};
    int64_t s_off[3] = {0, 2, 5}, d_off[3] = {0, 1, 3};
    int32_t s_tbl[5] = {3, 0, 4, 1, 5}, d_tbl[3] = {2, 1, 0};
    pdkv_batch_desc batch;
    size_t total = 0;
    const int64_t *req_off = NULL;
    const pdkv_tile *tiles = NULL;
    int64_t n_tiles = 0, launches = -1, v = -1;
    uint64_t rd = 0, wr = 0;
    int rc;

    printf("pool_bytes_src %zu\n", pdkv_pool_bytes(&ds));
    printf("pool_bytes_dst %zu\n", pdkv_pool_bytes(&dd));
    printf("strerror_ok %s\n", pdkv_strerror(PDKV_OK));
    if ((rc = pdkv_tune("dry_run", 1)) != PDKV_OK) return 10;
    if ((rc = pdkv_tune_get("tile_bytes", &v)) != PDKV_OK) return 11;
    printf("tile_bytes %lld\n", (long long)v);
    if (pdkv_tune("no_such_key", 1) != PDKV_ERR_INVALID_ARG) return 12;

    if ((rc = pdkv_pool_create(&ds, fake, pdkv_pool_bytes(&ds), 0, &ps)) != PDKV_OK) return 20;
    if ((rc = pdkv_pool_create(&dd, fake + ((size_t)1 << 40), pdkv_pool_bytes(&dd), 0, &pd)) != PDKV_OK) return 21;
    if (pdkv_pool_create(&dd, fake + 8, pdkv_pool_bytes(&dd), 0, &none) != PDKV_ERR_INVALID_ARG || none) return 22; /* misaligned */

    memset(&batch, 0, sizeof batch);
    batch.n_req = 2;
    batch.seq_len = seq_len;
    batch.src_tbl_off = s_off;
    batch.src_tbl = s_tbl;
    batch.dst_tbl_off = d_off;
    batch.dst_tbl = d_tbl;
    if ((rc = pdkv_plan_create(ps, pd, 8, &batch, NULL, &plan)) != PDKV_OK) return 30;
    if ((rc = pdkv_plan_buffer(plan, &total, &req_off)) != PDKV_OK) return 31;
    printf("buffer_bytes %zu\n", total);
    printf("req_off %lld %lld %lld\n", (long long)req_off[0], (long long)req_off[1], (long long)req_off[2]);
    if ((rc = pdkv_plan_traffic(plan, PDKV_OP_TRANSFER, &rd, &wr)) != PDKV_OK) return 32;
    printf("traffic %llu %llu\n", (unsigned long long)rd, (unsigned long long)wr);
    if ((rc = pdkv_plan_tiles(plan, PDKV_OP_PACK, &tiles, &n_tiles)) != PDKV_OK) return 33;
    printf("pack_tiles %lld first_src %lld first_dst %lld first_ntok %d\n", (long long)n_tiles,
           (long long)tiles[0].src_off, (long long)tiles[0].dst_off, (int)tiles[0].ntok);
    if ((rc = pdkv_plan_launches(plan, PDKV_OP_PACK, &launches)) != PDKV_OK) return 34;
    printf("pack_launches %lld\n", (long long)launches);
    {   /* what the plan would launch, and that it keeps the tunables it was created with */
        pdkv_launch_shape shape;
        int64_t frozen = -1;
        if ((rc = pdkv_plan_launch_shape(plan, PDKV_OP_TRANSFER, 0, 2, &shape)) != PDKV_OK) return 35;
        if ((rc = pdkv_tune("ctas_per_sm", 7)) != PDKV_OK) return 36;
        if ((rc = pdkv_plan_option(plan, "ctas_per_sm", &frozen)) != PDKV_OK) return 37;
        if ((rc = pdkv_tune("ctas_per_sm", 0)) != PDKV_OK) return 38;
        printf("launch_shape %d %d %d %d %lld\n", (int)shape.threads, (int)shape.vec_bytes, (int)shape.ctas_per_sm,
               (int)shape.variant, (long long)frozen);
        if (pdkv_plan_launch_shape(plan, PDKV_OP_TRANSFER, 1, 3, &shape) != PDKV_ERR_INVALID_ARG) return 39;
    }
    /* a dry-run plan cannot be launched */
    printf("transfer_on_dry_plan %d\n", pdkv_transfer(plan, 0, 2, NULL));

    d_tbl[2] = 1; /* decode block 1 written twice */
    {
        pdkv_plan *bad = NULL;
        printf("duplicate_decode_block %d\n", pdkv_plan_create(ps, pd, 8, &batch, NULL, &bad));
        if (bad) return 40;
    }
    if (pdkv_plan_destroy(plan) != PDKV_OK) return 50;
    if (pdkv_pool_destroy(ps) != PDKV_OK || pdkv_pool_destroy(pd) != PDKV_OK) return 51;
    if (pdkv_tune("dry_run", 0) != PDKV_OK) return 52;
    return 0;
}
