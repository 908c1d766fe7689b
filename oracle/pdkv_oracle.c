/*
 * TEST INFRASTRUCTURE -- not part of the product path.
 *
 * Plain, slow CPU statement of what the block-free KVCache transfer computes
 * (P/D-Serve, Sec. 3.5 "Block-free D2D KVCache Transfer"): the sender gathers a
 * request's discrete KV blocks into one contiguous buffer in which the K and V
 * of each layer follow one another ("Contiguous Buffer at Sender"), and the
 * receiver restores discrete blocks from those bytes ("RecvScatter at
 * Receiver").  Both sides keep block-fixed pools (Sec. 2.3 "Block-fixed
 * Management").  The result is a permutation of elements, so this file is the
 * definition written out: nested loops over the logical coordinate
 * (request r, layer l, K/V c, token t, head h, dim d), one element at a time.
 * No blocking, no vectorisation, no shared code with the CUDA library.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Pools (element offsets; b = table[t / B], tt = t mod B):
 *   layout 0, block-major  [block][layer][K/V][token][head][dim]
 *       off = ((((b*L + l)*2 + c)*B + tt)*H + h)*D + d
 *   layout 1, layer-major  [layer][K/V][block][head][token][dim]
 *       off = ((((l*2 + c)*NB + b)*H + h)*B + tt)*D + d
 *
 * Contiguous buffer: requests one after another in batch order; inside request
 * r, [layer][K/V][kept token][head][dim], so that layer l of request r is the
 * element range [off_r + l*2*n_r*H*D, +2*n_r*H*D) -- the "offset and length"
 * computed from prompt length, hidden size and precision in Sec. 3.5.
 *
 * Skip mask: entry j of request r's decode table may be marked resident; token
 * t is kept iff entry t / G is not marked (G = decode block tokens).  rank_r(t)
 * counts kept tokens before t; n_r is the number of kept tokens.
 */
#include <stdint.h>
#include <string.h>

typedef struct {
    int32_t layout, L, H, D, E, B;
    int64_t NB;
} okv_geom;

typedef struct {
    int32_t n_req;
    int32_t G;                   /* skip granule in tokens */
    const int32_t *seq_len;      /* [n_req] */
    const int64_t *src_tbl_off;  /* [n_req+1] */
    const int32_t *src_tbl;
    const int64_t *dst_tbl_off;  /* [n_req+1]; also indexes skip */
    const int32_t *dst_tbl;
    const uint8_t *skip;         /* parallel to dst_tbl, or NULL */
} okv_batch;

static int64_t pool_off(const okv_geom *g, int64_t b, int64_t l, int64_t c,
                        int64_t tt, int64_t h, int64_t d)
{
    if (g->layout == 0)
        return ((((b * g->L + l) * 2 + c) * g->B + tt) * g->H + h) * g->D + d;
    return ((((l * 2 + c) * g->NB + b) * g->H + h) * g->B + tt) * g->D + d;
}

static int kept(const okv_batch *bt, int r, int64_t t)
{
    if (!bt->skip)
        return 1;
    return bt->skip[bt->dst_tbl_off[r] + t / bt->G] == 0;
}

/* n_r: number of kept tokens of request r */
int64_t okv_kept_tokens(const okv_batch *bt, int r)
{
    int64_t n = 0;
    for (int64_t t = 0; t < bt->seq_len[r]; ++t)
        if (kept(bt, r, t))
            ++n;
    return n;
}

/* off_r in elements: exclusive prefix sum of 2*L*n_r*H*D in batch order */
int64_t okv_request_offset(const okv_batch *bt, int L, int H, int D, int r)
{
    int64_t off = 0;
    for (int q = 0; q < r; ++q)
        off += 2 * (int64_t)L * okv_kept_tokens(bt, q) * H * D;
    return off;
}

int64_t okv_buffer_elems(const okv_batch *bt, int L, int H, int D)
{
    return okv_request_offset(bt, L, H, D, bt->n_req);
}

static int64_t buf_off(int64_t off_r, int64_t n_r, int64_t l, int64_t c,
                       int64_t rank, int64_t h, int64_t d, int H, int D)
{
    return off_r + ((l * 2 + c) * n_r + rank) * H * D + h * D + d;
}

/* Sender side: blocks -> contiguous buffer, requests [r0,r1), layers [l0,l1). */
void okv_pack(const okv_geom *sg, const uint8_t *src, const okv_batch *bt,
              uint8_t *buf, int l0, int l1, int r0, int r1)
{
    const int E = sg->E;
    for (int r = r0; r < r1; ++r) {
        const int64_t n_r = okv_kept_tokens(bt, r);
        const int64_t off_r = okv_request_offset(bt, sg->L, sg->H, sg->D, r);
        for (int l = l0; l < l1; ++l)
            for (int c = 0; c < 2; ++c) {
                int64_t rank = 0;
                for (int64_t t = 0; t < bt->seq_len[r]; ++t) {
                    if (!kept(bt, r, t))
                        continue;
                    const int64_t b = bt->src_tbl[bt->src_tbl_off[r] + t / sg->B];
                    const int64_t tt = t % sg->B;
                    for (int h = 0; h < sg->H; ++h)
                        for (int d = 0; d < sg->D; ++d)
                            memcpy(buf + E * buf_off(off_r, n_r, l, c, rank, h, d, sg->H, sg->D),
                                   src + E * pool_off(sg, b, l, c, tt, h, d), E);
                    ++rank;
                }
            }
    }
}

/* Zero the token slots past the prompt's end in the request's last decode
 * block, unless that block is marked resident. */
static void zero_tail(const okv_geom *dg, uint8_t *dst, const okv_batch *bt,
                      int r, int l0, int l1)
{
    const int64_t len = bt->seq_len[r];
    const int64_t nblk = (len + dg->B - 1) / dg->B;
    if (nblk == 0)
        return;
    if (bt->skip && bt->skip[bt->dst_tbl_off[r] + nblk - 1])
        return;
    const int64_t b = bt->dst_tbl[bt->dst_tbl_off[r] + nblk - 1];
    for (int l = l0; l < l1; ++l)
        for (int c = 0; c < 2; ++c)
            for (int64_t tt = 0; tt < dg->B; ++tt) {
                if ((nblk - 1) * dg->B + tt < len)
                    continue;
                for (int h = 0; h < dg->H; ++h)
                    for (int d = 0; d < dg->D; ++d)
                        memset(dst + dg->E * pool_off(dg, b, l, c, tt, h, d), 0, dg->E);
            }
}

/* Receiver side (RecvScatter): contiguous buffer -> blocks. */
void okv_unpack(const okv_geom *dg, uint8_t *dst, const okv_batch *bt,
                const uint8_t *buf, int l0, int l1, int r0, int r1)
{
    const int E = dg->E;
    for (int r = r0; r < r1; ++r) {
        const int64_t n_r = okv_kept_tokens(bt, r);
        const int64_t off_r = okv_request_offset(bt, dg->L, dg->H, dg->D, r);
        for (int l = l0; l < l1; ++l)
            for (int c = 0; c < 2; ++c) {
                int64_t rank = 0;
                for (int64_t t = 0; t < bt->seq_len[r]; ++t) {
                    if (!kept(bt, r, t))
                        continue;
                    const int64_t b = bt->dst_tbl[bt->dst_tbl_off[r] + t / dg->B];
                    const int64_t tt = t % dg->B;
                    for (int h = 0; h < dg->H; ++h)
                        for (int d = 0; d < dg->D; ++d)
                            memcpy(dst + E * pool_off(dg, b, l, c, tt, h, d),
                                   buf + E * buf_off(off_r, n_r, l, c, rank, h, d, dg->H, dg->D), E);
                    ++rank;
                }
            }
        zero_tail(dg, dst, bt, r, l0, l1);
    }
}

/* Blocks -> blocks: every kept element goes from its place in the prefill pool
 * to its place in the decode pool; same tail rule as okv_unpack. */
void okv_transfer(const okv_geom *sg, const uint8_t *src, const okv_geom *dg,
                  uint8_t *dst, const okv_batch *bt, int l0, int l1, int r0, int r1)
{
    const int E = sg->E;
    for (int r = r0; r < r1; ++r) {
        for (int l = l0; l < l1; ++l)
            for (int c = 0; c < 2; ++c)
                for (int64_t t = 0; t < bt->seq_len[r]; ++t) {
                    if (!kept(bt, r, t))
                        continue;
                    const int64_t bs = bt->src_tbl[bt->src_tbl_off[r] + t / sg->B];
                    const int64_t bd = bt->dst_tbl[bt->dst_tbl_off[r] + t / dg->B];
                    for (int h = 0; h < sg->H; ++h)
                        for (int d = 0; d < sg->D; ++d)
                            memcpy(dst + E * pool_off(dg, bd, l, c, t % dg->B, h, d),
                                   src + E * pool_off(sg, bs, l, c, t % sg->B, h, d), E);
                }
        zero_tail(dg, dst, bt, r, l0, l1);
    }
}
