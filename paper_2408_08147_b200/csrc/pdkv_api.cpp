// C-ABI entry points and the host planner: validates a batch against the two
// pools, computes the contiguous buffer's per-request offsets (Sec. 3.5: a
// layer's offset and length follow from prompt length, hidden size and
// precision), cuts the batch into tiles and uploads the tile lists once.  This
// is the single-GPU counterpart of the meta exchange that precedes a transfer.
#include <algorithm>
#include <array>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>

#include "pdkv_internal.h"

struct pdkv_pool {
    pdkv_pool_desc d;
    char *base;
    size_t bytes;
    int device;
};

namespace {

using pdkv::Tile;

struct BlockGroup {     // one prefill block's share of the fused transfer (baseline)
    int32_t tile_begin, tile_end;
    int64_t memcpy_src, memcpy_dst, memcpy_bytes;  // memcpy_bytes > 0: plain copy suffices
};

thread_local std::string g_cuda_msg;
thread_local bool g_host_only_plan = false;  // set only around pdkv::create_host_plan()
thread_local unsigned g_plan_ops = 7u;       // tile lists to build (bit per pdkv_op); narrowed only there

int cuda_fail(cudaError_t e, const char *what)
{
    g_cuda_msg = std::string("CUDA error in ") + what + ": " + cudaGetErrorString(e);
    return PDKV_ERR_CUDA;
}

bool desc_ok(const pdkv_pool_desc *d)
{
    if (!d) return false;
    if (d->layout != PDKV_LAYOUT_BLOCK_MAJOR && d->layout != PDKV_LAYOUT_LAYER_MAJOR) return false;
    if (d->num_layers <= 0 || d->num_kv_heads <= 0 || d->head_dim <= 0 || d->block_tokens <= 0 ||
        d->num_blocks <= 0)
        return false;
    if (d->elem_bytes != 1 && d->elem_bytes != 2 && d->elem_bytes != 4 && d->elem_bytes != 8)
        return false;
    // every byte offset must fit a signed 64-bit integer with room to spare
    long double total = (long double)d->num_blocks * d->num_layers * 2.0L * d->block_tokens *
                        d->num_kv_heads * d->head_dim * d->elem_bytes;
    if (total > 4.0e18L) return false;
    // a single (block, layer, K/V) strip must stay below 2^31 vectors of one byte
    long double strip = (long double)d->block_tokens * d->num_kv_heads * d->head_dim * d->elem_bytes;
    if (strip > 2.0e9L) return false;
    return true;
}

using pdkv::DeviceGuard;

}  // namespace

struct pdkv_plan {
    bool has_src = false, has_dst = false;
    pdkv_pool src{}, dst{};
    int device = 0;
    int32_t L = 0, H = 0, D = 0, E = 0, G = 0;
    int64_t row_bytes = 0, hrow_bytes = 0;
    int32_t n_req = 0;
    std::vector<int64_t> kept;      // n_r
    std::vector<int64_t> req_off;   // bytes, n_req + 1
    uint64_t payload_bytes = 0, pad_bytes = 0;
    std::vector<Tile> tiles[3];
    const Tile *dev_tiles[3] = {nullptr, nullptr, nullptr};
    std::vector<BlockGroup> groups;
    bool same_blocks = false;   // both pools block-major with equal block size: a block's layer range is one byte range
    // maximal runs of consecutive block ids: prefill blocks the batch reads, decode blocks it writes
    std::vector<std::pair<int64_t, int64_t>> src_runs, dst_runs;  // (first id, count)
    void *dev_mem = nullptr;
    bool owns_dev_mem = true;   // false: dev_mem is a caller-provided workspace
    unsigned long long *dev_status = nullptr;
    int vec_bytes = 16;
    int64_t max_tile_bytes = 0;
    int64_t mean_tile_bytes[3] = {0, 0, 0};   // per operation, over its tile list
    int sm_count = 1;
    pdkv::LaunchOptions opt;   // the tunables as they stood when the plan was created
    // launch shape found by pdkv_plan_autotune() for each operation; threads == 0: not tuned
    struct Shape {
        int threads = 0, unroll = 0, ctas_per_sm = 0;
        int skew = -1;      // strip skew: -1 by the stride rule, 0 none, > 0 this many strips
        int variant = -1;   // kernel: -1 by the built-in rule, 0 register copy, 3 staged transpose
    } shape[3];
};

namespace {

int64_t pool_tile_off(const pdkv_pool_desc &d, int64_t b, int64_t tt, int64_t row, int64_t hrow)
{
    if (d.layout == PDKV_LAYOUT_BLOCK_MAJOR)
        return b * (2 * (int64_t)d.num_layers * d.block_tokens * hrow) + tt * hrow;
    return b * ((int64_t)d.num_kv_heads * d.block_tokens * row) + tt * row;
}

pdkv::Side pool_side(const pdkv_pool &p, int64_t row, int64_t hrow)
{
    pdkv::Side s;
    s.base = p.base;
    s.size = (int64_t)pdkv_pool_bytes(&p.d);
    if (p.d.layout == PDKV_LAYOUT_BLOCK_MAJOR) {
        s.lc_stride = (int64_t)p.d.block_tokens * hrow;
        s.tok_stride = hrow;
        s.head_stride = row;
    } else {
        s.lc_stride = p.d.num_blocks * (int64_t)p.d.num_kv_heads * p.d.block_tokens * row;
        s.tok_stride = row;
        s.head_stride = (int64_t)p.d.block_tokens * row;
    }
    if (p.d.num_kv_heads == 1) s.head_stride = row;   // one head: the head stride is never applied, and both layouts are token-major
    return s;
}

pdkv::Side buffer_side(const void *buf, size_t bytes, int64_t row, int64_t hrow)
{
    pdkv::Side s;
    s.base = (char *)buf;
    s.size = (int64_t)bytes;
    s.lc_stride = -1;
    s.tok_stride = hrow;
    s.head_stride = row;
    return s;
}

// Cut the batch into tiles for one operation.  A tile never crosses a block
// boundary of a paged side it touches, a skip-granule boundary, or the tile
// size cap; so a tile is all-copy or all-zero, never mixed.
void build_tiles(pdkv_plan &pl, int op, const pdkv_batch_desc &b, int64_t cap_tok)
{
    const bool use_src = op != PDKV_OP_UNPACK, use_dst = op != PDKV_OP_PACK;
    const int64_t Bp = use_src ? pl.src.d.block_tokens : 0;
    const int64_t Bd = use_dst ? pl.dst.d.block_tokens : 0;
    const int64_t G = pl.G;
    std::vector<Tile> &out = pl.tiles[op];
    const bool want_groups = op == PDKV_OP_TRANSFER;
    {   // upper bound on the tiles of this list, so that the vectors grow once
        size_t bound = 0;
        for (int32_t r = 0; r < pl.n_req; ++r) {
            const int64_t len = b.seq_len[r];
            bound += (size_t)(len / cap_tok + 2);
            if (use_src) bound += (size_t)(len / Bp + 1);
            if (use_dst) bound += (size_t)(len / Bd + 1 + Bd / cap_tok + 1);
            if (b.dst_skip) bound += (size_t)(len / G + 1);
        }
        out.reserve(bound);
        if (want_groups) pl.groups.reserve(bound);
    }
    const bool same_blocks = want_groups && pl.src.d.layout == PDKV_LAYOUT_BLOCK_MAJOR &&
                             pl.dst.d.layout == PDKV_LAYOUT_BLOCK_MAJOR && Bp == Bd;
    if (want_groups) pl.same_blocks = same_blocks;
    for (int32_t r = 0; r < pl.n_req; ++r) {
        const int64_t len = b.seq_len[r];
        const uint8_t *skip = b.dst_skip ? b.dst_skip + b.dst_tbl_off[r] : nullptr;
        int64_t t = 0, rank = 0;
        int64_t group_block = -1;
        while (t < len) {
            if (skip && skip[t / G]) {
                t = std::min(len, (t / G + 1) * G);
                continue;
            }
            // the run up to the next boundary is cut into equal pieces no longer than the cap,
            // not into full pieces and a short rest
            int64_t end = len;
            if (skip) end = std::min(end, (t / G + 1) * G);
            if (use_src) end = std::min(end, (t / Bp + 1) * Bp);
            if (use_dst) end = std::min(end, (t / Bd + 1) * Bd);
            {
                const int64_t run = end - t, pieces = (run + cap_tok - 1) / cap_tok;
                end = t + (run + pieces - 1) / pieces;
            }
            Tile tl;
            tl.ntok = (int32_t)(end - t);
            tl.n_kept = (int32_t)pl.kept[r];
            const int64_t in_buf = pl.req_off[r] + rank * pl.hrow_bytes;
            tl.src_off = use_src ? pool_tile_off(pl.src.d, b.src_tbl[b.src_tbl_off[r] + t / Bp], t % Bp,
                                                 pl.row_bytes, pl.hrow_bytes)
                                 : in_buf;
            tl.dst_off = use_dst ? pool_tile_off(pl.dst.d, b.dst_tbl[b.dst_tbl_off[r] + t / Bd], t % Bd,
                                                 pl.row_bytes, pl.hrow_bytes)
                                 : in_buf;
            if (want_groups) {
                if (t / Bp != group_block) {
                    group_block = t / Bp;
                    BlockGroup g{};
                    g.tile_begin = (int32_t)out.size();
                    g.tile_end = g.tile_begin;
                    const bool full = same_blocks && (group_block + 1) * Bp <= len;
                    if (full) {
                        const int64_t blk = 2 * (int64_t)pl.L * Bp * pl.hrow_bytes;
                        g.memcpy_src = (int64_t)b.src_tbl[b.src_tbl_off[r] + group_block] * blk;
                        g.memcpy_dst = (int64_t)b.dst_tbl[b.dst_tbl_off[r] + group_block] * blk;
                        g.memcpy_bytes = blk;
                    }
                    pl.groups.push_back(g);
                }
                pl.groups.back().tile_end = (int32_t)out.size() + 1;
            }
            out.push_back(tl);
            rank += end - t;
            t = end;
        }
        if (use_dst && len > 0) {
            const int64_t nb = (len + Bd - 1) / Bd;
            const int64_t first_pad = len - (nb - 1) * Bd;
            if (first_pad < Bd && !(skip && skip[nb - 1])) {
                const int64_t blk = b.dst_tbl[b.dst_tbl_off[r] + nb - 1];
                const int64_t pad_pieces = (Bd - first_pad + cap_tok - 1) / cap_tok;
                const int64_t pad_tok = (Bd - first_pad + pad_pieces - 1) / pad_pieces;
                for (int64_t tt = first_pad; tt < Bd; tt += pad_tok) {
                    Tile tl;
                    tl.ntok = (int32_t)std::min(pad_tok, Bd - tt);
                    tl.n_kept = (int32_t)pl.kept[r];
                    tl.src_off = -1;
                    tl.dst_off = pool_tile_off(pl.dst.d, blk, tt, pl.row_bytes, pl.hrow_bytes);
                    out.push_back(tl);
                    if (want_groups) pl.groups.back().tile_end = (int32_t)out.size();
                }
            }
        }
    }
}

int check_table(const int64_t *off, const int32_t *tbl, int32_t n_req, const int32_t *len,
                int64_t B, int64_t NB)
{
    if (!off || !tbl) return PDKV_ERR_INVALID_ARG;
    if (off[0] < 0) return PDKV_ERR_TABLE;
    for (int32_t r = 0; r < n_req; ++r) {
        if (off[r + 1] < off[r]) return PDKV_ERR_TABLE;
        const int64_t need = ((int64_t)len[r] + B - 1) / B;
        if (off[r + 1] - off[r] < need) return PDKV_ERR_TABLE;
        for (int64_t j = 0; j < need; ++j) {
            const int64_t id = tbl[off[r] + j];
            if (id < 0 || id >= NB) return PDKV_ERR_TABLE;
        }
    }
    return PDKV_OK;
}

int launch_op(const pdkv_plan *pl, int op, const pdkv::Side &src, const pdkv::Side &dst,
              int32_t tile_begin, int32_t n_tiles, int l0, int l1, cudaStream_t stream)
{
    if (!pl->dev_mem) return PDKV_ERR_INVALID_ARG;  // host-only plan
    pdkv::CopyParams p;
    p.src = src;
    p.dst = dst;
    if (pl->opt.debug_bounds && pl->opt.debug_shrink > 0) {
        p.src.size = std::max<int64_t>(0, p.src.size - pl->opt.debug_shrink);
        p.dst.size = std::max<int64_t>(0, p.dst.size - pl->opt.debug_shrink);
    }
    p.tiles = pl->dev_tiles[op];
    p.tile_begin = tile_begin;
    p.n_tiles = n_tiles;
    p.lc_begin = 2 * l0;
    p.n_lc = 2 * (l1 - l0);
    p.H = pl->H;
    p.row_bytes = (int32_t)pl->row_bytes;
    pdkv::ResolvedLaunch r;
    const int share = pdkv::partition_sms_of(stream);   // a stream of an SM partition: the grid fits its share
    pdkv::resolve_launch(pl, op, src, dst, p.n_lc, share > 0 ? share : pl->sm_count, &r);
    p.lc_fastest = r.lc_fastest;
    p.chunked = r.chunked;
    p.lc_skew = r.lc_skew;
    p.lc_skew_shift = r.lc_skew_shift;
    p.src_order = r.src_order;
    p.group_threads = 0;
    p.status = pl->dev_status;
    cudaError_t e;
    if (r.cfg.variant == 3 && pdkv::staged_supported(p, r.cfg)) {
        e = pdkv::launch_staged(p, r.cfg, stream);
    } else if ((r.cfg.variant == 1 || r.cfg.variant == 2) && pdkv::bulk_supported(r.cfg, p.row_bytes)) {
        r.cfg.vec_bytes = 16;
        e = pdkv::launch_bulk(p, r.cfg, stream);
    } else {
        e = pdkv::launch_copy(p, r.cfg, stream);
    }
    if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    return PDKV_OK;
}

bool layers_ok(const pdkv_plan *pl, int l0, int l1) { return l0 >= 0 && l0 <= l1 && l1 <= pl->L; }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The kernels read one side while writing the other, with no ordering between tiles.
bool ranges_overlap(const void *a, size_t a_bytes, const void *b, size_t b_bytes)
{
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a_bytes && b_bytes && a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

}  // namespace

namespace {

// Shapes found by pdkv_plan_autotune(), remembered per geometry for later plans of the process.
struct ShapeKey {
    int32_t v[12];
    bool operator<(const ShapeKey &o) const { return std::lexicographical_compare(v, v + 12, o.v, o.v + 12); }
};

ShapeKey shape_key(const pdkv_plan *pl)
{
    ShapeKey k{};
    const pdkv_pool_desc *s = pl->has_src ? &pl->src.d : nullptr, *d = pl->has_dst ? &pl->dst.d : nullptr;
    k.v[0] = pl->L; k.v[1] = pl->H; k.v[2] = pl->D; k.v[3] = pl->E;
    k.v[4] = s ? s->layout : -1; k.v[5] = s ? s->block_tokens : 0;
    k.v[6] = d ? d->layout : -1; k.v[7] = d ? d->block_tokens : 0;
    k.v[8] = (int32_t)std::min<int64_t>(pl->max_tile_bytes, INT32_MAX);
    for (int op = 0; op < 3; ++op) k.v[9 + op] = (int32_t)std::min<int64_t>(pl->mean_tile_bytes[op] >> 10, INT32_MAX);
    return k;
}

std::mutex g_shapes_mutex;
std::map<ShapeKey, std::array<pdkv_plan::Shape, 3>> g_shapes;

}  // namespace

namespace pdkv {
Tunables &tunables()
{
    static Tunables t;
    return t;
}
}  // namespace pdkv

namespace pdkv {

int create_host_plan(const pdkv_pool *src, const pdkv_pool *dst, const pdkv_batch_desc *batch, unsigned op_mask,
                     pdkv_plan **out)
{
    g_host_only_plan = true;
    g_plan_ops = op_mask & 7u;
    const int rc = pdkv_plan_create(src, dst, 0, batch, nullptr, out);
    g_plan_ops = 7u;
    g_host_only_plan = false;
    return rc;
}

LaunchOptions snapshot_options()
{
    const Tunables &t = tunables();
    LaunchOptions o;
    o.ctas_per_sm = (int)t.ctas_per_sm;
    o.max_ctas = (int)t.max_ctas;
    o.threads = (int)t.threads;
    o.unroll = (int)t.unroll;
    o.vec32 = (int)t.vec32;
    o.lc_fastest = (int)t.lc_fastest;
    o.group_threads = (int)t.group_threads;
    o.chunked = (int)t.chunked;
    o.lc_skew = (int)t.lc_skew;
    o.lc_skew_shift = (int)t.lc_skew_shift;
    o.debug_bounds = (int)t.debug_bounds;
    o.debug_shrink = t.debug_shrink;
    o.variant = (int)t.variant;
    o.stages = (int)t.stages;
    o.src_order = (int)t.src_order;
    o.tile_bytes = t.tile_bytes;
    return o;
}

void describe_transfer(const pdkv_plan *plan, Side *src, Side *dst, int *H, int *row_bytes,
                       int *vec_bytes, int *num_layers, int *device)
{
    *src = pool_side(plan->src, plan->row_bytes, plan->hrow_bytes);
    *dst = pool_side(plan->dst, plan->row_bytes, plan->hrow_bytes);
    *H = plan->H;
    *row_bytes = (int)plan->row_bytes;
    *vec_bytes = plan->vec_bytes;
    *num_layers = plan->L;
    *device = plan->device;
}

void resolve_launch(const pdkv_plan *pl, int op, const Side &src, const Side &dst, int n_lc, int sm_count,
                    ResolvedLaunch *out)
{
    const LaunchOptions &o = pl->opt;
    LaunchConfig &cfg = out->cfg;
    const int64_t hrow = pl->hrow_bytes, row = pl->row_bytes;
    const bool flat = src.head_stride == row && src.tok_stride == hrow && dst.head_stride == row &&
                      dst.tok_stride == hrow;
    const bool small = pl->mean_tile_bytes[op] < 24 * 1024;
    out->lc_fastest = o.lc_fastest;
    out->chunked = o.chunked;
    bool strip_first_rule = false;
    {   // Kernel.  Automatic: the register copy, except for tiles that go from a token-major side to
        // a head-major one in rows of more than 128 bytes that are not multiples of 256 (head sizes
        // such as 80, 96 or 112 at 2 bytes).  Those run the staged transpose, whose reads and writes
        // are both contiguous runs: measured on 8B- and 70B-shaped batches with 80 to 192 dims per
        // head, +3 to +12% over the register copy for tiles of 24 KiB and more.  Smaller tiles of such
        // rows (16 to 24 KiB: 16-token prefill blocks) gain 5-9% from it only in the fused call out of
        // a block-major pool and only with the work order turned round -- consecutive CTAs take the
        // consecutive (layer, K/V) strips of one block, which are one contiguous stretch of the pool --
        // and three stages; every other combination (256- and 128-byte rows, other calls) is slower
        // that way.  pdkv_plan_autotune() may have timed the other kernel.
        int variant = o.variant;
        if (variant < 0) {
            const bool tok_to_head = src.tok_stride >= src.head_stride && dst.tok_stride < dst.head_stride;
            // (rows under 128 bytes that are not multiples of 64 -- 80, 96 or 112 one-byte elements -- are worse
            // still on the register copy, 4.4-5.2 TB/s, and reach 5.9-6.4 staged; 64- and 128-byte rows do not)
            const bool odd_rows = row % 16 == 0 && ((row > 128 && row % 256 != 0) || (row < 128 && row % 64 != 0));
            variant = 0;
            if (tok_to_head && odd_rows && !small) {
                variant = 3;
            } else if (tok_to_head && odd_rows && op == PDKV_OP_TRANSFER && pl->mean_tile_bytes[op] >= 16 * 1024 &&
                       pl->src.d.layout == PDKV_LAYOUT_BLOCK_MAJOR && o.lc_fastest == 0 && n_lc >= 16) {
                variant = 3;
                strip_first_rule = true;
            }
            if (pl->shape[op].variant >= 0) {
                variant = pl->shape[op].variant;
                strip_first_rule = strip_first_rule && variant == 3;
            }
        }
        cfg.variant = variant;
        if (strip_first_rule) out->lc_fastest = 1;
    }
    {   // Strip skew (see pdkv_tune "lc_skew").  Automatic: only for calls that read (or, failing
        // that, write) a block-major pool whose block stride, stripped of its factors of two, is
        // divisible by 3, 5 or 17 (e.g. 80 layers x 64 tokens x 2 KiB = 5 x 4 MiB).  With such
        // strides the same-offset strips of many blocks, which one sweep touches at the same
        // time, collide in DRAM (measured on 37 strides: reads 4-12% and writes 2% slower, every
        // odd part sharing a factor with 255 and no other); skewing the strip by the block's
        // position in the batch spreads them and recovers most of it.  Tiles of one block keep
        // the same skew so that its strip is still moved in one piece.
        int64_t skew = o.lc_skew, shift = o.lc_skew_shift;
        if (skew < 0) {
            skew = 0;
            shift = 0;
            bool have_pool = false;
            auto consider = [&](const pdkv_pool &pool) {
                if (have_pool || pool.d.layout != PDKV_LAYOUT_BLOCK_MAJOR) return;
                const uint64_t strip = (uint64_t)pool.d.block_tokens * (uint64_t)pl->hrow_bytes;
                uint64_t odd = 2ull * (uint64_t)pl->L * strip;
                while (odd && !(odd & 1ull)) odd >>= 1;
                const bool slow_stride = !(odd % 3 && odd % 5 && odd % 17);
                if (!slow_stride && pl->shape[op].skew <= 0) return;
                have_pool = true;
                skew = 16;
                const uint64_t per_block = pl->max_tile_bytes > 0 ? strip / (uint64_t)pl->max_tile_bytes : 1;
                while ((2ull << shift) <= per_block) ++shift;
            };
            if (op != PDKV_OP_UNPACK && pl->has_src) consider(pl->src);   // the pool that is read comes first
            if (op != PDKV_OP_PACK && pl->has_dst) consider(pl->dst);
            // pdkv_plan_autotune() may have measured that this batch is better off without the rule's
            // skew (0), or with one although the rule sees no reason (> 0; needs a block-major pool)
            if (pl->shape[op].skew == 0) skew = 0;
            else if (pl->shape[op].skew > 0 && have_pool) skew = pl->shape[op].skew;
        }
        while (skew > 1 && skew > n_lc) skew >>= 1;   // a power of two within the strips of this call
        out->lc_skew = out->lc_fastest ? 0 : (int32_t)skew;
        out->lc_skew_shift = (int32_t)shift;
    }
    cfg.vec_bytes = pl->vec_bytes;
    const bool bases32 = ((reinterpret_cast<uintptr_t>(src.base) | reinterpret_cast<uintptr_t>(dst.base)) & 31u) == 0;
    if (pl->vec_bytes == 16 && o.vec32 && pl->row_bytes % 32 == 0 && bases32) cfg.vec_bytes = 32;
    if (flat) {   // a flat tile is one run of bytes on both sides, and every tile starts at a multiple of a token's
                  // bytes: the access width follows from those, whatever the row size (144-byte rows: 32, not 16)
        int w = (o.vec32 && bases32) ? 32 : 16;
        while (hrow % w) w >>= 1;
        if (w > cfg.vec_bytes) cfg.vec_bytes = w;
    }
    cfg.unroll = o.unroll;
    cfg.threads = o.threads;
    cfg.ctas_per_sm = o.ctas_per_sm;
    cfg.max_ctas = o.max_ctas;
    cfg.sm_count = sm_count;
    cfg.elem_bytes = pl->E;
    cfg.check_bounds = o.debug_bounds != 0;
    {   // Automatic launch shape, measured best per class of copy on B200.  Full tiles
        // (about 32 KiB): a flat copy (token-major on both sides) runs 512 threads with
        // one access in flight each, i.e. two passes per tile; a copy with a head-major
        // side runs 256 threads with four, i.e. one pass per tile.  Batches of small
        // tiles (few KV heads, short blocks): groups of threads that cover a tile in two
        // passes of one access each, 32 threads at least.
        const pdkv_plan::Shape &tuned = pl->shape[op];
        const bool use_tuned = tuned.threads > 0 && cfg.unroll == 0 && cfg.threads == 0;
        if (use_tuned) {   // found by pdkv_plan_autotune(): the whole CTA works on one tile
            cfg.threads = tuned.threads;
            cfg.unroll = tuned.unroll;
            cfg.ctas_per_sm = tuned.ctas_per_sm;
        }
        // Copies of 9-17 KiB tiles (16-token blocks of 128-byte rows: 1-byte elements or 64 dims per
        // head; four KV heads; 8-token blocks): one pass of 256 threads x 2 accesses per tile and three
        // CTAs per SM, i.e. 48 KiB in flight per SM.  Measured on six such batches of row-permuting
        // copies: +7 to +16% over two passes of 512 x 1 (5.5-5.9 -> 6.2-6.6 TB/s); tiles of 8 KiB, of
        // 18 KiB and of 32 KiB lose with it.  Flat copies neither gain nor lose at 16 KiB and gain 20%
        // at 10-14 KiB, so they take it too.  Keyed on this operation's own mean tile.
        const int64_t mean_vecs = pl->mean_tile_bytes[op] / cfg.vec_bytes;
        const bool half_tile = !use_tuned && cfg.variant == 0 && cfg.threads == 0 && cfg.unroll == 0 &&
                               o.group_threads == 0 && mean_vecs > 288 && mean_vecs <= 544;   // (zero-fill tiles may be larger)
        if (half_tile) {
            cfg.threads = 256;
            cfg.unroll = 2;
            if (cfg.ctas_per_sm == 0) cfg.ctas_per_sm = 3;
        }
        // Tiles of more than half but less than a full 256 x 4 pass (head sizes, head counts or
        // block sizes that are not powers of two): that one pass, whatever the class of copy.
        const int64_t max_vecs = pl->max_tile_bytes / cfg.vec_bytes;
        const bool odd_tile = !use_tuned && !half_tile && cfg.unroll == 0 && cfg.threads == 0 && max_vecs > 512 && max_vecs < 1024;
        if (odd_tile) {
            cfg.unroll = 4;
            cfg.threads = 256;
        }
        // staged transpose: 256 threads store what one warp's bulk loads fetched (and 256 x 4 is what
        // the register copy runs if the launch turns out not to qualify for the staged kernel)
        const bool staged = cfg.variant == 3 && cfg.threads == 0 && cfg.unroll == 0;
        if (staged) {
            cfg.threads = 256;
            cfg.unroll = 4;
        }
        if (cfg.unroll == 0) cfg.unroll = (flat || small) ? 1 : 4;
        if (cfg.threads == 0) cfg.threads = (flat || small) ? 512 : 256;
        cfg.group_threads = o.group_threads;
        if ((use_tuned || odd_tile || staged || half_tile) && cfg.group_threads == 0) cfg.group_threads = cfg.threads;
        if (cfg.group_threads == 0) {
            const int64_t vecs = std::max<int64_t>(1, pl->mean_tile_bytes[op] / cfg.vec_bytes);
            const int64_t want = vecs / ((flat || small) ? 2 : cfg.unroll);
            int g = 32;
            while (g < want && g < cfg.threads) g *= 2;
            cfg.group_threads = g;
        }
        if (cfg.ctas_per_sm == 0) cfg.ctas_per_sm = 2;
    }
    // Row order inside a tile of the register copy (see CopyParams::src_order).  Measured on
    // transposing copies with rows of 128 to 384 bytes: walking the rows in the order of the side
    // that is read is 3-13% faster for rows of more than 128 bytes that are not multiples of 256, and
    // for 128-byte rows in tiles under 24 KiB; for multiples of 256 bytes, and for 128-byte rows in
    // full tiles, the order of the side that is written wins by 5-10%.
    out->src_order = o.src_order >= 0 ? o.src_order : ((!flat && row % 256 != 0 && (row > 128 || small)) ? 1 : 0);
    // The staged transpose keeps stages x tile bytes of loads in flight per CTA; with two CTAs per SM
    // two stages are the measured optimum (three: -10% on 32 KiB tiles), so the automatic choice uses
    // two whatever "stages" says for the bulk-copy variants (three for the strip-first order of 16-24 KiB tiles).
    cfg.stages = (cfg.variant == 3 && o.variant < 0) ? (strip_first_rule ? 3 : 2) : o.stages;
    cfg.max_tile_bytes = pl->max_tile_bytes;
}

int report_cuda_error(cudaError_t e, const char *what) { return cuda_fail(e, what); }

int plan_num_layers(const pdkv_plan *plan) { return plan->L; }

}  // namespace pdkv

extern "C" {

size_t pdkv_pool_bytes(const pdkv_pool_desc *d)
{
    if (!desc_ok(d)) return 0;
    return (size_t)d->num_blocks * d->num_layers * 2 * d->block_tokens * d->num_kv_heads *
           d->head_dim * d->elem_bytes;
}

int pdkv_pool_create(const pdkv_pool_desc *desc, void *dev_base, size_t bytes, int device,
                     pdkv_pool **out)
{
    if (out) *out = nullptr;
    if (!desc || !out || !dev_base || device < 0) return PDKV_ERR_INVALID_ARG;
    if (!desc_ok(desc)) return PDKV_ERR_GEOMETRY;
    if (!aligned16(dev_base) || bytes < pdkv_pool_bytes(desc)) return PDKV_ERR_INVALID_ARG;
    pdkv_pool *p = new (std::nothrow) pdkv_pool;
    if (!p) return PDKV_ERR_NOMEM;
    p->d = *desc;
    p->base = static_cast<char *>(dev_base);
    p->bytes = bytes;
    p->device = device;
    *out = p;
    return PDKV_OK;
}

int pdkv_pool_destroy(pdkv_pool *pool)
{
    delete pool;
    return PDKV_OK;
}

int pdkv_plan_create(const pdkv_pool *src, const pdkv_pool *dst, int32_t skip_granule_tokens,
                     const pdkv_batch_desc *batch, void *stream, pdkv_plan **out)
{
    return pdkv_plan_create_in(src, dst, skip_granule_tokens, batch, nullptr, 0, nullptr, stream, out);
}

int pdkv_plan_create_in(const pdkv_pool *src, const pdkv_pool *dst, int32_t skip_granule_tokens,
                        const pdkv_batch_desc *batch, void *workspace, size_t workspace_bytes,
                        size_t *needed_bytes, void *stream, pdkv_plan **out)
{
    if (out) *out = nullptr;
    if (needed_bytes) *needed_bytes = 0;
    if (!out || !batch || (!src && !dst)) return PDKV_ERR_INVALID_ARG;
    if (batch->n_req < 0 || (batch->n_req > 0 && !batch->seq_len)) return PDKV_ERR_INVALID_ARG;
    if (src && dst) {
        if (src->d.num_layers != dst->d.num_layers || src->d.num_kv_heads != dst->d.num_kv_heads ||
            src->d.head_dim != dst->d.head_dim || src->d.elem_bytes != dst->d.elem_bytes)
            return PDKV_ERR_GEOMETRY;
        if (src->device != dst->device) return PDKV_ERR_INVALID_ARG;
        if (ranges_overlap(src->base, pdkv_pool_bytes(&src->d), dst->base, pdkv_pool_bytes(&dst->d)))
            return PDKV_ERR_INVALID_ARG;   // in-place re-blocking is not supported
    }
    int32_t G = skip_granule_tokens;
    if (dst) {
        if (G <= 0) G = dst->d.block_tokens;
        if (G != dst->d.block_tokens) return PDKV_ERR_INVALID_ARG;
    } else if (batch->dst_skip && G <= 0) {
        return PDKV_ERR_INVALID_ARG;
    }
    if (G <= 0) G = 1;
    for (int32_t r = 0; r < batch->n_req; ++r)
        if (batch->seq_len[r] < 0) return PDKV_ERR_INVALID_ARG;

    const pdkv_pool *any = src ? src : dst;
    try {
        pdkv_plan *pl = new pdkv_plan;
        struct Holder {
            pdkv_plan *p;
            ~Holder() { if (p) pdkv_plan_destroy(p); }
        } hold{pl};
        pl->has_src = src != nullptr;
        pl->has_dst = dst != nullptr;
        if (src) pl->src = *src;
        if (dst) pl->dst = *dst;
        pl->device = any->device;
        pl->L = any->d.num_layers;
        pl->H = any->d.num_kv_heads;
        pl->D = any->d.head_dim;
        pl->E = any->d.elem_bytes;
        pl->G = G;
        pl->row_bytes = (int64_t)pl->D * pl->E;
        pl->hrow_bytes = pl->row_bytes * pl->H;
        pl->n_req = batch->n_req;
        pl->opt = pdkv::snapshot_options();

        int rc;
        if (src && (rc = check_table(batch->src_tbl_off, batch->src_tbl, batch->n_req, batch->seq_len,
                                     src->d.block_tokens, src->d.num_blocks)) != PDKV_OK)
            return rc;
        if (dst && (rc = check_table(batch->dst_tbl_off, batch->dst_tbl, batch->n_req, batch->seq_len,
                                     dst->d.block_tokens, dst->d.num_blocks)) != PDKV_OK)
            return rc;
        if (batch->dst_skip) {
            if (!batch->dst_tbl_off) return PDKV_ERR_INVALID_ARG;
            if (batch->dst_tbl_off[0] < 0) return PDKV_ERR_TABLE;
            for (int32_t r = 0; r < batch->n_req; ++r) {
                const int64_t need = ((int64_t)batch->seq_len[r] + G - 1) / G;
                if (batch->dst_tbl_off[r + 1] - batch->dst_tbl_off[r] < need) return PDKV_ERR_TABLE;
            }
        }
        auto runs_of = [](const std::vector<uint8_t> &seen, std::vector<std::pair<int64_t, int64_t>> &out) {
            for (size_t i = 0; i < seen.size();) {
                if (!seen[i]) {
                    ++i;
                    continue;
                }
                size_t j = i;
                while (j < seen.size() && seen[j]) ++j;
                out.emplace_back((int64_t)i, (int64_t)(j - i));
                i = j;
            }
        };
        if (src) {  // prefill blocks holding at least one kept token
            std::vector<uint8_t> seen((size_t)src->d.num_blocks, 0);
            const int64_t Bp = src->d.block_tokens;
            for (int32_t r = 0; r < batch->n_req; ++r) {
                const int64_t len = batch->seq_len[r];
                const uint8_t *skip = batch->dst_skip ? batch->dst_skip + batch->dst_tbl_off[r] : nullptr;
                for (int64_t t = 0; t < len;) {
                    const int64_t next = std::min(len, std::min((t / Bp + 1) * Bp, (t / G + 1) * (int64_t)G));
                    if (!(skip && skip[t / G])) seen[(size_t)batch->src_tbl[batch->src_tbl_off[r] + t / Bp]] = 1;
                    t = next;
                }
            }
            runs_of(seen, pl->src_runs);
        }
        if (dst) {  // every written decode block has exactly one writer
            std::vector<uint8_t> seen((size_t)dst->d.num_blocks, 0);
            const int64_t Bd = dst->d.block_tokens;
            for (int32_t r = 0; r < batch->n_req; ++r) {
                const int64_t need = ((int64_t)batch->seq_len[r] + Bd - 1) / Bd;
                for (int64_t j = 0; j < need; ++j) {
                    const int64_t e = batch->dst_tbl_off[r] + j;
                    if (batch->dst_skip && batch->dst_skip[e]) continue;
                    uint8_t &s = seen[(size_t)batch->dst_tbl[e]];
                    if (s) return PDKV_ERR_TABLE;
                    s = 1;
                }
            }
            runs_of(seen, pl->dst_runs);
        }

        // kept tokens and buffer offsets
        pl->kept.resize((size_t)pl->n_req);
        pl->req_off.assign((size_t)pl->n_req + 1, 0);
        const int64_t tok_bytes = 2 * (int64_t)pl->L * pl->hrow_bytes;
        uint64_t pad_tokens = 0;
        for (int32_t r = 0; r < pl->n_req; ++r) {
            const int64_t len = batch->seq_len[r];
            int64_t n = len;
            if (batch->dst_skip) {
                n = 0;
                const uint8_t *skip = batch->dst_skip + batch->dst_tbl_off[r];
                for (int64_t j = 0; j * G < len; ++j)
                    if (!skip[j]) n += std::min<int64_t>(G, len - j * G);
            }
            pl->kept[(size_t)r] = n;
            pl->req_off[(size_t)r + 1] = pl->req_off[(size_t)r] + n * tok_bytes;
            if (dst && len > 0) {
                const int64_t Bd = dst->d.block_tokens;
                const int64_t nb = (len + Bd - 1) / Bd;
                if (!(batch->dst_skip && batch->dst_skip[batch->dst_tbl_off[r] + nb - 1]))
                    pad_tokens += (uint64_t)(nb * Bd - len);
            }
        }
        pl->payload_bytes = (uint64_t)pl->req_off[(size_t)pl->n_req];
        pl->pad_bytes = pad_tokens * (uint64_t)tok_bytes;

        // widest vector that divides a row (bases are 16-byte aligned)
        pl->vec_bytes = 16;
        while (pl->row_bytes % pl->vec_bytes) pl->vec_bytes >>= 1;

        // Tile size cap.  The kernels split a vector index with multiply-high
        // divisions that are exact while dividend * divisor < 2^32, so the cap
        // also keeps vectors * vectors-per-row and rows * max(H, tokens) below it.
        int64_t cap_tok = std::max<int64_t>(1, pl->opt.tile_bytes / pl->hrow_bytes);
        {
            const int64_t vpr = pl->row_bytes / pl->vec_bytes;
            const int64_t max_b = std::max<int64_t>(src ? src->d.block_tokens : 1, dst ? dst->d.block_tokens : 1);
            auto exact = [&](int64_t cap) {
                const long double tok = (long double)std::min(cap, max_b);
                const long double rows = tok * pl->H;
                return rows * vpr * vpr < 4.0e9L && rows * std::max<long double>(pl->H, tok) < 4.0e9L;
            };
            while (cap_tok > 1 && !exact(cap_tok)) cap_tok /= 2;
            if (!exact(cap_tok)) return PDKV_ERR_GEOMETRY;
        }
        if (src && (g_plan_ops & 1u)) build_tiles(*pl, PDKV_OP_PACK, *batch, cap_tok);
        if (dst && (g_plan_ops & 2u)) build_tiles(*pl, PDKV_OP_UNPACK, *batch, cap_tok);
        if (src && dst && (g_plan_ops & 4u)) build_tiles(*pl, PDKV_OP_TRANSFER, *batch, cap_tok);
        for (int op = 0; op < 3; ++op) {
            if (pl->tiles[op].size() > (size_t)INT32_MAX) return PDKV_ERR_INVALID_ARG;
            int64_t sum = 0;
            for (const Tile &t : pl->tiles[op]) {
                pl->max_tile_bytes = std::max<int64_t>(pl->max_tile_bytes, t.ntok * pl->hrow_bytes);
                sum += t.ntok * pl->hrow_bytes;
            }
            pl->mean_tile_bytes[op] = pl->tiles[op].empty() ? 0 : sum / (int64_t)pl->tiles[op].size();
        }

        if (pdkv::tunables().autotune_reuse) {   // shapes an earlier pdkv_plan_autotune() found for this geometry
            std::lock_guard<std::mutex> lock(g_shapes_mutex);
            auto it = g_shapes.find(shape_key(pl));
            if (it != g_shapes.end())
                for (int op = 0; op < 3; ++op) pl->shape[op] = it->second[(size_t)op];
        }

        // device bytes of the plan: [status words][pack tiles][unpack tiles][transfer tiles]
        const size_t head = 256;
        size_t total = head;
        for (int op = 0; op < 3; ++op) total += pl->tiles[op].size() * sizeof(Tile);
        if (needed_bytes) *needed_bytes = total;

        if (pdkv::tunables().dry_run || g_host_only_plan) {  // host-only plan: tile lists can be inspected, nothing can launch
            hold.p = nullptr;
            *out = pl;
            return PDKV_OK;
        }

        // one device allocation: [status words][pack tiles][unpack tiles][transfer tiles]
        DeviceGuard guard(pl->device);
        if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
        // (cudaGetDeviceProperties costs milliseconds; one attribute query does not)
        cudaError_t e = cudaDeviceGetAttribute(&pl->sm_count, cudaDevAttrMultiProcessorCount, pl->device);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        if (workspace) {  // caller-provided device memory: nothing is allocated or freed
            if (!aligned16(workspace)) return PDKV_ERR_INVALID_ARG;
            if (workspace_bytes < total) return PDKV_ERR_BUFFER_TOO_SMALL;
            pl->dev_mem = workspace;
            pl->owns_dev_mem = false;
        } else {
            e = cudaMalloc(&pl->dev_mem, total);
            if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc");
        }
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        e = cudaMemsetAsync(pl->dev_mem, 0, head, st);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
        pl->dev_status = static_cast<unsigned long long *>(pl->dev_mem);
        size_t at = head;
        for (int op = 0; op < 3; ++op) {
            const size_t bytes = pl->tiles[op].size() * sizeof(Tile);
            pl->dev_tiles[op] = reinterpret_cast<const Tile *>(static_cast<char *>(pl->dev_mem) + at);
            if (bytes) {
                e = cudaMemcpyAsync(static_cast<char *>(pl->dev_mem) + at, pl->tiles[op].data(), bytes,
                                    cudaMemcpyHostToDevice, st);
                if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync");
            }
            at += bytes;
        }
        e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
        hold.p = nullptr;
        *out = pl;
        return PDKV_OK;
    } catch (const std::bad_alloc &) {
        return PDKV_ERR_NOMEM;
    }
}

int pdkv_plan_autotune(pdkv_plan *plan, void *buf, size_t buf_bytes, void *stream)
{
    if (!plan || !plan->dev_mem) return PDKV_ERR_INVALID_ARG;
    const bool with_buf = buf != nullptr;
    if (with_buf && buf_bytes < plan->payload_bytes) return PDKV_ERR_BUFFER_TOO_SMALL;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e != cudaSuccess) {
        if (e0) cudaEventDestroy(e0);
        return cuda_fail(e, "cudaEventCreate");
    }
    // whole-model launches: a subset of the layers has fewer strips per sweep and was seen to rank shapes differently
    const int layers = plan->L;

    int rc = PDKV_OK;
    auto run = [&](int op) -> int {
        if (op == PDKV_OP_PACK) return pdkv_pack(plan, buf, buf_bytes, 0, layers, stream);
        if (op == PDKV_OP_UNPACK) return pdkv_unpack(plan, buf, buf_bytes, 0, layers, stream);
        return pdkv_transfer(plan, 0, layers, stream);
    };
    auto time_ms = [&](int op, float *ms) -> int {
        const int reps = 3;
        int r = run(op);   // warm-up, and the first touch of a new instantiation
        if (r != PDKV_OK) return r;
        cudaError_t ce = cudaEventRecord(e0, st);
        for (int i = 0; i < reps && r == PDKV_OK; ++i) r = run(op);
        if (r != PDKV_OK) return r;
        if (ce == cudaSuccess) ce = cudaEventRecord(e1, st);
        if (ce == cudaSuccess) ce = cudaEventSynchronize(e1);
        if (ce == cudaSuccess) ce = cudaEventElapsedTime(ms, e0, e1);
        if (ce != cudaSuccess) return cuda_fail(ce, "autotune timing");
        *ms /= reps;
        return PDKV_OK;
    };
    for (int op = 0; op < 3 && rc == PDKV_OK; ++op) {
        if (plan->tiles[op].empty() || plan->payload_bytes == 0) continue;
        if (op != PDKV_OP_TRANSFER && !with_buf) continue;
        if ((op != PDKV_OP_UNPACK && !plan->has_src) || (op != PDKV_OP_PACK && !plan->has_dst)) continue;
        if (plan->mean_tile_bytes[op] < 8 * 1024) continue;   // small tiles: thread groups, sized automatically
        const int vec = (plan->vec_bytes == 16 && plan->row_bytes % 32 == 0) ? 32 : plan->vec_bytes;
        const int64_t nvec = std::max<int64_t>(1, plan->mean_tile_bytes[op] / vec);
        std::vector<pdkv_plan::Shape> cand;
        auto add = [&](int64_t threads, int unroll, int ctas) {
            threads = (threads + 31) / 32 * 32;
            const int cap = vec * unroll >= 256 ? 256 : (vec * unroll >= 128 ? 512 : 1024);
            if (threads < 64 || threads > cap) return;
            for (const auto &c : cand)
                if (c.threads == threads && c.unroll == unroll && c.ctas_per_sm == ctas) return;
            pdkv_plan::Shape s;
            s.threads = (int)threads;
            s.unroll = unroll;
            s.ctas_per_sm = ctas;
            cand.push_back(s);
        };
        add(256, 4, 2); add(512, 1, 2); add(512, 2, 2); add(256, 1, 4); add(1024, 1, 1); add(256, 2, 2);
        add(nvec, 1, 2); add((nvec + 1) / 2, 2, 2); add((nvec + 3) / 4, 4, 2);       // one pass = one tile
        add((nvec + 1) / 2, 1, 2); add((nvec + 3) / 4, 2, 2);                         // two passes = one tile
        add((nvec + 1) / 2, 2, 3); add((nvec + 3) / 4, 4, 3); add((nvec + 3) / 4, 4, 4);   // one pass, more CTAs per SM
        plan->shape[op] = pdkv_plan::Shape();
        float best_ms = 0.f;
        rc = time_ms(op, &best_ms);              // the per-class default is the incumbent
        pdkv_plan::Shape best;
        for (size_t i = 0; i < cand.size() && rc == PDKV_OK; ++i) {
            plan->shape[op] = cand[i];
            float ms = 0.f;
            rc = time_ms(op, &ms);
            if (rc == PDKV_OK && ms < 0.975f * best_ms) {   // a candidate must win by more than the noise (2.5%)
                best_ms = ms;
                best = cand[i];
            }
        }
        plan->shape[op] = best;
        // the other kernel for tiles that are transposed on the way (register copy <-> staged transpose),
        // with that kernel's own built-in shape
        if (rc == PDKV_OK && plan->opt.variant < 0 && op != PDKV_OP_PACK && plan->has_dst &&
            plan->dst.d.layout == PDKV_LAYOUT_LAYER_MAJOR && (op == PDKV_OP_UNPACK || plan->src.d.layout == PDKV_LAYOUT_BLOCK_MAJOR) &&
            plan->row_bytes % 16 == 0) {
            const pdkv::Side buf_side = buffer_side(nullptr, 0, plan->row_bytes, plan->hrow_bytes);
            pdkv::ResolvedLaunch by_rule;
            plan->shape[op] = pdkv_plan::Shape();
            pdkv::resolve_launch(plan, op, op == PDKV_OP_UNPACK ? buf_side : pool_side(plan->src, plan->row_bytes, plan->hrow_bytes),
                                 pool_side(plan->dst, plan->row_bytes, plan->hrow_bytes), 2 * layers, plan->sm_count, &by_rule);
            pdkv_plan::Shape other;
            other.variant = by_rule.cfg.variant == 3 ? 0 : 3;
            plan->shape[op] = other;
            float ms = 0.f;
            rc = time_ms(op, &ms);
            if (rc == PDKV_OK && ms < 0.975f * best_ms) {
                best_ms = ms;
                best = other;
            }
            plan->shape[op] = best;
        }
        // the strip skew the other way round: on where the stride rule leaves it off, off where it is on
        if (rc == PDKV_OK && plan->opt.lc_skew < 0 && plan->opt.lc_fastest == 0) {
            const pdkv_pool *pools[2] = {op != PDKV_OP_UNPACK && plan->has_src ? &plan->src : nullptr,
                                         op != PDKV_OP_PACK && plan->has_dst ? &plan->dst : nullptr};
            bool block_major = false, rule_on = false;
            for (const pdkv_pool *pool : pools) {
                if (!pool || pool->d.layout != PDKV_LAYOUT_BLOCK_MAJOR) continue;
                block_major = true;
                uint64_t odd = 2ull * (uint64_t)plan->L * (uint64_t)pool->d.block_tokens * (uint64_t)plan->hrow_bytes;
                while (odd && !(odd & 1ull)) odd >>= 1;
                rule_on = rule_on || !(odd % 3 && odd % 5 && odd % 17);
            }
            if (block_major && 2 * layers >= 16) {
                plan->shape[op].skew = rule_on ? 0 : 16;
                float ms = 0.f;
                rc = time_ms(op, &ms);
                if (!(rc == PDKV_OK && ms < 0.975f * best_ms)) plan->shape[op].skew = -1;
            }
        }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != PDKV_OK) {
        for (int op = 0; op < 3; ++op) plan->shape[op] = pdkv_plan::Shape();
        return rc;
    }
    {
        std::lock_guard<std::mutex> lock(g_shapes_mutex);
        std::array<pdkv_plan::Shape, 3> all = {plan->shape[0], plan->shape[1], plan->shape[2]};
        g_shapes[shape_key(plan)] = all;
    }
    return PDKV_OK;
}

int pdkv_plan_set_shape(pdkv_plan *plan, int op, int32_t threads, int32_t unroll, int32_t ctas_per_sm)
{
    if (!plan || op < 0 || op > 2) return PDKV_ERR_INVALID_ARG;
    if (threads == 0 && unroll == 0 && ctas_per_sm == 0) {   // back to the built-in choice
        plan->shape[op] = pdkv_plan::Shape();
        return PDKV_OK;
    }
    plan->shape[op].skew = -1;
    if (threads < 32 || threads > 1024 || threads % 32 || (unroll != 1 && unroll != 2 && unroll != 4 && unroll != 8) ||
        ctas_per_sm < 1 || ctas_per_sm > 32)
        return PDKV_ERR_INVALID_ARG;
    plan->shape[op].threads = threads;
    plan->shape[op].unroll = unroll;
    plan->shape[op].ctas_per_sm = ctas_per_sm;
    return PDKV_OK;
}

int pdkv_plan_shape(const pdkv_plan *plan, int op, int32_t *threads, int32_t *unroll, int32_t *ctas_per_sm,
                    int32_t *lc_skew)
{
    if (!plan || op < 0 || op > 2) return PDKV_ERR_INVALID_ARG;
    if (lc_skew) *lc_skew = plan->shape[op].skew;
    if (threads) *threads = plan->shape[op].threads;
    if (unroll) *unroll = plan->shape[op].unroll;
    if (ctas_per_sm) *ctas_per_sm = plan->shape[op].ctas_per_sm;
    return PDKV_OK;
}

int pdkv_plan_option(const pdkv_plan *plan, const char *key, int64_t *value)
{
    if (!plan || !key || !value) return PDKV_ERR_INVALID_ARG;
    const pdkv::LaunchOptions &o = plan->opt;
    const std::string k(key);
    if (k == "tile_bytes") *value = o.tile_bytes;
    else if (k == "ctas_per_sm") *value = o.ctas_per_sm;
    else if (k == "max_ctas") *value = o.max_ctas;
    else if (k == "threads") *value = o.threads;
    else if (k == "unroll") *value = o.unroll;
    else if (k == "vec32") *value = o.vec32;
    else if (k == "lc_fastest") *value = o.lc_fastest;
    else if (k == "chunked") *value = o.chunked;
    else if (k == "lc_skew") *value = o.lc_skew;
    else if (k == "lc_skew_shift") *value = o.lc_skew_shift;
    else if (k == "group_threads") *value = o.group_threads;
    else if (k == "debug_bounds") *value = o.debug_bounds;
    else if (k == "debug_shrink") *value = o.debug_shrink;
    else if (k == "variant") *value = o.variant;
    else if (k == "stages") *value = o.stages;
    else if (k == "src_order") *value = o.src_order;
    else return PDKV_ERR_INVALID_ARG;
    return PDKV_OK;
}

int pdkv_plan_launch_shape(const pdkv_plan *plan, int op, int layer_begin, int layer_end, pdkv_launch_shape *out)
{
    if (!plan || !out || op < 0 || op > 2 || !layers_ok(plan, layer_begin, layer_end)) return PDKV_ERR_INVALID_ARG;
    if ((op != PDKV_OP_UNPACK && !plan->has_src) || (op != PDKV_OP_PACK && !plan->has_dst))
        return PDKV_ERR_INVALID_ARG;
    // the buffer's base is taken as 32-byte aligned, as device allocations are
    const pdkv::Side buf = buffer_side(nullptr, 0, plan->row_bytes, plan->hrow_bytes);
    const pdkv::Side s = op == PDKV_OP_UNPACK ? buf : pool_side(plan->src, plan->row_bytes, plan->hrow_bytes);
    const pdkv::Side d = op == PDKV_OP_PACK ? buf : pool_side(plan->dst, plan->row_bytes, plan->hrow_bytes);
    pdkv::ResolvedLaunch r;
    pdkv::resolve_launch(plan, op, s, d, 2 * (layer_end - layer_begin), plan->sm_count, &r);
    out->threads = r.cfg.threads;
    out->unroll = r.cfg.unroll;
    out->ctas_per_sm = r.cfg.ctas_per_sm;
    out->group_threads = r.cfg.group_threads;
    out->vec_bytes = r.cfg.vec_bytes;
    out->max_ctas = r.cfg.max_ctas;
    out->lc_skew = r.lc_skew;
    out->lc_skew_shift = r.lc_skew_shift;
    out->lc_fastest = r.lc_fastest;
    out->chunked = r.chunked;
    out->src_order = r.src_order;
    out->variant = r.cfg.variant;
    out->debug_bounds = r.cfg.check_bounds ? 1 : 0;
    return PDKV_OK;
}

int pdkv_plan_destroy(pdkv_plan *plan)
{
    if (!plan) return PDKV_OK;
    int rc = PDKV_OK;
    if (plan->dev_mem && plan->owns_dev_mem) {
        DeviceGuard guard(plan->device);
        cudaError_t e = cudaFree(plan->dev_mem);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaFree");
    }
    delete plan;
    return rc;
}

int pdkv_plan_buffer(const pdkv_plan *plan, size_t *total_bytes, const int64_t **req_off_bytes)
{
    if (!plan) return PDKV_ERR_INVALID_ARG;
    if (total_bytes) *total_bytes = (size_t)plan->payload_bytes;
    if (req_off_bytes) *req_off_bytes = plan->req_off.data();
    return PDKV_OK;
}

int pdkv_plan_traffic(const pdkv_plan *plan, int op, uint64_t *bytes_read, uint64_t *bytes_written)
{
    if (!plan || op < 0 || op > 2) return PDKV_ERR_INVALID_ARG;
    if ((op != PDKV_OP_UNPACK && !plan->has_src) || (op != PDKV_OP_PACK && !plan->has_dst))
        return PDKV_ERR_INVALID_ARG;
    if (bytes_read) *bytes_read = plan->payload_bytes;
    if (bytes_written) *bytes_written = plan->payload_bytes + (op == PDKV_OP_PACK ? 0 : plan->pad_bytes);
    return PDKV_OK;
}

int pdkv_pack(const pdkv_plan *plan, void *buf, size_t buf_bytes, int l0, int l1, void *stream)
{
    if (!plan || !plan->has_src || !layers_ok(plan, l0, l1)) return PDKV_ERR_INVALID_ARG;
    if (buf_bytes < plan->payload_bytes) return PDKV_ERR_BUFFER_TOO_SMALL;
    if (!plan->dev_mem) return PDKV_ERR_INVALID_ARG;  // host-only plan
    if (plan->payload_bytes == 0 || l0 == l1) return PDKV_OK;
    if (!buf || !aligned16(buf)) return PDKV_ERR_INVALID_ARG;
    if (ranges_overlap(buf, plan->payload_bytes, plan->src.base, pdkv_pool_bytes(&plan->src.d)))
        return PDKV_ERR_INVALID_ARG;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    return launch_op(plan, PDKV_OP_PACK, pool_side(plan->src, plan->row_bytes, plan->hrow_bytes),
                     buffer_side(buf, buf_bytes, plan->row_bytes, plan->hrow_bytes), 0,
                     (int32_t)plan->tiles[PDKV_OP_PACK].size(), l0, l1, static_cast<cudaStream_t>(stream));
}

int pdkv_unpack(const pdkv_plan *plan, const void *buf, size_t buf_bytes, int l0, int l1, void *stream)
{
    if (!plan || !plan->has_dst || !layers_ok(plan, l0, l1)) return PDKV_ERR_INVALID_ARG;
    if (buf_bytes < plan->payload_bytes) return PDKV_ERR_BUFFER_TOO_SMALL;
    if (!plan->dev_mem) return PDKV_ERR_INVALID_ARG;  // host-only plan
    if (plan->tiles[PDKV_OP_UNPACK].empty() || l0 == l1) return PDKV_OK;
    if (plan->payload_bytes && (!buf || !aligned16(buf))) return PDKV_ERR_INVALID_ARG;
    if (ranges_overlap(buf, plan->payload_bytes, plan->dst.base, pdkv_pool_bytes(&plan->dst.d)))
        return PDKV_ERR_INVALID_ARG;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    return launch_op(plan, PDKV_OP_UNPACK, buffer_side(buf, buf_bytes, plan->row_bytes, plan->hrow_bytes),
                     pool_side(plan->dst, plan->row_bytes, plan->hrow_bytes), 0,
                     (int32_t)plan->tiles[PDKV_OP_UNPACK].size(), l0, l1,
                     static_cast<cudaStream_t>(stream));
}

int pdkv_transfer(const pdkv_plan *plan, int l0, int l1, void *stream)
{
    if (!plan || !plan->has_src || !plan->has_dst || !layers_ok(plan, l0, l1))
        return PDKV_ERR_INVALID_ARG;
    if (!plan->dev_mem) return PDKV_ERR_INVALID_ARG;  // host-only plan
    if (plan->tiles[PDKV_OP_TRANSFER].empty() || l0 == l1) return PDKV_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    return launch_op(plan, PDKV_OP_TRANSFER, pool_side(plan->src, plan->row_bytes, plan->hrow_bytes),
                     pool_side(plan->dst, plan->row_bytes, plan->hrow_bytes), 0,
                     (int32_t)plan->tiles[PDKV_OP_TRANSFER].size(), l0, l1,
                     static_cast<cudaStream_t>(stream));
}

int pdkv_transfer_blockwise(const pdkv_plan *plan, void *stream)
{
    if (!plan || !plan->has_src || !plan->has_dst || !plan->dev_mem) return PDKV_ERR_INVALID_ARG;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const pdkv::Side s = pool_side(plan->src, plan->row_bytes, plan->hrow_bytes);
    const pdkv::Side d = pool_side(plan->dst, plan->row_bytes, plan->hrow_bytes);
    for (const BlockGroup &g : plan->groups) {
        if (g.memcpy_bytes > 0) {
            cudaError_t e = cudaMemcpyAsync(plan->dst.base + g.memcpy_dst, plan->src.base + g.memcpy_src,
                                            (size_t)g.memcpy_bytes, cudaMemcpyDeviceToDevice, st);
            if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync");
        } else {
            int rc = launch_op(plan, PDKV_OP_TRANSFER, s, d, g.tile_begin, g.tile_end - g.tile_begin, 0,
                               plan->L, st);
            if (rc != PDKV_OK) return rc;
        }
    }
    return PDKV_OK;
}

int pdkv_transfer_copies(const pdkv_plan *plan, int l0, int l1, void *stream)
{
    if (!plan || !plan->has_src || !plan->has_dst || !plan->dev_mem || !layers_ok(plan, l0, l1))
        return PDKV_ERR_INVALID_ARG;
    if (!plan->same_blocks) return PDKV_ERR_GEOMETRY;
    if (l0 == l1) return PDKV_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t strip = (size_t)plan->src.d.block_tokens * (size_t)plan->hrow_bytes;   // one (layer, K/V) of a block
    const size_t first = (size_t)2 * l0 * strip, n_lc = (size_t)2 * (l1 - l0);
    const std::vector<Tile> &tiles = plan->tiles[PDKV_OP_TRANSFER];
    for (const BlockGroup &g : plan->groups) {
        cudaError_t e = cudaSuccess;
        if (g.memcpy_bytes > 0) {   // a full block: its layers [l0, l1) are one contiguous range on both sides
            e = cudaMemcpyAsync(plan->dst.base + g.memcpy_dst + first, plan->src.base + g.memcpy_src + first,
                                n_lc * strip, cudaMemcpyDeviceToDevice, st);
        } else {                    // a partial block: the valid tokens of each strip, then zeros for the rest
            for (int32_t i = g.tile_begin; i < g.tile_end && e == cudaSuccess; ++i) {
                const Tile &t = tiles[(size_t)i];
                const size_t width = (size_t)t.ntok * (size_t)plan->hrow_bytes;
                if (t.src_off >= 0)
                    e = cudaMemcpy2DAsync(plan->dst.base + t.dst_off + first, strip, plan->src.base + t.src_off + first, strip,
                                          width, n_lc, cudaMemcpyDeviceToDevice, st);
                else
                    e = cudaMemset2DAsync(plan->dst.base + t.dst_off + first, strip, 0, width, n_lc, st);
            }
        }
        if (e != cudaSuccess) return cuda_fail(e, "block copy");
    }
    return PDKV_OK;
}

namespace {

// Copy whole blocks between a host image of a pool and the device pool, one
// (strided) copy per run of consecutive block ids.
int copy_block_runs(const pdkv_pool &pool, const std::vector<std::pair<int64_t, int64_t>> &runs,
                    char *host_base, bool to_device, int64_t row, int64_t hrow, cudaStream_t st)
{
    const pdkv_pool_desc &d = pool.d;
    const cudaMemcpyKind kind = to_device ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost;
    for (const auto &run : runs) {
        cudaError_t e;
        if (d.layout == PDKV_LAYOUT_BLOCK_MAJOR) {
            const size_t blk = (size_t)2 * d.num_layers * d.block_tokens * hrow;
            char *dev = pool.base + (size_t)run.first * blk, *host = host_base + (size_t)run.first * blk;
            e = cudaMemcpyAsync(to_device ? dev : host, to_device ? host : dev, (size_t)run.second * blk, kind, st);
        } else {  // [layer][K/V][block]...: 2*L pieces per run, one pitched copy
            const size_t blk = (size_t)d.num_kv_heads * d.block_tokens * row;
            const size_t pitch = (size_t)d.num_blocks * blk;
            char *dev = pool.base + (size_t)run.first * blk, *host = host_base + (size_t)run.first * blk;
            e = cudaMemcpy2DAsync(to_device ? dev : host, pitch, to_device ? host : dev, pitch,
                                  (size_t)run.second * blk, (size_t)2 * d.num_layers, kind, st);
        }
        if (e != cudaSuccess) return cuda_fail(e, to_device ? "host-to-device block copy" : "device-to-host block copy");
    }
    return PDKV_OK;
}

}  // namespace

int pdkv_upload_blocks(const pdkv_plan *plan, const void *host_src_pool, void *stream)
{
    if (!plan || !plan->has_src || !plan->dev_mem) return PDKV_ERR_INVALID_ARG;
    if (plan->src_runs.empty()) return PDKV_OK;
    if (!host_src_pool) return PDKV_ERR_INVALID_ARG;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    return copy_block_runs(plan->src, plan->src_runs, const_cast<char *>(static_cast<const char *>(host_src_pool)),
                           true, plan->row_bytes, plan->hrow_bytes, static_cast<cudaStream_t>(stream));
}

int pdkv_download_blocks(const pdkv_plan *plan, void *host_dst_pool, void *stream)
{
    if (!plan || !plan->has_dst || !plan->dev_mem) return PDKV_ERR_INVALID_ARG;
    if (plan->dst_runs.empty()) return PDKV_OK;
    if (!host_dst_pool) return PDKV_ERR_INVALID_ARG;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    return copy_block_runs(plan->dst, plan->dst_runs, static_cast<char *>(host_dst_pool), false, plan->row_bytes,
                           plan->hrow_bytes, static_cast<cudaStream_t>(stream));
}

int pdkv_plan_block_bytes(const pdkv_plan *plan, uint64_t *src_bytes, uint64_t *dst_bytes)
{
    if (!plan) return PDKV_ERR_INVALID_ARG;
    auto total = [&](const pdkv_pool &pool, const std::vector<std::pair<int64_t, int64_t>> &runs) {
        uint64_t n = 0;
        for (const auto &r : runs) n += (uint64_t)r.second;
        return n * 2ull * pool.d.num_layers * pool.d.block_tokens * (uint64_t)plan->hrow_bytes;
    };
    if (src_bytes) *src_bytes = plan->has_src ? total(plan->src, plan->src_runs) : 0;
    if (dst_bytes) *dst_bytes = plan->has_dst ? total(plan->dst, plan->dst_runs) : 0;
    return PDKV_OK;
}

int pdkv_plan_launches(const pdkv_plan *plan, int op, int64_t *launches)
{
    if (!plan || !launches || op < 0 || op > 3) return PDKV_ERR_INVALID_ARG;
    if (op == 3)
        *launches = (int64_t)plan->groups.size();
    else
        *launches = plan->tiles[op].empty() ? 0 : 1;
    return PDKV_OK;
}

int pdkv_plan_tiles(const pdkv_plan *plan, int op, const pdkv_tile **tiles, int64_t *n_tiles)
{
    if (!plan || op < 0 || op > 2 || !tiles || !n_tiles) return PDKV_ERR_INVALID_ARG;
    static_assert(sizeof(pdkv_tile) == sizeof(Tile), "public and internal tile records must match");
    *tiles = reinterpret_cast<const pdkv_tile *>(plan->tiles[op].data());
    *n_tiles = (int64_t)plan->tiles[op].size();
    return PDKV_OK;
}

int pdkv_plan_status(const pdkv_plan *plan, void *stream)
{
    if (!plan || !plan->dev_mem) return PDKV_ERR_INVALID_ARG;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    unsigned long long word[2] = {0, 0};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(word, plan->dev_status, sizeof(word), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "status read");
    if (word[0]) {
        char msg[96];
        if (word[0] == 2)
            std::snprintf(msg, sizeof(msg), "a bulk-copy wait gave up at work item %lld", (long long)word[1]);
        else
            std::snprintf(msg, sizeof(msg), "refused access at byte offset %lld", (long long)word[1]);
        g_cuda_msg = msg;
        return PDKV_ERR_DEVICE_BOUNDS;
    }
    return PDKV_OK;
}

int pdkv_tune(const char *key, int64_t value)
{
    if (!key) return PDKV_ERR_INVALID_ARG;
    pdkv::Tunables &t = pdkv::tunables();
    const std::string k(key);
    if (k == "tile_bytes" && value >= 1 && value <= (1ll << 30)) t.tile_bytes = value;
    else if (k == "ctas_per_sm" && value >= 0 && value <= 32) t.ctas_per_sm = value;
    else if (k == "max_ctas" && value >= 0 && value <= 65535) t.max_ctas = value;
    else if (k == "threads" && (value == 0 || (value >= 32 && value <= 1024 && value % 32 == 0))) t.threads = value;
    else if (k == "unroll" && (value == 0 || value == 1 || value == 2 || value == 4 || value == 8)) t.unroll = value;
    else if (k == "vec32" && (value == 0 || value == 1)) t.vec32 = value;
    else if (k == "lc_fastest" && (value == 0 || value == 1)) t.lc_fastest = value;
    else if (k == "chunked" && (value == 0 || value == 1)) t.chunked = value;
    else if (k == "lc_skew" && value >= -1 && value <= 1024 && (value < 0 || (value & (value - 1)) == 0)) t.lc_skew = value;
    else if (k == "lc_skew_shift" && value >= 0 && value <= 20) t.lc_skew_shift = value;
    else if (k == "group_threads" && (value == 0 || (value >= 32 && value <= 1024 && value % 32 == 0))) t.group_threads = value;
    else if (k == "debug_bounds" && (value == 0 || value == 1)) t.debug_bounds = value;
    else if (k == "debug_shrink" && value >= 0) t.debug_shrink = value;
    else if (k == "variant" && value >= -1 && value <= 3) t.variant = value;
    else if (k == "stages" && value >= 2 && value <= 16) t.stages = value;
    else if (k == "dry_run" && (value == 0 || value == 1)) t.dry_run = value;
    else if (k == "autotune_reuse" && (value == 0 || value == 1)) t.autotune_reuse = value;
    else if (k == "src_order" && value >= -1 && value <= 1) t.src_order = value;
    else return PDKV_ERR_INVALID_ARG;
    return PDKV_OK;
}

int pdkv_tune_get(const char *key, int64_t *value)
{
    if (!key || !value) return PDKV_ERR_INVALID_ARG;
    const pdkv::Tunables &t = pdkv::tunables();
    const std::string k(key);
    if (k == "tile_bytes") *value = t.tile_bytes;
    else if (k == "ctas_per_sm") *value = t.ctas_per_sm;
    else if (k == "max_ctas") *value = t.max_ctas;
    else if (k == "threads") *value = t.threads;
    else if (k == "unroll") *value = t.unroll;
    else if (k == "vec32") *value = t.vec32;
    else if (k == "lc_fastest") *value = t.lc_fastest;
    else if (k == "chunked") *value = t.chunked;
    else if (k == "lc_skew") *value = t.lc_skew;
    else if (k == "lc_skew_shift") *value = t.lc_skew_shift;
    else if (k == "group_threads") *value = t.group_threads;
    else if (k == "debug_bounds") *value = t.debug_bounds;
    else if (k == "debug_shrink") *value = t.debug_shrink;
    else if (k == "variant") *value = t.variant;
    else if (k == "stages") *value = t.stages;
    else if (k == "dry_run") *value = t.dry_run;
    else if (k == "autotune_reuse") *value = t.autotune_reuse;
    else if (k == "src_order") *value = t.src_order;
    else return PDKV_ERR_INVALID_ARG;
    return PDKV_OK;
}

const char *pdkv_strerror(int status)
{
    switch (status) {
    case PDKV_OK: return "ok";
    case PDKV_ERR_INVALID_ARG: return "invalid argument";
    case PDKV_ERR_GEOMETRY: return "invalid or mismatched pool geometry";
    case PDKV_ERR_TABLE: return "invalid block table";
    case PDKV_ERR_BUFFER_TOO_SMALL: return "contiguous buffer too small";
    case PDKV_ERR_CUDA: return g_cuda_msg.empty() ? "CUDA error" : g_cuda_msg.c_str();
    case PDKV_ERR_DEVICE_BOUNDS: return g_cuda_msg.empty() ? "device bounds check refused an access" : g_cuda_msg.c_str();
    case PDKV_ERR_NOMEM: return "out of host memory";
    case PDKV_ERR_BUSY: return "no free receive slot";
    case PDKV_ERR_LIMIT: return "batch exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
    }
}

}  // extern "C"
