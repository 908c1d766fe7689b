// Bulk-copy variant of the tile copy: one warp per CTA drives the TMA unit
// (cp.async.bulk global -> shared -> global, mbarrier-tracked) through a ring
// of shared-memory stages, one tile per stage.  No data passes through
// registers, so the kernel occupies one warp and a few registers per CTA: this
// is the "operator" form of RecvScatter that leaves the SMs' issue slots and
// register file to whatever else runs in the stream (Sec. 3.5: as an operator the
// scatter runs beside the stream's other operators without holding them up).
//
// A tile is staged in *destination order*.  Towards a head-major pool that is
// [head][token][row]: the H stores are contiguous runs of ntok*ROW bytes and
// the loads are one bulk copy per row when the source is token-major (the
// head<->token transpose happens in the load addresses), or one per head when
// the source is head-major too.  Towards a token-major side (block-major pool
// or the contiguous buffer) the stage is [token][head][row] and the store is a
// single bulk copy.
//
// With "variant" 2 the transpose of a token-major source into a head-major
// destination is done by the TMA unit itself: the source side (a block-major
// pool or the contiguous buffer, both a dense [token row][head][dim] array) is
// described by a 3-D tensor map, and one tiled load with the box
// (dim = D, head = 1, tokens = T) fetches the T strided rows of one head into a
// dense [T][D] piece of the stage -- H loads per tile instead of one per row.
// The innermost coordinate of every load is 0 (16-byte rule), stage pieces are
// 128-byte aligned, and a box may over-read past a ragged tile (reads only;
// out-of-range rows are zero-filled by the hardware and never stored).
// The opposite direction (head-major source, token-major destination) uses the
// same map for tiled *stores*: the stage is filled by one contiguous run per
// head and one tiled store per head scatters its T rows; a ragged tile (fewer
// than T tokens) must not write a full box and falls back to per-row stores.
//
// Every wait is bounded: after kSpinLimit failed polls the warp records an
// error word, drains its own stores and returns.
#include <cstring>

#include <cuda.h>

#include "pdkv_device.cuh"
#include "pdkv_internal.h"

namespace pdkv {

namespace {

constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kBarrierBytes = 128;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *b, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect(uint64_t *b, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *b)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *b, uint32_t phase)
{
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(smem_u32(b)), "r"(phase)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(void *sdst, const void *gsrc, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(sdst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// Tiled 3-D load: box (D, 1, T) at coordinates (0, head, token row).
__device__ __forceinline__ void tensor_g2s(void *sdst, const CUtensorMap *map, int head, int tok_row, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
            smem_u32(sdst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(head), "r"(tok_row), "r"(smem_u32(bar))
        : "memory");
}
// Tiled 3-D store of a dense [T][D] piece to the box at (0, head, token row); never negative coordinates.
__device__ __forceinline__ void tensor_s2g(const CUtensorMap *map, int head, int tok_row, const void *ssrc)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(0), "r"(head), "r"(tok_row), "r"(smem_u32(ssrc))
                 : "memory");
}
__device__ __forceinline__ void bulk_s2g(void *gdst, const void *ssrc, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(ssrc)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

struct Item {
    int64_t s_base, d_base;
    uint32_t ntok;
    bool zero;
};

// Vector type of the staged kernel's stores: 16 bytes (one shared-memory load) or 32 (two).
template <int W> struct StoreVec;
template <> struct StoreVec<16> {
    using type = uint4;
    static __device__ __forceinline__ uint4 zero() { return make_uint4(0, 0, 0, 0); }
    static __device__ __forceinline__ uint4 load_shared(const unsigned char *s) { return *reinterpret_cast<const uint4 *>(s); }
    static __device__ __forceinline__ void store_global(char *g, const uint4 &v) { __stcs(reinterpret_cast<uint4 *>(g), v); }
};
template <> struct StoreVec<32> {
    struct type {
        uint4 lo, hi;
    };
    static __device__ __forceinline__ type zero() { return {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)}; }
    static __device__ __forceinline__ type load_shared(const unsigned char *s)
    {
        return {*reinterpret_cast<const uint4 *>(s), *reinterpret_cast<const uint4 *>(s + 16)};
    }
    static __device__ __forceinline__ void store_global(char *g, const type &v)
    {
        asm volatile("st.global.cs.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};" ::"r"(v.lo.x), "r"(v.lo.y), "r"(v.lo.z),
                     "r"(v.lo.w), "r"(v.hi.x), "r"(v.hi.y), "r"(v.hi.z), "r"(v.hi.w), "l"(g)
                     : "memory");
    }
};

}  // namespace

__global__ void __launch_bounds__(32)
bulk_tiles_kernel(const CopyParams p, const int stages, const uint32_t stage_bytes,
                  const __grid_constant__ CUtensorMap tok_map, const int map_tokens)
{
    // map_tokens > 0: tok_map describes the token-major side (source or destination) as
    // [token row][head][dim] and its box holds map_tokens tokens of one head; used for tiles
    // whose two sides differ in order
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem);
    unsigned char *data = smem + kBarrierBytes;
    const uint32_t lane = threadIdx.x;
    const uint32_t H = (uint32_t)p.H;
    const uint32_t row = (uint32_t)p.row_bytes;
    const int64_t hrow = (int64_t)p.H * p.row_bytes;
    const bool src_tok_major = p.src.tok_stride >= p.src.head_stride;
    const bool dst_tok_major = p.dst.tok_stride >= p.dst.head_stride;
    const bool src_flat = p.src.head_stride == p.row_bytes && p.src.tok_stride == hrow;
    const bool dst_flat = p.dst.head_stride == p.row_bytes && p.dst.tok_stride == hrow;
    const uint32_t m_H = div_magic(H);
    const bool tiled = map_tokens > 0 && src_tok_major && !dst_tok_major;       // tiled loads
    const bool tiled_out = map_tokens > 0 && !src_tok_major && dst_tok_major;   // tiled stores
    const uint32_t piece = (tiled || tiled_out) ? (uint32_t)map_tokens * row : 0;   // stage bytes per head

    if (lane == 0) {
        for (int i = 0; i < stages; ++i) mbar_init(full + i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    int64_t first, step, n_mine;
    if (p.chunked) {
        const int64_t per = (n_work + gridDim.x - 1) / gridDim.x;
        first = (int64_t)blockIdx.x * per;
        const int64_t end = first + per < n_work ? first + per : n_work;
        n_mine = end > first ? end - first : 0;
        step = 1;
    } else {
        first = blockIdx.x;
        step = gridDim.x;
        n_mine = n_work > first ? (n_work - first + step - 1) / step : 0;
    }

    auto item = [&](int64_t j) {
        const int64_t w = first + j * step;
        int32_t ti, lci;
        if (p.lc_fastest) {
            ti = (int32_t)(w / p.n_lc);
            lci = (int32_t)(w - (int64_t)ti * p.n_lc);
        } else {
            lci = (int32_t)(w / p.n_tiles);
            ti = (int32_t)(w - (int64_t)lci * p.n_tiles);
        }
        const Tile t = p.tiles[p.tile_begin + ti];
        const int64_t lc = p.lc_begin + lci;
        const int64_t buf_lc = (int64_t)t.n_kept * hrow;
        Item it;
        it.s_base = t.src_off + lc * (p.src.lc_stride >= 0 ? p.src.lc_stride : buf_lc);
        it.d_base = t.dst_off + lc * (p.dst.lc_stride >= 0 ? p.dst.lc_stride : buf_lc);
        it.ntok = (uint32_t)t.ntok;
        it.zero = t.src_off < 0;
        return it;
    };

    // Fill stage (j % stages) with item j, laid out in destination order.
    auto issue_load = [&](int64_t j) {
        const Item it = item(j);
        uint64_t *bar = full + (j % stages);
        unsigned char *st = data + (size_t)(j % stages) * stage_bytes;
        const uint32_t bytes = it.ntok * H * row;
        if (it.zero) {                      // nothing to fetch; the store side writes zeros itself
            if (lane == 0) mbar_arrive(bar);
            return;
        }
        if (tiled) {                        // H boxes of map_tokens x row bytes, whatever ntok is
            if (lane == 0) mbar_arrive_expect(bar, H * piece);
            __syncwarp();
            const int tok_row = (int)(it.s_base / hrow);
            for (uint32_t hd = lane; hd < H; hd += 32) tensor_g2s(st + (size_t)hd * piece, &tok_map, (int)hd, tok_row, bar);
            return;
        }
        if (lane == 0) mbar_arrive_expect(bar, bytes);
        __syncwarp();
        const char *src = p.src.base + it.s_base;
        if (tiled_out) {                    // stage [head][map_tokens][row]: one contiguous run per head
            const uint32_t run = it.ntok * row;
            for (uint32_t hd = lane; hd < H; hd += 32) bulk_g2s(st + (size_t)hd * piece, src + hd * p.src.head_stride, run, bar);
            return;
        }
        if (src_flat && dst_flat) {                     // one contiguous run on both sides
            if (lane == 0) bulk_g2s(st, src, bytes, bar);
        } else if (src_tok_major == dst_tok_major) {    // same order: one run per head (or per token)
            const uint32_t outer = dst_tok_major ? it.ntok : H;
            const uint32_t run = (dst_tok_major ? H : it.ntok) * row;
            const int64_t s_outer = dst_tok_major ? p.src.tok_stride : p.src.head_stride;
            const int64_t s_inner = dst_tok_major ? p.src.head_stride : p.src.tok_stride;
            if (s_inner == (int64_t)row) {
                for (uint32_t o = lane; o < outer; o += 32) bulk_g2s(st + (size_t)o * run, src + o * s_outer, run, bar);
            } else {                                    // rows of a run are not adjacent in the source
                const uint32_t inner = dst_tok_major ? H : it.ntok;
                const uint32_t m_in = dst_tok_major ? m_H : div_magic(inner);
                for (uint32_t r = lane; r < outer * inner; r += 32) {
                    const uint32_t o = fast_div(r, m_in), i = r - o * inner;
                    bulk_g2s(st + (size_t)r * row, src + o * s_outer + i * s_inner, row, bar);
                }
            }
        } else {                                        // transpose: one bulk copy per row
            const uint32_t inner = dst_tok_major ? H : it.ntok;   // inner index of the stage layout
            const uint32_t m_in = dst_tok_major ? m_H : div_magic(inner);
            const uint32_t rows = it.ntok * H;
            for (uint32_t r = lane; r < rows; r += 32) {
                const uint32_t o = fast_div(r, m_in), i = r - o * inner;
                const uint32_t tk = dst_tok_major ? o : i, hd = dst_tok_major ? i : o;
                bulk_g2s(st + (size_t)r * row, src + tk * p.src.tok_stride + hd * p.src.head_stride, row, bar);
            }
        }
    };

    // Write item j from its stage (or zeros) to the destination.
    auto issue_store = [&](int64_t j) {
        const Item it = item(j);
        unsigned char *st = data + (size_t)(j % stages) * stage_bytes;
        char *dst = p.dst.base + it.d_base;
        if (it.zero) {                      // tail slots: plain 16-byte stores of zeros
            const uint32_t vpr = row / 16;
            const uint32_t outer = dst_tok_major ? it.ntok : H, inner = dst_tok_major ? H : it.ntok;
            const int64_t d_outer = dst_tok_major ? p.dst.tok_stride : p.dst.head_stride;
            const int64_t d_inner = dst_tok_major ? p.dst.head_stride : p.dst.tok_stride;
            const uint32_t m_vpr = div_magic(vpr), m_in = div_magic(inner);
            const uint32_t nvec = outer * inner * vpr;
            for (uint32_t v = lane; v < nvec; v += 32) {
                const uint32_t r = fast_div(v, m_vpr), vv = v - r * vpr;
                const uint32_t o = fast_div(r, m_in), i = r - o * inner;
                __stcs(reinterpret_cast<uint4 *>(dst + o * d_outer + i * d_inner + (int64_t)vv * 16),
                       make_uint4(0, 0, 0, 0));
            }
            return;
        }
        if (tiled_out) {
            if (it.ntok == (uint32_t)map_tokens) {      // a full box per head
                const int tok_row = (int)(it.d_base / hrow);
                for (uint32_t hd = lane; hd < H; hd += 32) tensor_s2g(&tok_map, (int)hd, tok_row, st + (size_t)hd * piece);
            } else {                                    // ragged tile: row by row, nothing past its end
                const uint32_t rows = it.ntok * H;
                for (uint32_t r = lane; r < rows; r += 32) {
                    const uint32_t tk = fast_div(r, m_H), hd = r - tk * H;
                    bulk_s2g(dst + tk * p.dst.tok_stride + hd * p.dst.head_stride, st + (size_t)hd * piece + (size_t)tk * row, row);
                }
            }
        } else if (dst_flat) {
            if (lane == 0) bulk_s2g(dst, st, it.ntok * H * row);
        } else if (dst_tok_major) {         // token-major with gaps between tokens cannot occur for our sides,
            for (uint32_t tk = lane; tk < it.ntok; tk += 32)   // but keep it correct: one run per token
                bulk_s2g(dst + tk * p.dst.tok_stride, st + (size_t)tk * H * row, H * row);
        } else {                            // head-major: one run per head
            const uint32_t run = it.ntok * row;
            const uint32_t pitch = tiled ? piece : run;   // tiled stages keep map_tokens rows per head
            for (uint32_t hd = lane; hd < H; hd += 32) bulk_s2g(dst + hd * p.dst.head_stride, st + (size_t)hd * pitch, run);
        }
        bulk_commit();
    };

    int64_t head = 0;
    for (int64_t tail = 0; tail < n_mine; ++tail) {
        while (head < n_mine && head < tail + stages) {
            if (head >= stages) {           // the stage was read by an earlier store of this warp
                bulk_wait_read_all();
                __syncwarp();
            }
            issue_load(head);
            ++head;
        }
        uint64_t *bar = full + (tail % stages);
        const uint32_t phase = (uint32_t)((tail / stages) & 1);
        uint32_t spins = 0;
        bool ok = true;
        while (!mbar_try_wait(bar, phase)) {
            if (++spins > kSpinLimit) {
                ok = false;
                break;
            }
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {                           // give up: record where, drain our stores, leave
            if (lane == 0 && atomicCAS(p.status, 0ull, 2ull) == 0ull) p.status[1] = (unsigned long long)tail;
            bulk_wait_all();
            for (int64_t j = tail + 1; j < head; ++j) {   // loads still aimed at our stages: bounded wait each
                uint32_t s2 = 0;
                while (!mbar_try_wait(full + (j % stages), (uint32_t)((j / stages) & 1)) && ++s2 <= kSpinLimit) {}
            }
            return;
        }
        issue_store(tail);
    }
    bulk_wait_all();
}

// "variant" 3: staged transpose.  For tiles whose two sides differ in order (one token-major,
// one head-major) the tile is fetched in the order of the side that is READ -- one bulk copy of
// the whole contiguous [token][head][dim] strip when that side is token-major, one contiguous
// run per head when it is head-major -- into a ring of shared-memory stages, and all threads of
// the CTA then write it out in the order of the side that is WRITTEN with coalesced vector stores
// (consecutive lanes, consecutive addresses).  Neither side ever sees a lone row: every DRAM
// sector pair that is fetched is used in full, whatever the row size (rows of 160 bytes read one
// at a time fetch 192).  One mbarrier per stage counts the bytes of its loads; one
// __syncthreads per tile hands the stage back.  Waits are bounded as in bulk_tiles_kernel.
template <int W>
__global__ void __launch_bounds__(512)
staged_tiles_kernel(const CopyParams p, const int stages, const uint32_t stage_bytes)
{
    using V = typename StoreVec<W>::type;
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem);
    unsigned char *data = smem + kBarrierBytes;
    const uint32_t tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31u;
    const uint32_t H = (uint32_t)p.H;
    const uint32_t row = (uint32_t)p.row_bytes;
    const uint32_t vpr = row / W;
    const int64_t hrow = (int64_t)p.H * p.row_bytes;
    const bool src_tok_major = p.src.tok_stride >= p.src.head_stride;   // the destination is the other way round
    const uint32_t m_H = div_magic(H), m_vpr = div_magic(vpr);

    if (tid == 0) {
        for (int i = 0; i < stages; ++i) mbar_init(full + i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    int64_t first, step, n_mine;
    if (p.chunked) {
        const int64_t per = (n_work + gridDim.x - 1) / gridDim.x;
        first = (int64_t)blockIdx.x * per;
        const int64_t end = first + per < n_work ? first + per : n_work;
        n_mine = end > first ? end - first : 0;
        step = 1;
    } else {
        first = blockIdx.x;
        step = gridDim.x;
        n_mine = n_work > first ? (n_work - first + step - 1) / step : 0;
    }

    auto item = [&](int64_t j) {
        const int64_t w = first + j * step;
        int32_t ti, lci;
        if (p.lc_fastest) {
            ti = (int32_t)(w / p.n_lc);
            lci = (int32_t)(w - (int64_t)ti * p.n_lc);
        } else {
            lci = (int32_t)(w / p.n_tiles);
            ti = (int32_t)(w - (int64_t)lci * p.n_tiles);
        }
        if (p.lc_skew > 1) {   // as in the register-copy kernel: neighbouring tiles take different strips
            lci += (ti >> p.lc_skew_shift) & (p.lc_skew - 1);
            if (lci >= p.n_lc) lci -= p.n_lc;
        }
        const Tile t = p.tiles[p.tile_begin + ti];
        const int64_t lc = p.lc_begin + lci;
        const int64_t buf_lc = (int64_t)t.n_kept * hrow;
        Item it;
        it.s_base = t.src_off + lc * (p.src.lc_stride >= 0 ? p.src.lc_stride : buf_lc);
        it.d_base = t.dst_off + lc * (p.dst.lc_stride >= 0 ? p.dst.lc_stride : buf_lc);
        it.ntok = (uint32_t)t.ntok;
        it.zero = t.src_off < 0;
        return it;
    };

    // Warp 0 fills stage (j % stages) with item j in the order of the source.
    auto issue_load = [&](int64_t j) {
        const Item it = item(j);
        uint64_t *bar = full + (j % stages);
        unsigned char *st = data + (size_t)(j % stages) * stage_bytes;
        if (it.zero) {                      // nothing to fetch: the stores write zeros
            if (lane == 0) mbar_arrive(bar);
            return;
        }
        if (lane == 0) mbar_arrive_expect(bar, it.ntok * H * row);
        __syncwarp();
        const char *src = p.src.base + it.s_base;
        if (src_tok_major) {                // the tile is one contiguous strip of the source
            if (lane == 0) bulk_g2s(st, src, it.ntok * H * row, bar);
        } else {                            // one contiguous run of ntok rows per head
            const uint32_t run = it.ntok * row;
            for (uint32_t hd = lane; hd < H; hd += 32) bulk_g2s(st + (size_t)hd * run, src + hd * p.src.head_stride, run, bar);
        }
    };

    int64_t head = 0;
    for (int64_t tail = 0; tail < n_mine; ++tail) {
        if (tid < 32) {                     // the stages being refilled were handed back at the last barrier
            while (head < n_mine && head < tail + stages) {
                issue_load(head);
                ++head;
            }
        }
        const Item it = item(tail);
        const unsigned char *st = data + (size_t)(tail % stages) * stage_bytes;
        uint32_t spins = 0;
        bool ok = true;
        while (!mbar_try_wait(full + (tail % stages), (uint32_t)((tail / stages) & 1))) {
            if (++spins > kSpinLimit) {
                ok = false;
                break;
            }
        }
        if (ok) {
            // vectors in the order of the destination: (head, token) towards a head-major side,
            // (token, head) towards a token-major one; the stage holds the order of the source
            char *dst = p.dst.base + it.d_base;
            const uint32_t ntok = it.ntok;
            const uint32_t nvec = ntok * H * vpr;
            const uint32_t inner = src_tok_major ? ntok : H;
            const uint32_t m_inner = src_tok_major ? div_magic(ntok) : m_H;
            constexpr int U = 4;
            for (uint32_t i0 = tid; i0 < nvec; i0 += nthr * U) {
                V v[U];
                int64_t doff[U];
#pragma unroll
                for (int k = 0; k < U; ++k) {
                    const uint32_t i = i0 + k * nthr;
                    doff[k] = -1;
                    if (i < nvec) {
                        const uint32_t r = fast_div(i, m_vpr), vv = i - r * vpr;
                        const uint32_t o = fast_div(r, m_inner), in = r - o * inner;
                        const uint32_t hd = src_tok_major ? o : in, tk = src_tok_major ? in : o;
                        const uint32_t soff = (src_tok_major ? tk * H + hd : hd * ntok + tk) * row + vv * W;
                        doff[k] = tk * p.dst.tok_stride + hd * p.dst.head_stride + (int64_t)vv * W;
                        v[k] = it.zero ? StoreVec<W>::zero() : StoreVec<W>::load_shared(st + soff);
                    }
                }
#pragma unroll
                for (int k = 0; k < U; ++k)
                    if (doff[k] >= 0) StoreVec<W>::store_global(dst + doff[k], v[k]);
            }
        }
        // hands the stage back to warp 0, and makes the outcome of the wait CTA-wide
        if (!__syncthreads_and(ok ? 1 : 0)) {
            if (tid == 0 && atomicCAS(p.status, 0ull, 2ull) == 0ull) p.status[1] = (unsigned long long)tail;
            if (tid < 32)                    // loads still aimed at our stages: bounded wait each
                for (int64_t j = tail + 1; j < head; ++j) {
                    uint32_t s2 = 0;
                    while (!mbar_try_wait(full + (j % stages), (uint32_t)((j / stages) & 1)) && ++s2 <= kSpinLimit) {}
                }
            return;
        }
    }
}

namespace {

using EncodeTiled = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiled encode_tiled()
{
    static EncodeTiled fn = [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            sym = nullptr;
        return reinterpret_cast<EncodeTiled>(sym);
    }();
    return fn;
}

// Tensor map of a token-major side (a block-major pool or the contiguous buffer, flat
// [token rows][H][D]); box = (D, 1, tokens).
// Returns false when the geometry does not meet the TMA rules (the caller then
// uses per-row bulk copies).
bool make_token_major_map(const CopyParams &p, const Side &side, int elem_bytes, int tokens, CUtensorMap *out)
{
    const int64_t row = p.row_bytes, hrow = (int64_t)p.H * row;
    if (elem_bytes != 1 && elem_bytes != 2 && elem_bytes != 4 && elem_bytes != 8) return false;
    const int64_t D = row / elem_bytes;
    const int64_t rows = side.size / hrow;
    if (!encode_tiled() || D < 1 || D > 256 || tokens < 1 || tokens > 256 || row % 16 || rows < 1 ||
        rows > 0x7FFFFFFFll || ((int64_t)tokens * row) % 128 || (reinterpret_cast<uintptr_t>(side.base) & 15u) ||
        hrow >= (1ll << 40))
        return false;
    const CUtensorMapDataType dt = elem_bytes == 1   ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                   : elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16
                                   : elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32
                                                     : CU_TENSOR_MAP_DATA_TYPE_UINT64;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)p.H, (cuuint64_t)rows};
    const cuuint64_t strides[2] = {(cuuint64_t)row, (cuuint64_t)hrow};   // bytes, dimensions 1 and 2
    const cuuint32_t box[3] = {(cuuint32_t)D, 1u, (cuuint32_t)tokens};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    return encode_tiled()(out, dt, 3, side.base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_bulk(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream)
{
    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    if (n_work <= 0) return cudaSuccess;
    const uint32_t stage_bytes = (uint32_t)((cfg.max_tile_bytes + 127) / 128 * 128);
    CUtensorMap map;
    std::memset(&map, 0, sizeof(map));
    int map_tokens = 0;
    const bool src_tok_major = p.src.tok_stride >= p.src.head_stride;
    const bool dst_tok_major = p.dst.tok_stride >= p.dst.head_stride;
    if (cfg.variant == 2 && src_tok_major != dst_tok_major) {
        const Side &side = src_tok_major ? p.src : p.dst;
        const int64_t hrow = (int64_t)p.H * p.row_bytes;
        const bool side_flat = side.head_stride == p.row_bytes && side.tok_stride == hrow;
        const int tokens = (int)(cfg.max_tile_bytes / hrow);
        if (side_flat && make_token_major_map(p, side, cfg.elem_bytes, tokens, &map)) map_tokens = tokens;
    }
    const int stages = cfg.stages;
    const size_t smem = kBarrierBytes + (size_t)stages * stage_bytes;
    cudaError_t e = cudaFuncSetAttribute(bulk_tiles_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, bulk_tiles_kernel, 32, smem);
    if (e != cudaSuccess) return e;
    if (occ < 1) return cudaErrorInvalidConfiguration;
    if (occ > cfg.ctas_per_sm) occ = cfg.ctas_per_sm;
    int64_t grid = (int64_t)cfg.sm_count * occ;
    if (cfg.max_ctas > 0 && grid > cfg.max_ctas) grid = cfg.max_ctas;
    if (grid > n_work) grid = n_work;
    bulk_tiles_kernel<<<(unsigned)grid, 32, smem, stream>>>(p, stages, stage_bytes, map, map_tokens);
    return cudaGetLastError();
}

// Staged transpose ("variant" 3): the two sides differ in order, the token-major one is a dense
// [token][head][dim] array, the head-major one keeps the tokens of a head adjacent.
bool staged_supported(const CopyParams &p, const LaunchConfig &cfg)
{
    const int64_t row = p.row_bytes, hrow = (int64_t)p.H * row;
    const bool src_tok_major = p.src.tok_stride >= p.src.head_stride;
    const bool dst_tok_major = p.dst.tok_stride >= p.dst.head_stride;
    if (src_tok_major == dst_tok_major) return false;
    const Side &tm = src_tok_major ? p.src : p.dst, &hm = src_tok_major ? p.dst : p.src;
    const size_t smem = kBarrierBytes + (size_t)cfg.stages * ((cfg.max_tile_bytes + 127) / 128 * 128);
    return row % 16 == 0 && tm.tok_stride == hrow && tm.head_stride == row && hm.tok_stride == row &&
           cfg.max_tile_bytes > 0 && cfg.max_tile_bytes <= 131072 && smem <= 220 * 1024 && cfg.stages >= 2 &&
           !cfg.check_bounds && ((reinterpret_cast<uintptr_t>(p.src.base) | reinterpret_cast<uintptr_t>(p.dst.base)) & 15u) == 0;
}

cudaError_t launch_staged(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream)
{
    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    if (n_work <= 0) return cudaSuccess;
    const uint32_t stage_bytes = (uint32_t)((cfg.max_tile_bytes + 127) / 128 * 128);
    const int stages = cfg.stages;
    const size_t smem = kBarrierBytes + (size_t)stages * stage_bytes;
    const bool wide = p.row_bytes % 32 == 0 &&
                      ((reinterpret_cast<uintptr_t>(p.dst.base) | (uintptr_t)p.dst.head_stride | (uintptr_t)p.dst.tok_stride) & 31u) == 0;
    auto kern = wide ? staged_tiles_kernel<32> : staged_tiles_kernel<16>;
    int threads = cfg.threads < 64 ? 64 : (cfg.threads > 512 ? 512 : cfg.threads / 32 * 32);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, threads, smem);
    if (e != cudaSuccess) return e;
    if (occ < 1) return cudaErrorInvalidConfiguration;
    if (occ > cfg.ctas_per_sm) occ = cfg.ctas_per_sm;
    int64_t grid = (int64_t)cfg.sm_count * occ;
    if (cfg.max_ctas > 0 && grid > cfg.max_ctas) grid = cfg.max_ctas;
    if (grid > n_work) grid = n_work;
    kern<<<(unsigned)grid, threads, smem, stream>>>(p, stages, stage_bytes);
    return cudaGetLastError();
}

// The bulk path needs 16-byte rows and a tile that fits a stage (and the
// mbarrier's transaction counter); otherwise the register path is used.
bool bulk_supported(const LaunchConfig &cfg, int row_bytes)
{
    const size_t smem = kBarrierBytes + (size_t)cfg.stages * ((cfg.max_tile_bytes + 127) / 128 * 128);
    return row_bytes % 16 == 0 && cfg.vec_bytes >= 16 && cfg.max_tile_bytes > 0 && cfg.max_tile_bytes <= 131072 &&
           smem <= 220 * 1024 && cfg.stages >= 2 && !cfg.check_bounds;
}

}  // namespace pdkv
