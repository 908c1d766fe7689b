// sm_100a kernels for the paged-KVCache transfer: one persistent grid walks a
// list of (tile, layer, K/V) work items and moves whole head rows (D*E bytes)
// between a block-fixed pool and the contiguous buffer, or pool to pool.
//
// The path is pure data movement (Sec. 3.5: organise blocks into a contiguous
// buffer, restore blocks from bytes), so the only resource that matters is HBM
// bandwidth: accesses are 32 (or 16) bytes per lane, every warp touches whole
// rows, and the number of bytes each SM keeps in flight is a launch parameter
// (threads x CTAs x unroll), because on B200 a copy runs fastest with about
// 32-64 KiB of loads outstanding per SM, not with as many as fit.
#pragma once

#include "pdkv_device.cuh"
#include "pdkv_internal.h"

namespace pdkv {

struct alignas(32) Vec32 {
    unsigned int a[8];
};

template <int W> struct VecT;
template <> struct VecT<32> { using type = Vec32; };
template <> struct VecT<16> { using type = uint4; };
template <> struct VecT<8> { using type = uint2; };
template <> struct VecT<4> { using type = unsigned int; };
template <> struct VecT<2> { using type = unsigned short; };
template <> struct VecT<1> { using type = unsigned char; };

template <typename V> __device__ __forceinline__ V zero_vec();
template <> __device__ __forceinline__ Vec32 zero_vec<Vec32>()
{
    Vec32 v;
#pragma unroll
    for (int i = 0; i < 8; ++i) v.a[i] = 0u;
    return v;
}
template <> __device__ __forceinline__ uint4 zero_vec<uint4>() { return make_uint4(0, 0, 0, 0); }
template <> __device__ __forceinline__ uint2 zero_vec<uint2>() { return make_uint2(0, 0); }
template <> __device__ __forceinline__ unsigned int zero_vec<unsigned int>() { return 0u; }
template <> __device__ __forceinline__ unsigned short zero_vec<unsigned short>() { return 0; }
template <> __device__ __forceinline__ unsigned char zero_vec<unsigned char>() { return 0; }

// Threads per CTA the register budget allows: W*U/4 data registers per thread
// plus addressing must stay below 65536 / threads.
constexpr int max_threads(int w, int u) { return w * u >= 256 ? 256 : (w * u >= 128 ? 512 : 1024); }

// Streaming (evict-first) global accesses; the 32-byte forms are single
// 256-bit instructions on sm_100.
template <typename V> __device__ __forceinline__ V ld_stream(const char *p)
{
    return __ldcs(reinterpret_cast<const V *>(p));
}
template <> __device__ __forceinline__ Vec32 ld_stream<Vec32>(const char *p)
{
    Vec32 v;
    asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.a[0]), "=r"(v.a[1]), "=r"(v.a[2]), "=r"(v.a[3]), "=r"(v.a[4]), "=r"(v.a[5]),
                   "=r"(v.a[6]), "=r"(v.a[7])
                 : "l"(p));
    return v;
}
template <typename V> __device__ __forceinline__ void st_stream(char *p, const V &v)
{
    __stcs(reinterpret_cast<V *>(p), v);
}
template <> __device__ __forceinline__ void st_stream<Vec32>(char *p, const Vec32 &v)
{
    asm volatile("st.global.cs.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};" ::"r"(v.a[0]), "r"(v.a[1]),
                 "r"(v.a[2]), "r"(v.a[3]), "r"(v.a[4]), "r"(v.a[5]), "r"(v.a[6]), "r"(v.a[7]), "l"(p)
                 : "memory");
}

__device__ __forceinline__ bool in_bounds(int64_t off, int width, int64_t size)
{
    return off >= 0 && off + width <= size;
}

__device__ __forceinline__ void refuse(unsigned long long *status, int64_t off)
{
    if (atomicCAS(status, 0ull, 1ull) == 0ull) status[1] = (unsigned long long)off;
}

// Register copy: every thread issues U independent streaming loads, then
// the matching stores.  Work item w = (tile, lc); a tile is ntok tokens x H
// heads x row_bytes, addressed on each side by a token stride and a head
// stride, so the head<->token transpose between the two pool layouts is a
// permutation of whole rows and needs no shuffling inside a row.
//
// GROUPED = false: the whole CTA works on one item at a time; everything that
// depends only on the item stays CTA-uniform (uniform registers, no redundant
// per-thread address arithmetic), which is worth 3% on 32 KiB tiles.
// GROUPED = true: the CTA is split into independent groups of `group_threads`
// threads (a multiple of the warp size), each walking its own items, so that
// batches of small tiles (few KV heads, short blocks) do not leave most of a
// CTA idle.  Nothing synchronises across groups.
template <int W, int U, bool CHECK, bool GROUPED>
__global__ void __launch_bounds__(max_threads(W, U))
copy_tiles_kernel(const CopyParams p)
{
    using V = typename VecT<W>::type;
    const uint32_t vpr = (uint32_t)p.row_bytes / W;  // vectors per row (a flat copy may use vectors wider than a row)
    const uint32_t H = (uint32_t)p.H;
    const int64_t hrow = (int64_t)p.H * p.row_bytes;
    // Rows of a tile are walked in the order of the side that is written, or (src_order) of the
    // side that is read.  When a row is not a whole number of 64-byte sector pairs (160-byte
    // rows of 80 bf16, say) a lone row read drags in the neighbouring row's half pair; walking
    // in the order of the reads makes those neighbours part of the same pass.
    const bool head_inner = p.src_order ? p.src.tok_stride >= p.src.head_stride : p.dst.tok_stride >= p.dst.head_stride;
    const bool flat = p.src.head_stride == p.row_bytes && p.src.tok_stride == hrow &&
                      p.dst.head_stride == p.row_bytes && p.dst.tok_stride == hrow;
    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    const uint32_t nthr = GROUPED ? (uint32_t)p.group_threads : blockDim.x;
    const uint32_t tig = GROUPED ? threadIdx.x % nthr : threadIdx.x;
    const uint32_t groups_per_cta = GROUPED ? blockDim.x / nthr : 1u;
    const int64_t group_id = GROUPED ? (int64_t)blockIdx.x * groups_per_cta + threadIdx.x / nthr : (int64_t)blockIdx.x;
    const int64_t n_groups = GROUPED ? (int64_t)gridDim.x * groups_per_cta : (int64_t)gridDim.x;
    const uint32_t m_vpr = vpr ? div_magic(vpr) : 0u;
    // vectors per token: a flat copy's W divides the bytes of a token, not necessarily a row
    const uint32_t tok_vecs = flat ? (uint32_t)(hrow / W) : H * vpr;
    const uint32_t m_H = div_magic(H);

    // Work items of this group: either every n_groups-th item (the groups sweep the
    // batch as one moving window) or one contiguous run per group.
    int64_t w, w_end, w_step;
    if (p.chunked) {
        const int64_t per = (n_work + n_groups - 1) / n_groups;
        w = group_id * per;
        w_end = w + per < n_work ? w + per : n_work;
        w_step = 1;
    } else {
        w = group_id;
        w_end = n_work;
        w_step = n_groups;
    }
    const bool narrow = n_work <= 0xFFFFFFFFll;   // 32-bit divisions are several times cheaper
    auto split = [&](int64_t x, int32_t &ti, int32_t &lci) {
        if (narrow) {
            const uint32_t x32 = (uint32_t)x;
            if (p.lc_fastest) {
                ti = (int32_t)(x32 / (uint32_t)p.n_lc);
                lci = (int32_t)(x32 - (uint32_t)ti * (uint32_t)p.n_lc);
            } else {
                lci = (int32_t)(x32 / (uint32_t)p.n_tiles);
                ti = (int32_t)(x32 - (uint32_t)lci * (uint32_t)p.n_tiles);
            }
        } else if (p.lc_fastest) {
            ti = (int32_t)(x / p.n_lc);
            lci = (int32_t)(x - (int64_t)ti * p.n_lc);
        } else {
            lci = (int32_t)(x / p.n_tiles);
            ti = (int32_t)(x - (int64_t)lci * p.n_tiles);
        }
        if (p.lc_skew > 1) {   // neighbouring tiles take different strips in the same sweep
            lci += (ti >> p.lc_skew_shift) & (p.lc_skew - 1);
            if (lci >= p.n_lc) lci -= p.n_lc;
        }
    };
    // The next item's tile record is fetched while the current one is being
    // copied, so its latency is off the critical path between two tiles.
    Tile t_next = {};
    int32_t lci_next = 0;
    if (w < w_end) {
        int32_t ti;
        split(w, ti, lci_next);
        t_next = p.tiles[p.tile_begin + ti];
    }
    for (; w < w_end; w += w_step) {
        const Tile t = t_next;
        const int32_t lci = lci_next;
        if (w + w_step < w_end) {
            int32_t ti;
            split(w + w_step, ti, lci_next);
            t_next = p.tiles[p.tile_begin + ti];
        }
        const int64_t lc = p.lc_begin + lci;
        const int64_t buf_lc = (int64_t)t.n_kept * hrow;
        const int64_t s_base = t.src_off + lc * (p.src.lc_stride >= 0 ? p.src.lc_stride : buf_lc);
        const int64_t d_base = t.dst_off + lc * (p.dst.lc_stride >= 0 ? p.dst.lc_stride : buf_lc);
        const bool zero = t.src_off < 0;
        const uint32_t ntok = (uint32_t)t.ntok;
        const uint32_t nvec = ntok * tok_vecs;
        const uint32_t m_inner = head_inner ? m_H : div_magic(ntok);
        const uint32_t inner = head_inner ? H : ntok;

        for (uint32_t i0 = tig; i0 < nvec; i0 += nthr * U) {
            V v[U];
            int64_t doff[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const uint32_t i = i0 + k * nthr;
                v[k] = zero_vec<V>();
                doff[k] = -1;
                if (i < nvec) {
                    int64_t so, dof;
                    if (flat) {
                        so = (int64_t)i * W;
                        dof = so;
                    } else {
                        const uint32_t row = fast_div(i, m_vpr);
                        const uint32_t vv = i - row * vpr;
                        const uint32_t outer = fast_div(row, m_inner);
                        const uint32_t in = row - outer * inner;
                        const uint32_t tk = head_inner ? outer : in;
                        const uint32_t hd = head_inner ? in : outer;
                        so = tk * p.src.tok_stride + hd * p.src.head_stride + (int64_t)vv * W;
                        dof = tk * p.dst.tok_stride + hd * p.dst.head_stride + (int64_t)vv * W;
                    }
                    so += s_base;
                    dof += d_base;
                    if (CHECK) {
                        if (!in_bounds(dof, W, p.dst.size) || (!zero && !in_bounds(so, W, p.src.size))) {
                            refuse(p.status, zero || in_bounds(so, W, p.src.size) ? dof : so);
                            continue;
                        }
                    }
                    doff[k] = dof;
                    if (!zero) v[k] = ld_stream<V>(p.src.base + so);
                }
            }
#pragma unroll
            for (int k = 0; k < U; ++k)
                if (doff[k] >= 0) st_stream<V>(p.dst.base + doff[k], v[k]);
        }
    }
}

}  // namespace pdkv
