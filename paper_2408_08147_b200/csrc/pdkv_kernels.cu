// sm_100a kernels for the paged-KVCache transfer: one persistent grid walks a
// list of (tile, layer, K/V) work items and moves whole head rows (D*E bytes)
// between a block-fixed pool and the contiguous buffer, or pool to pool.
//
// The path is pure data movement (Sec. 3.5: organise blocks into a contiguous
// buffer, restore blocks from bytes), so the only resource that matters is HBM
// bandwidth: accesses are 16 bytes per lane, every warp touches whole rows, and
// each thread keeps several independent loads in flight before storing.
#include "pdkv_internal.h"

namespace pdkv {

template <int W> struct VecT;
template <> struct VecT<16> { using type = uint4; };
template <> struct VecT<8> { using type = uint2; };
template <> struct VecT<4> { using type = unsigned int; };
template <> struct VecT<2> { using type = unsigned short; };
template <> struct VecT<1> { using type = unsigned char; };

template <typename V> __device__ __forceinline__ V zero_vec();
template <> __device__ __forceinline__ uint4 zero_vec<uint4>() { return make_uint4(0, 0, 0, 0); }
template <> __device__ __forceinline__ uint2 zero_vec<uint2>() { return make_uint2(0, 0); }
template <> __device__ __forceinline__ unsigned int zero_vec<unsigned int>() { return 0u; }
template <> __device__ __forceinline__ unsigned short zero_vec<unsigned short>() { return 0; }
template <> __device__ __forceinline__ unsigned char zero_vec<unsigned char>() { return 0; }

constexpr int kMaxThreads = 512;
constexpr int kUnroll = 8;

__device__ __forceinline__ bool in_bounds(int64_t off, int width, int64_t size)
{
    return off >= 0 && off + width <= size;
}

__device__ __forceinline__ void refuse(unsigned long long *status, int64_t off)
{
    if (atomicCAS(status, 0ull, 1ull) == 0ull) status[1] = (unsigned long long)off;
}

// Register copy: every thread issues kUnroll independent streaming loads, then
// the matching stores.  Work item w = (tile, lc); a tile is ntok tokens x H
// heads x row_bytes, addressed on each side by a token stride and a head
// stride, so the head<->token transpose between the two pool layouts is a
// permutation of whole rows and needs no shuffling inside a row.
template <int W, bool CHECK>
__global__ void __launch_bounds__(kMaxThreads)
copy_tiles_kernel(const CopyParams p)
{
    using V = typename VecT<W>::type;
    const uint32_t vpr = (uint32_t)p.row_bytes / W;  // vectors per row
    const uint32_t H = (uint32_t)p.H;
    const int64_t hrow = (int64_t)p.H * p.row_bytes;
    const bool head_inner = p.dst.tok_stride >= p.dst.head_stride;
    const bool flat = p.src.head_stride == p.row_bytes && p.src.tok_stride == hrow &&
                      p.dst.head_stride == p.row_bytes && p.dst.tok_stride == hrow;
    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    const uint32_t nthr = blockDim.x;

    for (int64_t w = blockIdx.x; w < n_work; w += gridDim.x) {
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
        const int64_t s_base = t.src_off + lc * (p.src.lc_stride >= 0 ? p.src.lc_stride : buf_lc);
        const int64_t d_base = t.dst_off + lc * (p.dst.lc_stride >= 0 ? p.dst.lc_stride : buf_lc);
        const bool zero = t.src_off < 0;
        const uint32_t ntok = (uint32_t)t.ntok;
        const uint32_t nvec = ntok * H * vpr;

        for (uint32_t i0 = threadIdx.x; i0 < nvec; i0 += nthr * kUnroll) {
            V v[kUnroll];
            int64_t doff[kUnroll];
#pragma unroll
            for (int k = 0; k < kUnroll; ++k) {
                const uint32_t i = i0 + k * nthr;
                v[k] = zero_vec<V>();
                doff[k] = -1;
                if (i < nvec) {
                    int64_t so, dof;
                    if (flat) {
                        so = (int64_t)i * W;
                        dof = so;
                    } else {
                        const uint32_t row = i / vpr;
                        const uint32_t vv = i - row * vpr;
                        uint32_t tk, hd;
                        if (head_inner) {
                            tk = row / H;
                            hd = row - tk * H;
                        } else {
                            hd = row / ntok;
                            tk = row - hd * ntok;
                        }
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
                    if (!zero) v[k] = __ldcs(reinterpret_cast<const V *>(p.src.base + so));
                }
            }
#pragma unroll
            for (int k = 0; k < kUnroll; ++k)
                if (doff[k] >= 0) __stcs(reinterpret_cast<V *>(p.dst.base + doff[k]), v[k]);
        }
    }
}

template <int W>
static cudaError_t launch_w(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream)
{
    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    if (n_work <= 0) return cudaSuccess;
    int threads = cfg.threads;
    if (threads > kMaxThreads) threads = kMaxThreads;
    if (threads < 32) threads = 32;
    threads = (threads / 32) * 32;
    auto kern = cfg.check_bounds ? copy_tiles_kernel<W, true> : copy_tiles_kernel<W, false>;
    int occ = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, threads, 0);
    if (e != cudaSuccess) return e;
    if (occ < 1) occ = 1;
    if (occ > cfg.ctas_per_sm) occ = cfg.ctas_per_sm;
    int64_t grid = (int64_t)cfg.sm_count * occ;
    if (grid > n_work) grid = n_work;
    kern<<<(unsigned)grid, threads, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_copy(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream)
{
    switch (cfg.vec_bytes) {
    case 16: return launch_w<16>(p, cfg, stream);
    case 8: return launch_w<8>(p, cfg, stream);
    case 4: return launch_w<4>(p, cfg, stream);
    case 2: return launch_w<2>(p, cfg, stream);
    case 1: return launch_w<1>(p, cfg, stream);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace pdkv
