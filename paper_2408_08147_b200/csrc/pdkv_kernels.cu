// Launchers of the register-copy kernels (pdkv_copy_kernel.cuh): pick the instantiation for the
// access width, unroll, bounds checking and grouping, size the persistent grid, enqueue.
#include "pdkv_copy_kernel.cuh"

namespace pdkv {

template <int W, int U>
static cudaError_t launch_wu(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream)
{
    const int64_t n_work = (int64_t)p.n_tiles * p.n_lc;
    if (n_work <= 0) return cudaSuccess;
    int threads = cfg.threads;
    if (threads > max_threads(W, U)) threads = max_threads(W, U);
    if (threads < 32) threads = 32;
    threads = (threads / 32) * 32;
    int group = cfg.group_threads;
    if (group < 32) group = 32;
    group = (group / 32) * 32;
    while (group < threads && threads % group) group += 32;
    if (group > threads) group = threads;
    const bool grouped = group < threads;
    auto kern = cfg.check_bounds ? (grouped ? copy_tiles_kernel<W, U, true, true> : copy_tiles_kernel<W, U, true, false>)
                                 : (grouped ? copy_tiles_kernel<W, U, false, true> : copy_tiles_kernel<W, U, false, false>);
    // CTAs of this instantiation that fit one SM: asked once per shape and kept (the library
    // is built for one architecture, so every device of the process gives the same answer)
    static std::atomic<int> occ_of[2][2][33];
    std::atomic<int> &slot = occ_of[cfg.check_bounds ? 1 : 0][grouped ? 1 : 0][threads / 32];
    int occ = slot.load(std::memory_order_relaxed);
    if (occ == 0) {
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, threads, 0);
        if (e != cudaSuccess) return e;
        if (occ < 1) occ = 1;
        slot.store(occ, std::memory_order_relaxed);
    }
    if (occ > cfg.ctas_per_sm) occ = cfg.ctas_per_sm;
    CopyParams q = p;
    q.group_threads = group;
    const int64_t per_cta = threads / group;
    int64_t grid = (int64_t)cfg.sm_count * occ;
    if (cfg.max_ctas > 0 && grid > cfg.max_ctas) grid = cfg.max_ctas;
    if (grid * per_cta > n_work) grid = (n_work + per_cta - 1) / per_cta;
    kern<<<(unsigned)grid, threads, 0, stream>>>(q);
    return cudaGetLastError();
}

template <int W>
static cudaError_t launch_w(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream)
{
    switch (cfg.unroll) {
    case 1: return launch_wu<W, 1>(p, cfg, stream);
    case 2: return launch_wu<W, 2>(p, cfg, stream);
    case 4: return launch_wu<W, 4>(p, cfg, stream);
    case 8: return launch_wu<W, 8>(p, cfg, stream);
    default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_copy(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream)
{
    switch (cfg.vec_bytes) {
    case 32: return launch_w<32>(p, cfg, stream);
    case 16: return launch_w<16>(p, cfg, stream);
    case 8: return launch_wu<8, 4>(p, cfg, stream);
    case 4: return launch_wu<4, 4>(p, cfg, stream);
    case 2: return launch_wu<2, 4>(p, cfg, stream);
    case 1: return launch_wu<1, 4>(p, cfg, stream);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace pdkv
