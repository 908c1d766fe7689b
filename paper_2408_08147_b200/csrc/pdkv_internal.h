// Internal declarations shared by the host planner and the kernel launchers.
#pragma once

#include <atomic>
#include <cstdint>
#include <vector>

#include <cuda_runtime.h>

#include "pdkv.h"

namespace pdkv {

// One unit of work along the token axis: `ntok` consecutive kept tokens of one
// request that lie inside one block on every paged side of the copy.  Offsets
// are bytes from the side's base for layer 0 / K; the kernel adds the (l, c)
// step.  src_off < 0 marks a zero-fill tile (tail slots of a last decode block).
struct Tile {
    int64_t src_off;
    int64_t dst_off;
    int32_t ntok;
    int32_t n_kept;  // kept tokens of the request: the buffer's per-(l,c) stride is n_kept * H * ROW
};

// Addressing of one side of a copy (a pool in either layout, or the buffer).
struct Side {
    char *base;
    int64_t size;         // addressable bytes, for the bounds-checked build of the kernels
    int64_t lc_stride;    // bytes per (l,c) step; < 0: request dependent (contiguous buffer)
    int64_t tok_stride;   // bytes between consecutive tokens of one head
    int64_t head_stride;  // bytes between consecutive heads of one token
};

struct CopyParams {
    Side src, dst;
    const Tile *tiles;
    int32_t tile_begin, n_tiles;
    int32_t lc_begin, n_lc;
    int32_t H;
    int32_t row_bytes;   // D * E
    int32_t lc_fastest;
    int32_t chunked;     // 1: each group takes one contiguous run of work items
    int32_t lc_skew;       // power of two <= n_lc, or <= 1 for none: tile t works on strip (s + ((t >> shift) & (skew-1))) mod n_lc in sweep s
    int32_t lc_skew_shift;
    int32_t group_threads;  // threads that cooperate on one work item (set by the launcher)
    int32_t src_order;      // 1: the rows of a tile are walked in the order of the side that is read, 0: of the side written
    unsigned long long *status;  // [0] != 0: an access was refused; [1] offending offset
};

struct LaunchConfig {
    int vec_bytes;   // 32, 16, 8, 4, 2 or 1
    int unroll;      // independent accesses per thread: 1, 2, 4 or 8
    int group_threads;  // threads per work item; the launcher rounds it to a divisor of `threads`
    int threads;
    int ctas_per_sm;
    int max_ctas;    // 0: no cap; else the grid is limited to this many CTAs (leaves SMs to other kernels)
    int sm_count;
    int variant;             // 0 register copy, 1 bulk copies, 2 bulk copies with tiled TMA loads, 3 staged transpose
    int elem_bytes;          // element size, for the tensor map's data type
    int stages;              // bulk variant: shared-memory stages per CTA
    int64_t max_tile_bytes;  // bulk variant: largest tile of the launch
    bool check_bounds;
};

// Enqueue one persistent copy kernel.  Returns the CUDA status of the launch.
cudaError_t launch_copy(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream);

// Bulk-copy (TMA) variant: same contract; bulk_supported() says whether a launch qualifies.
cudaError_t launch_bulk(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream);
bool bulk_supported(const LaunchConfig &cfg, int row_bytes);
// Staged transpose (bulk loads in read order, coalesced stores in write order): same contract.
cudaError_t launch_staged(const CopyParams &p, const LaunchConfig &cfg, cudaStream_t stream);
bool staged_supported(const CopyParams &p, const LaunchConfig &cfg);

// Makes `dev` current for the lifetime of the object and restores the caller's device.
struct DeviceGuard {
    int prev = -1;
    bool changed = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev)
    {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) {
            err = cudaSetDevice(dev);
            changed = (err == cudaSuccess);
        }
    }
    ~DeviceGuard()
    {
        if (changed) cudaSetDevice(prev);
    }
    DeviceGuard(const DeviceGuard &) = delete;
    DeviceGuard &operator=(const DeviceGuard &) = delete;
};

// Process-wide settings; atomics because pdkv_tune may race with launches on other threads.
struct Tunables {
    std::atomic<int64_t> tile_bytes{32768};
    std::atomic<int64_t> ctas_per_sm{0};   // 0: chosen per class of copy (2, or 3 for half-size tiles)
    std::atomic<int64_t> max_ctas{0};
    std::atomic<int64_t> threads{0};   // 0: chosen with unroll, per class of copy
    std::atomic<int64_t> unroll{0};    // 0: chosen per class of copy
    std::atomic<int64_t> vec32{1};
    std::atomic<int64_t> lc_fastest{0};
    std::atomic<int64_t> group_threads{0};   // 0: sized from the plan's mean tile
    std::atomic<int64_t> chunked{0};
    std::atomic<int64_t> lc_skew{-1};   // -1: chosen per call from the prefill pool's block stride
    std::atomic<int64_t> lc_skew_shift{0};
    std::atomic<int64_t> debug_bounds{0};
    std::atomic<int64_t> debug_shrink{0};   // with debug_bounds: treat the last N bytes of each side as out of range
    std::atomic<int64_t> variant{-1};   // -1: chosen per call (register copy or staged transpose)
    std::atomic<int64_t> stages{3};
    std::atomic<int64_t> dry_run{0};
    std::atomic<int64_t> autotune_reuse{1};
    std::atomic<int64_t> src_order{-1};   // -1: by the row size (see CopyParams::src_order)
};
Tunables &tunables();

// The tunables that steer a launch, copied into a plan when it is created: a plan keeps
// launching the way it was set up, whatever pdkv_tune() is told afterwards (by this or
// another thread).  pdkv_tune() only sets the defaults of plans created later.
struct LaunchOptions {
    int ctas_per_sm = 0, max_ctas = 0, threads = 0, unroll = 0, vec32 = 1, lc_fastest = 0, group_threads = 0,
        chunked = 0, lc_skew = -1, lc_skew_shift = 0, debug_bounds = 0, variant = -1, stages = 3, src_order = -1;
    int64_t debug_shrink = 0;
    int64_t tile_bytes = 32768;
};
LaunchOptions snapshot_options();

// Everything launch_copy()/launch_bulk() need besides the sides, the tile list and the layer range.
struct ResolvedLaunch {
    LaunchConfig cfg;
    int32_t lc_fastest, chunked, lc_skew, lc_skew_shift, src_order;
};

// Used by the no-allocation entry point and the retrieval queue (their own translation units).
// A host-only plan: validated batch and tile lists, no CUDA call, nothing on the device.
// `op_mask` (bit per pdkv_op) says which tile lists to build.
int create_host_plan(const pdkv_pool *src, const pdkv_pool *dst, const pdkv_batch_desc *batch, unsigned op_mask,
                     pdkv_plan **out);
// The launch shape, work order and strip skew the plan uses for `op` between these two sides over
// `n_lc` (layer, K/V) strips: the one chooser behind every entry point.
void resolve_launch(const pdkv_plan *plan, int op, const Side &src, const Side &dst, int n_lc, int sm_count,
                    ResolvedLaunch *out);
void describe_transfer(const pdkv_plan *plan, Side *src, Side *dst, int *H, int *row_bytes,
                       int *vec_bytes, int *num_layers, int *device);
int report_cuda_error(cudaError_t e, const char *what);
// SMs of the partition a stream belongs to (a stream handed out by pdkv_sm_partition_stream), else 0:
// launches on such a stream size their persistent grid to the partition's share.
int partition_sms_of(cudaStream_t stream);
int plan_num_layers(const pdkv_plan *plan);

}  // namespace pdkv
