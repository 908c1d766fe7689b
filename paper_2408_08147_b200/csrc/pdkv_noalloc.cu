// Fused transfer without any device allocation: the tile list that the copy
// kernel walks is staged in a fixed device array that ships with the library.
//
// Intended for callers that may not call cudaMalloc: engines that gave all of
// HBM to their own block allocator, processes under a frozen memory pool, or
// latency paths that cannot afford cudaMalloc's device-wide synchronisation.
#include <mutex>

#include "pdkv_internal.h"

namespace {

constexpr size_t kHeaderBytes = 256;  // status words of the kernels, cleared by every call
static_assert(sizeof(pdkv::Tile) == 24, "PDKV_NOALLOC_SCRATCH_BYTES assumes 24-byte tiles");
static_assert(PDKV_NOALLOC_SCRATCH_BYTES == kHeaderBytes + PDKV_NOALLOC_MAX_TILES * sizeof(pdkv::Tile),
              "scratch size and tile limit must agree");

// Scratch shared by every call on a device: [status words][tile list].  Each
// GPU that loads this library keeps its own copy until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[PDKV_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
struct DeviceSlot {
    unsigned char *scratch = nullptr;  // device address of g_noalloc_scratch on that device
    int sm_count = 0;
};
DeviceSlot g_slots[kMaxDevices];
std::mutex g_slots_mutex;

// Once per device, with that device current: the array's name is only a
// host-side handle, so the kernel must be given the address looked up here.
cudaError_t device_slot(int device, DeviceSlot *out)
{
    std::lock_guard<std::mutex> lock(g_slots_mutex);
    DeviceSlot &s = g_slots[device];
    if (!s.scratch) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return e;
        s.sm_count = sms;
        s.scratch = static_cast<unsigned char *>(ptr);
    }
    *out = s;
    return cudaSuccess;
}

struct PlanHolder {
    pdkv_plan *p = nullptr;
    ~PlanHolder() { if (p) pdkv_plan_destroy(p); }
};

}  // namespace

extern "C" int pdkv_transfer_noalloc(const pdkv_pool *src, const pdkv_pool *dst,
                                     const pdkv_batch_desc *batch, int layer_begin, int layer_end,
                                     void *stream)
{
    if (!src || !dst || !batch) return PDKV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {   // The tile list below is staged from host memory that this call frees on return, so the
        // call cannot be recorded: a capturing stream is refused before anything is enqueued.
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        cudaError_t ce = cudaStreamIsCapturing(st, &capturing);
        if (ce != cudaSuccess) return pdkv::report_cuda_error(ce, "cudaStreamIsCapturing");
        if (capturing != cudaStreamCaptureStatusNone) return PDKV_ERR_INVALID_ARG;
    }
    PlanHolder plan;  // host memory only: validated batch and the tile list of the fused transfer
    int rc = pdkv::create_host_plan(src, dst, batch, 1u << PDKV_OP_TRANSFER, &plan.p);
    if (rc != PDKV_OK) return rc;

    pdkv::CopyParams p;
    int vec_bytes = 16, num_layers = 0, device = 0, H = 0, row_bytes = 0;
    pdkv::describe_transfer(plan.p, &p.src, &p.dst, &H, &row_bytes, &vec_bytes, &num_layers, &device);
    if (layer_begin < 0 || layer_begin > layer_end || layer_end > num_layers) return PDKV_ERR_INVALID_ARG;
    if (device < 0 || device >= kMaxDevices) return PDKV_ERR_INVALID_ARG;

    const pdkv_tile *tiles = nullptr;
    int64_t n_tiles = 0;
    rc = pdkv_plan_tiles(plan.p, PDKV_OP_TRANSFER, &tiles, &n_tiles);
    if (rc != PDKV_OK) return rc;
    if (n_tiles > PDKV_NOALLOC_MAX_TILES) return PDKV_ERR_LIMIT;
    if (n_tiles == 0 || layer_begin == layer_end) return PDKV_OK;

    int prev = -1;
    cudaError_t e = cudaGetDevice(&prev);
    if (e != cudaSuccess) return pdkv::report_cuda_error(e, "cudaGetDevice");
    if (prev != device && (e = cudaSetDevice(device)) != cudaSuccess)
        return pdkv::report_cuda_error(e, "cudaSetDevice");

    rc = PDKV_OK;
    DeviceSlot slot;
    if ((e = device_slot(device, &slot)) != cudaSuccess) {
        rc = pdkv::report_cuda_error(e, "cudaGetSymbolAddress");
    } else if ((e = cudaMemsetAsync(slot.scratch, 0, kHeaderBytes, st)) != cudaSuccess) {
        rc = pdkv::report_cuda_error(e, "cudaMemsetAsync");
    } else if ((e = cudaMemcpyAsync(slot.scratch + kHeaderBytes, tiles, (size_t)n_tiles * sizeof(pdkv::Tile),
                                    cudaMemcpyHostToDevice, st)) != cudaSuccess) {
        rc = pdkv::report_cuda_error(e, "cudaMemcpyAsync");
    } else {
        p.tiles = reinterpret_cast<const pdkv::Tile *>(slot.scratch + kHeaderBytes);
        p.tile_begin = 0;
        p.n_tiles = (int32_t)n_tiles;
        p.lc_begin = 2 * layer_begin;
        p.n_lc = 2 * (layer_end - layer_begin);
        p.H = H;
        p.row_bytes = row_bytes;
        // launch shape, work order and strip skew from the chooser every plan-based call uses
        pdkv::ResolvedLaunch r;
        const int share = pdkv::partition_sms_of(st);
        pdkv::resolve_launch(plan.p, PDKV_OP_TRANSFER, p.src, p.dst, p.n_lc, share > 0 ? share : slot.sm_count, &r);
        p.lc_fastest = r.lc_fastest;
        p.chunked = r.chunked;
        p.lc_skew = r.lc_skew;
        p.lc_skew_shift = r.lc_skew_shift;
        p.src_order = r.src_order;
        p.group_threads = 0;
        p.status = reinterpret_cast<unsigned long long *>(slot.scratch);
        r.cfg.variant = 0;            // the register-copy kernel: it needs nothing but the tile list
        r.cfg.check_bounds = false;   // there is no plan to report a refusal through
        if ((e = pdkv::launch_copy(p, r.cfg, st)) != cudaSuccess) rc = pdkv::report_cuda_error(e, "kernel launch");
    }
    if (prev != device) cudaSetDevice(prev);
    return rc;
}
