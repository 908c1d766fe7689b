// Process-local split of a GPU's SMs into a small set for the transfer kernels and the rest for
// compute, through CUDA green contexts.  Sec. 3.5 wants RecvScatter, in its operator form, to run
// beside the stream's other operators without holding them up.  On one GPU a copy kernel that
// shares SMs with a compute kernel only gets a CTA slot when a compute CTA retires; with a
// partition of its own it runs from the first cycle and the compute kernel keeps every SM it was
// given.  Nothing here outlasts the process and no device setting is touched: a green context is
// an object of this process's primary context and dies with it.
//
// The driver entry points are looked up at run time (the library links only the runtime).
#include <atomic>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include <cuda.h>

#include "pdkv_internal.h"

namespace {

struct Driver {
    CUresult (*DeviceGet)(CUdevice *, int) = nullptr;
    CUresult (*DeviceGetDevResource)(CUdevice, CUdevResource *, CUdevResourceType) = nullptr;
    CUresult (*DevSmResourceSplitByCount)(CUdevResource *, unsigned int *, const CUdevResource *, CUdevResource *,
                                          unsigned int, unsigned int) = nullptr;
    CUresult (*DevResourceGenerateDesc)(CUdevResourceDesc *, CUdevResource *, unsigned int) = nullptr;
    CUresult (*GreenCtxCreate)(CUgreenCtx *, CUdevResourceDesc, CUdevice, unsigned int) = nullptr;
    CUresult (*GreenCtxDestroy)(CUgreenCtx) = nullptr;
    CUresult (*GreenCtxStreamCreate)(CUstream *, CUgreenCtx, unsigned int, int) = nullptr;
    CUresult (*StreamDestroy)(CUstream) = nullptr;
    bool ok = false;
};

template <typename F> bool lookup(const char *name, F *fn)
{
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint(name, &sym, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !sym)
        return false;
    *fn = reinterpret_cast<F>(sym);
    return true;
}

const Driver &driver()
{
    static Driver d = [] {
        Driver x;
        x.ok = lookup("cuDeviceGet", &x.DeviceGet) && lookup("cuDeviceGetDevResource", &x.DeviceGetDevResource) &&
               lookup("cuDevSmResourceSplitByCount", &x.DevSmResourceSplitByCount) &&
               lookup("cuDevResourceGenerateDesc", &x.DevResourceGenerateDesc) &&
               lookup("cuGreenCtxCreate", &x.GreenCtxCreate) && lookup("cuGreenCtxDestroy", &x.GreenCtxDestroy) &&
               lookup("cuGreenCtxStreamCreate", &x.GreenCtxStreamCreate) && lookup("cuStreamDestroy", &x.StreamDestroy);
        return x;
    }();
    return d;
}

// Streams of live partitions with their SM counts, so that a launch can size its grid to the
// share of the stream it is given.  Read on every launch: the count keeps the common case
// (no partition exists) to one relaxed load.
std::mutex g_streams_mutex;
std::vector<std::pair<cudaStream_t, int>> g_streams;
std::atomic<int> g_stream_count{0};

void register_stream(cudaStream_t st, int sms)
{
    std::lock_guard<std::mutex> lock(g_streams_mutex);
    g_streams.emplace_back(st, sms);
    g_stream_count.store((int)g_streams.size(), std::memory_order_release);
}

void unregister_stream(cudaStream_t st)
{
    std::lock_guard<std::mutex> lock(g_streams_mutex);
    for (size_t i = 0; i < g_streams.size(); ++i)
        if (g_streams[i].first == st) {
            g_streams.erase(g_streams.begin() + (long)i);
            break;
        }
    g_stream_count.store((int)g_streams.size(), std::memory_order_release);
}

}  // namespace

namespace pdkv {
int partition_sms_of(cudaStream_t stream)
{
    if (g_stream_count.load(std::memory_order_acquire) == 0) return 0;
    std::lock_guard<std::mutex> lock(g_streams_mutex);
    for (const auto &e : g_streams)
        if (e.first == stream) return e.second;
    return 0;
}
}  // namespace pdkv

struct pdkv_sm_partition {
    int device = 0;
    CUgreenCtx ctx[2] = {nullptr, nullptr};     // 0: transfer SMs, 1: the rest
    CUstream stream[2] = {nullptr, nullptr};
    int sms[2] = {0, 0};
};

extern "C" {

int pdkv_sm_partition_create(int device, int transfer_sms, pdkv_sm_partition **out)
{
    if (out) *out = nullptr;
    if (!out || device < 0 || transfer_sms < 1) return PDKV_ERR_INVALID_ARG;
    pdkv::DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return pdkv::report_cuda_error(guard.err, "cudaSetDevice");
    cudaError_t e = cudaFree(nullptr);            // makes sure the primary context exists
    if (e != cudaSuccess) return pdkv::report_cuda_error(e, "context set-up");
    const Driver &d = driver();
    if (!d.ok) return pdkv::report_cuda_error(cudaErrorNotSupported, "green-context entry points (driver too old)");
    pdkv_sm_partition *p = new (std::nothrow) pdkv_sm_partition;
    if (!p) return PDKV_ERR_NOMEM;
    p->device = device;
    auto fail = [&](const char *what) {
        pdkv_sm_partition_destroy(p);
        return pdkv::report_cuda_error(cudaErrorNotSupported, what);
    };
    CUdevice dev;
    if (d.DeviceGet(&dev, device) != CUDA_SUCCESS) return fail("cuDeviceGet");
    CUdevResource all, part[1], rest;
    if (d.DeviceGetDevResource(dev, &all, CU_DEV_RESOURCE_TYPE_SM) != CUDA_SUCCESS) return fail("cuDeviceGetDevResource");
    if ((unsigned)transfer_sms >= all.sm.smCount) return fail("SM partition: the transfer share must leave SMs to compute");
    unsigned int groups = 1;
    if (d.DevSmResourceSplitByCount(part, &groups, &all, &rest, 0, (unsigned)transfer_sms) != CUDA_SUCCESS || groups != 1 ||
        rest.sm.smCount == 0)
        return fail("cuDevSmResourceSplitByCount");
    CUdevResource *res[2] = {&part[0], &rest};
    for (int i = 0; i < 2; ++i) {
        CUdevResourceDesc desc;
        if (d.DevResourceGenerateDesc(&desc, res[i], 1) != CUDA_SUCCESS) return fail("cuDevResourceGenerateDesc");
        if (d.GreenCtxCreate(&p->ctx[i], desc, dev, CU_GREEN_CTX_DEFAULT_STREAM) != CUDA_SUCCESS) return fail("cuGreenCtxCreate");
        if (d.GreenCtxStreamCreate(&p->stream[i], p->ctx[i], CU_STREAM_NON_BLOCKING, 0) != CUDA_SUCCESS)
            return fail("cuGreenCtxStreamCreate");
        p->sms[i] = (int)res[i]->sm.smCount;
        register_stream(p->stream[i], p->sms[i]);
    }
    *out = p;
    return PDKV_OK;
}

int pdkv_sm_partition_info(const pdkv_sm_partition *p, int *transfer_sms, int *compute_sms)
{
    if (!p) return PDKV_ERR_INVALID_ARG;
    if (transfer_sms) *transfer_sms = p->sms[0];
    if (compute_sms) *compute_sms = p->sms[1];
    return PDKV_OK;
}

int pdkv_sm_partition_stream(const pdkv_sm_partition *p, int which, void **stream)
{
    if (!p || !stream || which < 0 || which > 1) return PDKV_ERR_INVALID_ARG;
    *stream = p->stream[which];
    return PDKV_OK;
}

int pdkv_sm_partition_destroy(pdkv_sm_partition *p)
{
    if (!p) return PDKV_OK;
    const Driver &d = driver();
    pdkv::DeviceGuard guard(p->device);
    for (int i = 0; i < 2; ++i) {
        if (p->stream[i]) {
            unregister_stream(p->stream[i]);
            cudaStreamSynchronize(p->stream[i]);
            d.StreamDestroy(p->stream[i]);
        }
        if (p->ctx[i]) d.GreenCtxDestroy(p->ctx[i]);
    }
    delete p;
    return PDKV_OK;
}

}  // extern "C"
