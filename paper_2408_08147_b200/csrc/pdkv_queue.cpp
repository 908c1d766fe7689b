// Asynchronous retrieval (Sec. 3.5): the decode side keeps a small, fixed set
// of receive slots.  A transfer is admitted only if a slot is free (otherwise
// the caller is told at once, nothing waits inside the library), runs on the
// slot's own stream concurrently with whatever the decode engine is doing, and
// its completion is polled; the slot is handed back when the engine has taken
// the request into its running batch.
#include <mutex>
#include <new>
#include <vector>

#include "pdkv_internal.h"

namespace {

struct Slot {
    cudaStream_t stream = nullptr;
    cudaEvent_t done = nullptr;
    pdkv_plan *plan = nullptr;
    void *workspace = nullptr;   // device memory for the slot's plan, reused across tickets
    int64_t ticket = -1;   // -1: free
};

}  // namespace

struct pdkv_queue {
    const pdkv_pool *src = nullptr, *dst = nullptr;
    int device = 0;
    bool host_only = false;   // built under "dry_run": admission logic only, no CUDA objects
    std::vector<Slot> slots;
    int64_t next_ticket = 0;
    int64_t submitted = 0, rejected = 0;
    std::mutex mu;
};

namespace {

constexpr size_t kSlotWorkspaceBytes = 1 << 20;   // tile lists of ~14k tiles; larger batches fall back to cudaMalloc

Slot *find(pdkv_queue *q, int64_t ticket)
{
    if (ticket < 0) return nullptr;
    for (Slot &s : q->slots)
        if (s.ticket == ticket) return &s;
    return nullptr;
}

using DevGuard = pdkv::DeviceGuard;

}  // namespace

extern "C" {

int pdkv_queue_create(const pdkv_pool *src, const pdkv_pool *dst, int device, int capacity, pdkv_queue **out)
{
    if (out) *out = nullptr;
    if (!out || !src || !dst || capacity < 1 || capacity > 64 || device < 0) return PDKV_ERR_INVALID_ARG;
    pdkv_queue *q = new (std::nothrow) pdkv_queue;
    if (!q) return PDKV_ERR_NOMEM;
    q->src = src;
    q->dst = dst;
    q->device = device;
    q->host_only = pdkv::tunables().dry_run != 0;
    q->slots.resize((size_t)capacity);
    if (!q->host_only) {
        DevGuard guard(device);
        cudaError_t e = guard.err;
        for (Slot &s : q->slots) {
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaMalloc(&s.workspace, kSlotWorkspaceBytes);
        }
        if (e != cudaSuccess) {
            const int rc = pdkv::report_cuda_error(e, "queue set-up");
            pdkv_queue_destroy(q);
            return rc;
        }
    }
    *out = q;
    return PDKV_OK;
}

int pdkv_queue_submit(pdkv_queue *q, const pdkv_batch_desc *batch, const void *host_src_pool,
                      void *host_dst_pool, void *wait_event, int64_t *ticket)
{
    if (ticket) *ticket = -1;
    if (!q || !batch || !ticket) return PDKV_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(q->mu);
    Slot *slot = nullptr;
    for (Slot &s : q->slots)
        if (s.ticket < 0) {
            slot = &s;
            break;
        }
    if (!slot) {
        ++q->rejected;
        return PDKV_ERR_BUSY;
    }
    int rc;
    if (q->host_only) {
        rc = pdkv::create_host_plan(q->src, q->dst, batch, 7u, &slot->plan);
        if (rc != PDKV_OK) return rc;
    } else {
        DevGuard guard(q->device);
        if (guard.err != cudaSuccess) return pdkv::report_cuda_error(guard.err, "cudaSetDevice");
        rc = pdkv_plan_create_in(q->src, q->dst, 0, batch, slot->workspace, kSlotWorkspaceBytes, nullptr,
                                 slot->stream, &slot->plan);
        if (rc == PDKV_ERR_BUFFER_TOO_SMALL)   // a batch with more tiles than the slot's workspace holds
            rc = pdkv_plan_create(q->src, q->dst, 0, batch, slot->stream, &slot->plan);
        if (rc != PDKV_OK) return rc;
        if (wait_event) {   // the slot's stream runs beside the caller's: order it after the producer of the blocks
            cudaError_t e = cudaStreamWaitEvent(slot->stream, static_cast<cudaEvent_t>(wait_event), 0);
            if (e != cudaSuccess) rc = pdkv::report_cuda_error(e, "cudaStreamWaitEvent");
        }
        if (rc == PDKV_OK && host_src_pool) rc = pdkv_upload_blocks(slot->plan, host_src_pool, slot->stream);
        if (rc == PDKV_OK) rc = pdkv_transfer(slot->plan, 0, pdkv::plan_num_layers(slot->plan), slot->stream);
        if (rc == PDKV_OK && host_dst_pool) rc = pdkv_download_blocks(slot->plan, host_dst_pool, slot->stream);
        if (rc == PDKV_OK) {
            cudaError_t e = cudaEventRecord(slot->done, slot->stream);
            if (e != cudaSuccess) rc = pdkv::report_cuda_error(e, "cudaEventRecord");
        }
        if (rc != PDKV_OK) {           // let what was enqueued finish before the plan's arrays go away
            cudaStreamSynchronize(slot->stream);
            pdkv_plan_destroy(slot->plan);
            slot->plan = nullptr;
            return rc;
        }
    }
    slot->ticket = q->next_ticket++;
    ++q->submitted;
    *ticket = slot->ticket;
    return PDKV_OK;
}

int pdkv_queue_poll(pdkv_queue *q, int64_t ticket, int *done)
{
    if (!q || !done) return PDKV_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(q->mu);
    Slot *s = find(q, ticket);
    if (!s) return PDKV_ERR_INVALID_ARG;
    if (q->host_only) {
        *done = 1;
        return PDKV_OK;
    }
    const cudaError_t e = cudaEventQuery(s->done);
    if (e == cudaSuccess) *done = 1;
    else if (e == cudaErrorNotReady) *done = 0;
    else return pdkv::report_cuda_error(e, "cudaEventQuery");
    return PDKV_OK;
}

int pdkv_queue_wait(pdkv_queue *q, int64_t ticket)
{
    if (!q) return PDKV_ERR_INVALID_ARG;
    cudaEvent_t ev;
    {
        std::lock_guard<std::mutex> lock(q->mu);
        Slot *s = find(q, ticket);
        if (!s) return PDKV_ERR_INVALID_ARG;
        if (q->host_only) return PDKV_OK;
        ev = s->done;
    }
    const cudaError_t e = cudaEventSynchronize(ev);
    return e == cudaSuccess ? PDKV_OK : pdkv::report_cuda_error(e, "cudaEventSynchronize");
}

int pdkv_queue_release(pdkv_queue *q, int64_t ticket)
{
    if (!q) return PDKV_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(q->mu);
    Slot *s = find(q, ticket);
    if (!s) return PDKV_ERR_INVALID_ARG;
    int rc = PDKV_OK;
    if (!q->host_only) {               // a slot may only be reused once its transfer has finished
        const cudaError_t e = cudaEventSynchronize(s->done);
        if (e != cudaSuccess) rc = pdkv::report_cuda_error(e, "cudaEventSynchronize");
    }
    const int rc2 = pdkv_plan_destroy(s->plan);
    s->plan = nullptr;
    s->ticket = -1;
    return rc != PDKV_OK ? rc : rc2;
}

int pdkv_queue_stats(const pdkv_queue *q, int *capacity, int *in_use, int64_t *submitted, int64_t *rejected)
{
    if (!q) return PDKV_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(const_cast<pdkv_queue *>(q)->mu);
    int used = 0;
    for (const Slot &s : q->slots) used += s.ticket >= 0;
    if (capacity) *capacity = (int)q->slots.size();
    if (in_use) *in_use = used;
    if (submitted) *submitted = q->submitted;
    if (rejected) *rejected = q->rejected;
    return PDKV_OK;
}

int pdkv_queue_destroy(pdkv_queue *q)
{
    if (!q) return PDKV_OK;
    int rc = PDKV_OK;
    {
        DevGuard guard(q->device);
        for (Slot &s : q->slots) {
            if (s.stream) cudaStreamSynchronize(s.stream);
            if (s.plan) pdkv_plan_destroy(s.plan);
            if (s.done) cudaEventDestroy(s.done);
            if (s.workspace) cudaFree(s.workspace);
            if (s.stream && cudaStreamDestroy(s.stream) != cudaSuccess) rc = PDKV_ERR_CUDA;
        }
    }
    delete q;
    return rc;
}

}  // extern "C"
