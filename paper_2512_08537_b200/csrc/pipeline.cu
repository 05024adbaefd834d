// Host-buffer front end: copies a batch to the device, runs gate -> head, copies results back.
//
// Two ways in. ardiff_pipeline_run_host does all of it on the caller's stream and waits.
// ardiff_pipeline_submit / _wait run batches through `slots` sets of staging buffers on three
// streams the pipeline owns (copy-in, compute, copy-out), so the host->device copy of batch i+1
// and the device->host copy of batch i-1 overlap the kernels of batch i. Compute is one stream
// because all batches share the head's scratch; the events below order everything else:
//
//   in_done[s]    copy-in of slot s finished          -> compute may read the staging buffers
//   comp_done[s]  gate + head of slot s finished      -> copy-out may read, next copy-in may overwrite
//   out_done[s]   copy-out of slot s finished         -> the host may read; next compute may overwrite
#include <cuda_runtime.h>
#include <stdint.h>

#include <new>

#include "../../include/ardiff.h"
#include "common.cuh"

namespace {

struct Slot {
    void* feat = nullptr;
    void* cond = nullptr;
    float* noise = nullptr;
    float* out = nullptr;
    uint8_t* mask = nullptr;
    int32_t* idx = nullptr;
    int32_t* count = nullptr;
    int32_t* count_pinned = nullptr;   // host: a pageable destination would make the copy-out block the submitting thread
    int32_t* count_user = nullptr;     // where ardiff_pipeline_wait delivers it
    cudaEvent_t in_done = nullptr, comp_done = nullptr, out_done = nullptr;
    bool used = false;      // has a submission whose events are recorded
    int rc = ARDIFF_OK;     // what the submission's launches returned
};

}  // namespace

struct ardiff_pipeline {
    ardiff_head* head;
    int device;
    int64_t max_n;
    int32_t d, Dc, C;
    int n_slots;
    Slot slot[ARDIFF_PIPELINE_MAX_SLOTS];
    cudaStream_t s_in = nullptr, s_comp = nullptr, s_out = nullptr;
    cudaEvent_t ev_caller = nullptr;
};

// zero-byte copies are skipped: an empty batch may come with NULL host pointers
static bool copy_async(void* dst, const void* src, size_t bytes, cudaMemcpyKind kind, cudaStream_t st) {
    return bytes == 0 || cudaMemcpyAsync(dst, src, bytes, kind, st) == cudaSuccess;
}

static void free_all(ardiff_pipeline* p) {
    for (int s = 0; s < p->n_slots; ++s) {
        Slot& q = p->slot[s];
        cudaFree(q.feat); cudaFree(q.cond); cudaFree(q.noise); cudaFree(q.out);
        cudaFree(q.mask); cudaFree(q.idx); cudaFree(q.count);
        if (q.count_pinned) cudaFreeHost(q.count_pinned);
        if (q.in_done) cudaEventDestroy(q.in_done);
        if (q.comp_done) cudaEventDestroy(q.comp_done);
        if (q.out_done) cudaEventDestroy(q.out_done);
    }
    if (p->s_in) cudaStreamDestroy(p->s_in);
    if (p->s_comp) cudaStreamDestroy(p->s_comp);
    if (p->s_out) cudaStreamDestroy(p->s_out);
    if (p->ev_caller) cudaEventDestroy(p->ev_caller);
    (void)cudaGetLastError();
}

extern "C" int ardiff_pipeline_create_slots(ardiff_head* head, int64_t max_n, int32_t d, int32_t Dc, int32_t C,
                                            int32_t n_slots, ardiff_pipeline** out) {
    if (!head || !out) return ARDIFF_ERR_NULL;
    *out = nullptr;
    if (max_n < 1 || max_n >= ((int64_t)1 << 31) || d < 1 || d > 65536 || Dc < 1 || C < 1) return ARDIFF_ERR_SHAPE;
    if (n_slots < 1 || n_slots > ARDIFF_PIPELINE_MAX_SLOTS) return ARDIFF_ERR_SHAPE;
    // the head kernel indexes the staging buffers with the head's own widths and runs at most max_tokens survivors
    const ardiff_head_desc* hd = ardiff::head_desc(head);
    if (Dc != hd->Dc || C != hd->C || max_n > hd->max_tokens) return ARDIFF_ERR_SHAPE;
    ardiff_pipeline* p = new (std::nothrow) ardiff_pipeline();
    if (!p) return ARDIFF_ERR_NOMEM;
    p->head = head;
    p->max_n = max_n;
    p->d = d; p->Dc = Dc; p->C = C;
    p->n_slots = n_slots;
    if (cudaGetDevice(&p->device) != cudaSuccess) { delete p; return ARDIFF_ERR_CUDA; }
    bool ok = true;
    for (int s = 0; s < n_slots; ++s) {
        Slot& q = p->slot[s];
        ok &= cudaMalloc(&q.feat, (size_t)max_n * d * 2) == cudaSuccess;
        ok &= cudaMalloc(&q.cond, (size_t)max_n * Dc * 2) == cudaSuccess;
        ok &= cudaMalloc(&q.noise, (size_t)max_n * C * 4) == cudaSuccess;
        ok &= cudaMalloc(&q.out, (size_t)max_n * C * 4) == cudaSuccess;
        ok &= cudaMalloc(&q.mask, (size_t)max_n) == cudaSuccess;
        ok &= cudaMalloc(&q.idx, (size_t)max_n * 4) == cudaSuccess;
        ok &= cudaMalloc(&q.count, 4) == cudaSuccess;
    }
    if (!ok) {
        (void)cudaGetLastError();
        free_all(p);
        delete p;
        return ARDIFF_ERR_NOMEM;
    }
    // streams and events only when the asynchronous calls can be used; one slot keeps create() as light as before
    if (n_slots > 1) {
        ok &= cudaStreamCreateWithFlags(&p->s_in, cudaStreamNonBlocking) == cudaSuccess;
        ok &= cudaStreamCreateWithFlags(&p->s_comp, cudaStreamNonBlocking) == cudaSuccess;
        ok &= cudaStreamCreateWithFlags(&p->s_out, cudaStreamNonBlocking) == cudaSuccess;
        ok &= cudaEventCreateWithFlags(&p->ev_caller, cudaEventDisableTiming) == cudaSuccess;
        for (int s = 0; s < n_slots; ++s) {
            Slot& q = p->slot[s];
            ok &= cudaHostAlloc(reinterpret_cast<void**>(&q.count_pinned), sizeof(int32_t), cudaHostAllocDefault) ==
                  cudaSuccess;
            ok &= cudaEventCreateWithFlags(&q.in_done, cudaEventDisableTiming) == cudaSuccess;
            ok &= cudaEventCreateWithFlags(&q.comp_done, cudaEventDisableTiming) == cudaSuccess;
            ok &= cudaEventCreateWithFlags(&q.out_done, cudaEventDisableTiming) == cudaSuccess;
        }
        if (!ok) {
            free_all(p);
            delete p;
            return ARDIFF_ERR_CUDA;
        }
    }
    *out = p;
    return ARDIFF_OK;
}

extern "C" int ardiff_pipeline_create(ardiff_head* head, int64_t max_n, int32_t d, int32_t Dc, int32_t C,
                                      ardiff_pipeline** out) {
    return ardiff_pipeline_create_slots(head, max_n, d, Dc, C, 1, out);
}

extern "C" int ardiff_pipeline_destroy(ardiff_pipeline* p) {
    if (!p) return ARDIFF_OK;
    cudaSetDevice(p->device);
    cudaDeviceSynchronize();
    free_all(p);
    delete p;
    return ARDIFF_OK;
}

extern "C" int ardiff_pipeline_run_host(ardiff_pipeline* p, const void* feat, const void* cond, const float* noise,
                                        int64_t n, float tau, const float* t_sched, int32_t K, float* out,
                                        uint8_t* mask, int32_t* count, void* stream) {
    if (!p || !t_sched || !count) return ARDIFF_ERR_NULL;
    if (n > 0 && (!feat || !cond || !noise || !out || !mask)) return ARDIFF_ERR_NULL;  // an empty batch may pass NULL
    if (n < 0 || n > p->max_n) return ARDIFF_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Slot& q = p->slot[0];
    // Batches submitted earlier may still be in flight on the pipeline's own streams, and they use the same
    // head (its scratch, its counters): this call's work is ordered on the device after every one of them.
    // Slot 0's staging buffers are reused here, so its batch is waited for and delivered as _wait would.
    for (int s = 1; s < p->n_slots; ++s)
        if (p->slot[s].used && cudaStreamWaitEvent(st, p->slot[s].out_done, 0) != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (q.used) {
        if (cudaEventSynchronize(q.out_done) != cudaSuccess) return ARDIFF_ERR_CUDA;
        if (q.rc == ARDIFF_OK && q.count_user) *q.count_user = *q.count_pinned;
        q.used = false;
    }
    const size_t nn = (size_t)n;
    bool ok = true;
    ok &= copy_async(q.feat, feat, nn * p->d * 2, cudaMemcpyHostToDevice, st);
    ok &= copy_async(q.cond, cond, nn * p->Dc * 2, cudaMemcpyHostToDevice, st);
    ok &= copy_async(q.noise, noise, nn * p->C * 4, cudaMemcpyHostToDevice, st);
    ok &= (nn == 0 || cudaMemsetAsync(q.out, 0, nn * p->C * 4, st) == cudaSuccess);
    if (!ok) return ARDIFF_ERR_CUDA;
    int rc = ardiff_entropy_gate(q.feat, n, p->d, tau, q.mask, q.idx, q.count, st);
    if (rc != ARDIFF_OK) return rc;
    int launches = ardiff::get_launch_count();
    rc = ardiff_head_sample(p->head, q.cond, q.noise, t_sched, K, q.idx, q.count, q.out, st);
    if (rc != ARDIFF_OK) return rc;
    launches += ardiff::get_launch_count();
    ok &= copy_async(out, q.out, nn * p->C * 4, cudaMemcpyDeviceToHost, st);
    ok &= copy_async(mask, q.mask, nn, cudaMemcpyDeviceToHost, st);
    ok &= copy_async(count, q.count, 4, cudaMemcpyDeviceToHost, st);
    if (!ok || cudaStreamSynchronize(st) != cudaSuccess) return ARDIFF_ERR_CUDA;
    ardiff::set_launch_count(launches);
    return ARDIFF_OK;
}

extern "C" int ardiff_pipeline_submit(ardiff_pipeline* p, int32_t slot, const void* feat, const void* cond,
                                      const float* noise, int64_t n, float tau, const float* t_sched, int32_t K,
                                      float* out, uint8_t* mask, int32_t* count, void* stream) {
    if (!p || !t_sched || !count) return ARDIFF_ERR_NULL;
    if (n > 0 && (!feat || !cond || !noise || !out || !mask)) return ARDIFF_ERR_NULL;  // an empty batch may pass NULL
    if (p->n_slots < 2) return ARDIFF_ERR_UNSUPPORTED;
    if (slot < 0 || slot >= p->n_slots || n < 0 || n > p->max_n) return ARDIFF_ERR_SHAPE;
    Slot& q = p->slot[slot];
    const size_t nn = (size_t)n;
    bool ok = true;
    // everything of this submission comes after what the caller's stream holds now
    ok &= cudaEventRecord(p->ev_caller, static_cast<cudaStream_t>(stream)) == cudaSuccess;
    ok &= cudaStreamWaitEvent(p->s_in, p->ev_caller, 0) == cudaSuccess;
    if (q.used) {
        // the slot's previous batch: its kernels are done with the inputs, its results have left
        ok &= cudaStreamWaitEvent(p->s_in, q.comp_done, 0) == cudaSuccess;
        ok &= cudaStreamWaitEvent(p->s_comp, q.out_done, 0) == cudaSuccess;
    }
    ok &= copy_async(q.feat, feat, nn * p->d * 2, cudaMemcpyHostToDevice, p->s_in);
    ok &= copy_async(q.cond, cond, nn * p->Dc * 2, cudaMemcpyHostToDevice, p->s_in);
    ok &= copy_async(q.noise, noise, nn * p->C * 4, cudaMemcpyHostToDevice, p->s_in);
    ok &= cudaEventRecord(q.in_done, p->s_in) == cudaSuccess;

    ok &= cudaStreamWaitEvent(p->s_comp, q.in_done, 0) == cudaSuccess;
    ok &= (nn == 0 || cudaMemsetAsync(q.out, 0, nn * p->C * 4, p->s_comp) == cudaSuccess);
    int rc = ARDIFF_OK;
    int launches = 0;
    if (ok) {
        rc = ardiff_entropy_gate(q.feat, n, p->d, tau, q.mask, q.idx, q.count, p->s_comp);
        launches = ardiff::get_launch_count();
        if (rc == ARDIFF_OK) {
            rc = ardiff_head_sample(p->head, q.cond, q.noise, t_sched, K, q.idx, q.count, q.out, p->s_comp);
            launches += ardiff::get_launch_count();
        }
    }
    // the events are recorded even after a failed launch so that wait() and later submissions never block
    ok &= cudaEventRecord(q.comp_done, p->s_comp) == cudaSuccess;
    ok &= cudaStreamWaitEvent(p->s_out, q.comp_done, 0) == cudaSuccess;
    if (ok && rc == ARDIFF_OK) {
        ok &= copy_async(out, q.out, nn * p->C * 4, cudaMemcpyDeviceToHost, p->s_out);
        ok &= copy_async(mask, q.mask, nn, cudaMemcpyDeviceToHost, p->s_out);
        ok &= copy_async(q.count_pinned, q.count, 4, cudaMemcpyDeviceToHost, p->s_out);
    }
    q.count_user = count;
    ok &= cudaEventRecord(q.out_done, p->s_out) == cudaSuccess;
    q.used = true;
    q.rc = !ok ? ARDIFF_ERR_CUDA : rc;
    ardiff::set_launch_count(launches);
    return q.rc;
}

extern "C" int ardiff_pipeline_wait(ardiff_pipeline* p, int32_t slot) {
    if (!p) return ARDIFF_ERR_NULL;
    if (p->n_slots < 2) return ARDIFF_ERR_UNSUPPORTED;
    if (slot < 0 || slot >= p->n_slots) return ARDIFF_ERR_SHAPE;
    Slot& q = p->slot[slot];
    if (!q.used) return ARDIFF_OK;
    if (cudaEventSynchronize(q.out_done) != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (q.rc == ARDIFF_OK && q.count_user) *q.count_user = *q.count_pinned;
    return q.rc;
}

extern "C" int ardiff_pipeline_join(ardiff_pipeline* p, void* stream) {
    if (!p) return ARDIFF_ERR_NULL;
    if (p->n_slots < 2) return ARDIFF_ERR_UNSUPPORTED;
    bool ok = true;
    for (int s = 0; s < p->n_slots; ++s)
        if (p->slot[s].used)
            ok &= cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), p->slot[s].out_done, 0) == cudaSuccess;
    return ok ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}
