// Host-buffer front end: copies one batch to the device, runs gate -> head, copies results back.
#include <cuda_runtime.h>
#include <stdint.h>

#include <new>

#include "../../include/ardiff.h"
#include "common.cuh"

struct ardiff_pipeline {
    ardiff_head* head;
    int device;
    int64_t max_n;
    int32_t d, Dc, C;
    void* feat;
    void* cond;
    float* noise;
    float* out;
    uint8_t* mask;
    int32_t* idx;
    int32_t* count;
};

extern "C" int ardiff_pipeline_create(ardiff_head* head, int64_t max_n, int32_t d, int32_t Dc, int32_t C,
                                      ardiff_pipeline** out) {
    if (!head || !out) return ARDIFF_ERR_NULL;
    *out = nullptr;
    if (max_n < 1 || max_n >= ((int64_t)1 << 31) || d < 1 || d > 65536 || Dc < 1 || C < 1) return ARDIFF_ERR_SHAPE;
    ardiff_pipeline* p = new (std::nothrow) ardiff_pipeline();
    if (!p) return ARDIFF_ERR_NOMEM;
    p->head = head;
    p->max_n = max_n;
    p->d = d; p->Dc = Dc; p->C = C;
    if (cudaGetDevice(&p->device) != cudaSuccess) { delete p; return ARDIFF_ERR_CUDA; }
    bool ok = true;
    ok &= cudaMalloc(&p->feat, (size_t)max_n * d * 2) == cudaSuccess;
    ok &= cudaMalloc(&p->cond, (size_t)max_n * Dc * 2) == cudaSuccess;
    ok &= cudaMalloc(&p->noise, (size_t)max_n * C * 4) == cudaSuccess;
    ok &= cudaMalloc(&p->out, (size_t)max_n * C * 4) == cudaSuccess;
    ok &= cudaMalloc(&p->mask, (size_t)max_n) == cudaSuccess;
    ok &= cudaMalloc(&p->idx, (size_t)max_n * 4) == cudaSuccess;
    ok &= cudaMalloc(&p->count, 4) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        cudaFree(p->feat); cudaFree(p->cond); cudaFree(p->noise); cudaFree(p->out);
        cudaFree(p->mask); cudaFree(p->idx); cudaFree(p->count);
        delete p;
        return ARDIFF_ERR_NOMEM;
    }
    *out = p;
    return ARDIFF_OK;
}

extern "C" int ardiff_pipeline_destroy(ardiff_pipeline* p) {
    if (!p) return ARDIFF_OK;
    cudaSetDevice(p->device);
    cudaDeviceSynchronize();
    cudaFree(p->feat); cudaFree(p->cond); cudaFree(p->noise); cudaFree(p->out);
    cudaFree(p->mask); cudaFree(p->idx); cudaFree(p->count);
    delete p;
    return ARDIFF_OK;
}

extern "C" int ardiff_pipeline_run_host(ardiff_pipeline* p, const void* feat, const void* cond, const float* noise,
                                        int64_t n, float tau, const float* t_sched, int32_t K, float* out,
                                        uint8_t* mask, int32_t* count, void* stream) {
    if (!p || !feat || !cond || !noise || !t_sched || !out || !mask || !count) return ARDIFF_ERR_NULL;
    if (n < 0 || n > p->max_n) return ARDIFF_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t nn = (size_t)n;
    bool ok = true;
    ok &= cudaMemcpyAsync(p->feat, feat, nn * p->d * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(p->cond, cond, nn * p->Dc * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(p->noise, noise, nn * p->C * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemsetAsync(p->out, 0, nn * p->C * 4, st) == cudaSuccess;
    if (!ok) return ARDIFF_ERR_CUDA;
    int rc = ardiff_entropy_gate(p->feat, n, p->d, tau, p->mask, p->idx, p->count, st);
    if (rc != ARDIFF_OK) return rc;
    int launches = ardiff::get_launch_count();
    rc = ardiff_head_sample(p->head, p->cond, p->noise, t_sched, K, p->idx, p->count, p->out, st);
    if (rc != ARDIFF_OK) return rc;
    launches += ardiff::get_launch_count();
    ok &= cudaMemcpyAsync(out, p->out, nn * p->C * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(mask, p->mask, nn, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(count, p->count, 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (!ok || cudaStreamSynchronize(st) != cudaSuccess) return ARDIFF_ERR_CUDA;
    ardiff::set_launch_count(launches);
    return ARDIFF_OK;
}
