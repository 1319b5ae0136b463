// Register-only FP64 tensor-core (DMMA) throughput probe: the denominator of the
// FP64 roofline fraction.  Eight independent m16n8k8 accumulator chains per warp,
// 16 warps per SM, no memory traffic.
#include <cuda_runtime.h>

#include "../../include/tbsyrk.h"
#include "device_utils.cuh"
#include "runtime.h"

namespace {

__global__ void __launch_bounds__(512) dmma_probe_kernel(double* out, int iters, double seed) {
    double a[4], b[2], c[8][4];
    for (int i = 0; i < 4; ++i) a[i] = seed * (threadIdx.x + i);
    for (int i = 0; i < 2; ++i) b[i] = seed * (threadIdx.x * 3 + i);
    for (int j = 0; j < 8; ++j)
        for (int i = 0; i < 4; ++i) c[j][i] = 0.0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            asm volatile(
                "mma.sync.aligned.m16n8k8.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                : "+d"(c[j][0]), "+d"(c[j][1]), "+d"(c[j][2]), "+d"(c[j][3])
                : "d"(a[0]), "d"(a[1]), "d"(a[2]), "d"(a[3]), "d"(b[0]), "d"(b[1]));
    }
    double s = 0;
    for (int j = 0; j < 8; ++j)
        for (int i = 0; i < 4; ++i) s += c[j][i];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// Self-test of the bounded waits: one warp waits on an mbarrier that nothing ever arrives on.  The wait
// gives up after its time limit (about two seconds), the kernel records the status bit and returns
// normally, exactly as the SYRK kernels do when a pipeline stalls.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(int* status) {
    __shared__ uint64_t bar;
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tbsyrk::mbar_init(&bar, 1);
        tbsyrk::mbar_fence_init();
    }
    __syncwarp();
    if (threadIdx.x == 0 && !tbsyrk::mbar_wait_bounded(&bar, 0, &abort_flag)) atomicOr(status, tbsyrk::kStatusWaitFull);
    __syncwarp();
}

}  // namespace

extern "C" int syrk_probe_f64_mma_peak(int iters, double* tflops) {
    if (!tflops) return SYRK_ERR_NULL;
    if (iters < 1 || iters > 1000000) return SYRK_ERR_SIZE;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return SYRK_ERR_NO_DEVICE;
    }
    const int threads = 512, blocks = sms;
    double* out = nullptr;
    if (cudaMalloc(&out, sizeof(double) * blocks * threads) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_ALLOC; }
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    float best = 1e30f;
    dmma_probe_kernel<<<blocks, threads>>>(out, iters / 10 + 1, 1e-9);   // warm-up
    for (int rep = 0; rep < 3; ++rep) {
        cudaEventRecord(e0);
        dmma_probe_kernel<<<blocks, threads>>>(out, iters, 1e-9);
        cudaEventRecord(e1);
        if (cudaEventSynchronize(e1) != cudaSuccess) { cudaGetLastError(); best = -1.f; break; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (ms < best) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(out);
    if (best <= 0.f) return SYRK_ERR_CUDA;
    const double flops = double(blocks) * (threads / 32) * double(iters) * 8 * (2.0 * 16 * 8 * 8);
    *tflops = flops / (double(best) * 1e-3) * 1e-12;
    return SYRK_OK;
}

int syrk_selftest_bounded_wait(void* stream) {
    std::lock_guard<std::mutex> lock(tbsyrk::runtime().mu);
    tbsyrk::DeviceState* ds = nullptr;
    int rc = tbsyrk::get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        tbsyrk::status_for_stream(ds, static_cast<cudaStream_t>(stream)));
    return cudaGetLastError() == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}
