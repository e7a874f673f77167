// Experiment support: which SMs sit close to which part of the L2 (Sec. 2.1 describes chiplets with their own L2 and
// HBM stacks; a B200 is two dies behind one address space, and nothing in CUDA says which SM is on which die).
// ccl_probe_l2_latency measures, from every SM, the round-trip time of loads that bypass L1 to a set of cache lines.
// A line lives in one L2 partition; SMs of the die that holds it see it faster than SMs of the other die, so the
// per-line latency vectors of the SMs fall into two clusters (report.py --topology does the clustering).
#include <cuda_runtime.h>

#include <cstdint>

#include "ccl.h"
#include "ccl_common.h"

namespace ccl {

constexpr int kProbeLoads = 64;     // dependent loads per line and measurement

__global__ void __launch_bounds__(32) probe_l2_latency_kernel(const unsigned int* buf, int nlines, int64_t stride_words, float* lat, int* smid_out) {
    if (threadIdx.x != 0) return;
    unsigned int smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    smid_out[blockIdx.x] = (int)smid;
    for (int i = 0; i < nlines; ++i) {
        const unsigned int* p = buf + (int64_t)i * stride_words;
        unsigned int v = 0;
        // the buffer holds zeros: the next address depends on the value just loaded, so the loads form a chain
        for (int k = 0; k < 4; ++k) asm volatile("ld.global.cv.u32 %0, [%1];" : "=r"(v) : "l"(p + (v >> 31)) : "memory");
        const long long t0 = clock64();
#pragma unroll 1
        for (int k = 0; k < kProbeLoads; ++k) asm volatile("ld.global.cv.u32 %0, [%1];" : "=r"(v) : "l"(p + (v >> 31)) : "memory");
        const long long t1 = clock64();
        lat[(int64_t)blockIdx.x * nlines + i] = (float)(t1 - t0) / kProbeLoads + (float)(v >> 31);
    }
}

}  // namespace ccl

using namespace ccl;

extern "C" ccl_status ccl_probe_l2_latency(const void* zero_buf_dev, int32_t nlines, int64_t stride_bytes, int32_t nctas, float* lat_dev,
                                           int32_t* smid_dev, void* cuda_stream) {
    if (!zero_buf_dev || !lat_dev || !smid_dev) return fail(CCL_ERR_INVALID_ARG, "ccl_probe_l2_latency: NULL buffer");
    if (nlines < 1 || nctas < 1 || nctas > 4096 || stride_bytes < 4 || stride_bytes % 4) return fail(CCL_ERR_INVALID_ARG, "ccl_probe_l2_latency: bad sizes");
    if (reinterpret_cast<uintptr_t>(zero_buf_dev) & 3) return fail(CCL_ERR_ALIGN, "ccl_probe_l2_latency: buffer is not 4-byte aligned");
    // 200 KB of dynamic shared memory per CTA: at most one CTA per SM, so `nctas` = SM count puts one on every SM
    const int smem = 200 * 1024;
    static bool configured = false;
    if (!configured) {
        CCL_CUDA_TRY(cudaFuncSetAttribute(probe_l2_latency_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured = true;
    }
    probe_l2_latency_kernel<<<(unsigned)nctas, 32, smem, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const unsigned int*>(zero_buf_dev), nlines, stride_bytes / 4, lat_dev, smid_dev);
    count_launch();
    CCL_CUDA_TRY(cudaGetLastError());
    return CCL_OK;
}
