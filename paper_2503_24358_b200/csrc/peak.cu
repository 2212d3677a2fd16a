// Measurement aid: a register-resident chain of single-precision multiply-adds that saturates the FP32 pipes, so
// that the benchmark can quote the key kernel's in-block work against a MEASURED FP32 peak of the GPU it runs on
// instead of the nominal 148 SMs x 128 lanes x 2 x clock.  No part of the method runs here.
#include "squat_internal.cuh"

namespace {

constexpr int PEAK_THREADS = 1024;       // 8 warps per scheduler
constexpr int PEAK_ACC = 8;              // independent chains per thread (scalar: 8 floats, packed: 8 pairs)
constexpr int PEAK_UNROLL = 8;

template <bool PACKED>
__global__ void __launch_bounds__(PEAK_THREADS, 1) fp32_peak_kernel(int iters, float seed, float *sink)
{
    const float a = 1.0f + 1e-7f * seed, b = 1e-9f * (float)threadIdx.x;
    if (PACKED) {
        unsigned long long acc[PEAK_ACC], aa, bb;
        asm("mov.b64 %0, {%1, %1};" : "=l"(aa) : "f"(a));
        asm("mov.b64 %0, {%1, %1};" : "=l"(bb) : "f"(b));
#pragma unroll
        for (int i = 0; i < PEAK_ACC; ++i) {
            const float v = (float)(i + 1);
            asm("mov.b64 %0, {%1, %1};" : "=l"(acc[i]) : "f"(v));
        }
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int u = 0; u < PEAK_UNROLL; ++u)
#pragma unroll
                for (int i = 0; i < PEAK_ACC; ++i)
                    asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(acc[i]) : "l"(aa), "l"(bb));
        }
        float s = 0.0f;
#pragma unroll
        for (int i = 0; i < PEAK_ACC; ++i) {
            float lo, hi;
            asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc[i]));
            s += lo + hi;
        }
        if (s == -1.0f) *sink = s;           // never true: keeps the chains alive
    } else {
        float acc[PEAK_ACC];
#pragma unroll
        for (int i = 0; i < PEAK_ACC; ++i) acc[i] = (float)(i + 1);
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int u = 0; u < PEAK_UNROLL; ++u)
#pragma unroll
                for (int i = 0; i < PEAK_ACC; ++i)
                    asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(acc[i]) : "f"(a), "f"(b));
        }
        float s = 0.0f;
#pragma unroll
        for (int i = 0; i < PEAK_ACC; ++i) s += acc[i];
        if (s == -1.0f) *sink = s;
    }
}

}  // namespace

extern "C" int squat_fp32_peak_probe(int packed, int iters, float *sink, long long *flops_host, void *stream)
{
    if (!sink || iters <= 0 || iters > (1 << 20) || (packed != 0 && packed != 1)) return SQUAT_ERR_INVALID_ARG;
    int dev = 0, sms = 148;
    SQUAT_CUDA(cudaGetDevice(&dev));
    SQUAT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int grid = 2 * sms;                // two waves of one CTA per SM
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (packed) fp32_peak_kernel<true><<<grid, PEAK_THREADS, 0, st>>>(iters, 0.0f, sink);
    else fp32_peak_kernel<false><<<grid, PEAK_THREADS, 0, st>>>(iters, 0.0f, sink);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    if (flops_host)
        *flops_host = 2LL * (packed ? 2 : 1) * PEAK_ACC * PEAK_UNROLL * (long long)iters * PEAK_THREADS * grid;
    return SQUAT_OK;
}
