// ftp_fma_peak: a register-only fp32 FMA loop on every SM, the measured ceiling that the
// roofline fractions of the fp32 (CUDA-core) kernels are quoted against.  It moves no memory: the
// only global access is one store per thread at the end, which keeps the compiler from removing
// the arithmetic.
#include <cuda_runtime.h>

#include "ftp.h"

namespace {

constexpr int kChains = 16;     // independent accumulators per thread: enough to cover the FMA latency at 4 warps per scheduler
constexpr int kUnroll = 8;

__global__ void __launch_bounds__(512, 2) fma_peak_kernel(float* __restrict__ out, long long iters, float a, float b)
{
    float acc[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc[c] = (float)(threadIdx.x + c);
    for (long long i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
#pragma unroll
            for (int c = 0; c < kChains; ++c) acc[c] = fmaf(acc[c], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += acc[c];
    out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace

extern "C" int ftp_fma_peak(float* out, size_t out_count, long long iters, double* flops, void* stream)
{
    int dev = 0, sms = 0;
    if (!out || iters <= 0) return FTP_ERR_ARG;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return FTP_ERR_CUDA;
    const int blocks = sms * 2, threads = 512;
    if (out_count < (size_t)blocks * threads) return FTP_ERR_ARG;
    fma_peak_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(out, iters, 0.999f, 0.001f);
    if (flops) *flops = 2.0 * (double)blocks * threads * (double)iters * kUnroll * kChains;
    return cudaGetLastError() == cudaSuccess ? FTP_OK : FTP_ERR_CUDA;
}
