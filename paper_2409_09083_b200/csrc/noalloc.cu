// ftp_loss_mse_static: the mean-squared-error loss and its delta for callers that must not
// allocate device memory.  The per-block partial sums that ftp_loss_mse keeps in the caller's
// workspace live here in a fixed array that is part of the library image, so the call needs no
// workspace, no plan and no allocation of any kind.
#include <cuda_runtime.h>

#include <mutex>

#include "ftp.h"

namespace {

constexpr int    kChunk     = 16384;                                  // elements per block
constexpr int    kMaxBlocks = (int)(FTP_LOSS_STATIC_MAX_COUNT / kChunk);   // 4096 partial sums
constexpr int    kThreads   = 256;
constexpr int    kMaxDevices = 64;

// One partial sum per block.  Every GPU that loads the library holds these 16 KB until the
// process exits.  In host code this name is only a handle for cudaGetSymbolAddress; it is not a
// device address and must never be handed to a kernel as is.
static __device__ __align__(256) float g_loss_partials[kMaxBlocks];

std::mutex g_mutex;
float*     g_partials_on_device[kMaxDevices];     // resolved once per device, see scratch_for_current_device

// Device address of the array on the current device (each device has its own copy).
int scratch_for_current_device(float** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return FTP_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return FTP_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_partials_on_device[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_loss_partials) != cudaSuccess || !p) {
            cudaGetLastError();
            return FTP_ERR_CUDA;
        }
        g_partials_on_device[dev] = static_cast<float*>(p);
    }
    *out = g_partials_on_device[dev];
    return FTP_OK;
}

// Block b handles elements [b * kChunk, (b + 1) * kChunk): writes the delta and its partial sum
// of squared differences.  Every launched block overwrites its own slot, so nothing left in
// the array by an earlier call is ever read.
__global__ void __launch_bounds__(kThreads) loss_static_delta_kernel(const float* __restrict__ y, const float* __restrict__ t,
                                                                     float* __restrict__ d, size_t count, float scale,
                                                                     float* __restrict__ partials)
{
    __shared__ float red[kThreads];
    const size_t begin = (size_t)blockIdx.x * kChunk;
    const size_t end = begin + kChunk < count ? begin + kChunk : count;
    float s = 0.f;
    for (size_t e = begin + threadIdx.x; e < end; e += kThreads) {
        const float diff = y[e] - t[e];
        if (d) d[e] = scale * diff;
        s += diff * diff;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int k = kThreads / 2; k >= 1; k >>= 1) {
        if ((int)threadIdx.x < k) red[threadIdx.x] += red[threadIdx.x + k];
        __syncthreads();
    }
    if (threadIdx.x == 0) partials[blockIdx.x] = red[0];
}

// Sums the first n partials in a fixed order (strided per thread, then a tree) and writes the mean.
__global__ void __launch_bounds__(kThreads) loss_static_finish_kernel(const float* __restrict__ partials, int n, float inv_count,
                                                                      float* __restrict__ loss)
{
    __shared__ float red[kThreads];
    float s = 0.f;
    for (int i = threadIdx.x; i < n; i += kThreads) s += partials[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int k = kThreads / 2; k >= 1; k >>= 1) {
        if ((int)threadIdx.x < k) red[threadIdx.x] += red[threadIdx.x + k];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = red[0] * inv_count;
}

}  // namespace

extern "C" int ftp_loss_mse_static(const float* y, const float* target, float* dy, float* loss_out, size_t count,
                                   void* stream)
{
    if (!y || !target || (!dy && !loss_out) || count == 0) return FTP_ERR_ARG;
    if (count > (size_t)FTP_LOSS_STATIC_MAX_COUNT) return FTP_ERR_TOO_LARGE;
    float* partials = nullptr;
    const int rc = scratch_for_current_device(&partials);
    if (rc != FTP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int blocks = (int)((count + kChunk - 1) / kChunk);
    loss_static_delta_kernel<<<blocks, kThreads, 0, st>>>(y, target, dy, count, 2.0f / (float)count, partials);
    if (loss_out) loss_static_finish_kernel<<<1, kThreads, 0, st>>>(partials, blocks, 1.0f / (float)count, loss_out);
    return cudaGetLastError() == cudaSuccess ? FTP_OK : FTP_ERR_CUDA;
}
