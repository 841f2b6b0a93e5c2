// Host-side launchers of the weight-stationary kernels: a translation unit of their own, so that the kernels
// compile beside the fused-stack kernels instead of after them.
#include <cuda_runtime.h>

#include <algorithm>

#include "stationary.cuh"

namespace ftp {

namespace {

template <int K, int CO, int VEC, int T>
void launch_conv(const ConvRowsArgs& a, int blocks, cudaStream_t st)
{
    conv_rows_kernel<K, CO, VEC, T><<<blocks, T, StGeom<K, CO, T>::smem_bytes, st>>>(a);
}

template <int K, int CO, int T>
void launch_conv_vec(const ConvRowsArgs& a, int blocks, cudaStream_t st)
{
    if ((a.W & 3) == 0) launch_conv<K, CO, 4, T>(a, blocks, st);
    else if ((a.W & 1) == 0) launch_conv<K, CO, 2, T>(a, blocks, st);
    else launch_conv<K, CO, 1, T>(a, blocks, st);
}

template <int K, int CO, int T>
bool conv_attr_t()
{
    return cudaFuncSetAttribute(conv_rows_kernel<K, CO, 4, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, StGeom<K, CO, T>::smem_bytes) == cudaSuccess &&
           cudaFuncSetAttribute(conv_rows_kernel<K, CO, 2, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, StGeom<K, CO, T>::smem_bytes) == cudaSuccess &&
           cudaFuncSetAttribute(conv_rows_kernel<K, CO, 1, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, StGeom<K, CO, T>::smem_bytes) == cudaSuccess;
}
template <int K, int CO> bool conv_attr() { return conv_attr_t<K, CO, 256>() && conv_attr_t<K, CO, 128>(); }

}  // namespace

bool st_prepare_device()
{
    return conv_attr<1, 64>() && conv_attr<3, 64>() && conv_attr<1, 32>() && conv_attr<3, 32>() &&
           cudaFuncSetAttribute(thin_bwd_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kThinSmemBytes) == cudaSuccess &&
           cudaFuncSetAttribute(thin_bwd_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kThinSmemBytes) == cudaSuccess &&
           cudaFuncSetAttribute(thin_bwd_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kThinSmemBytes) == cudaSuccess &&
           cudaFuncSetAttribute(thin_bwd_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kThinSmemBytes) == cudaSuccess &&
           cudaFuncSetAttribute(filter_grad_1x1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kF1SmemBytes) == cudaSuccess &&
           cudaFuncSetAttribute(filter_grad_rows_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, FgGeom<3>::smem_bytes) == cudaSuccess;
}

size_t st_conv_smem_bytes(int k, int co_tile, int threads)
{
    if (threads == 128)
        return k == 3 ? (co_tile == 64 ? StGeom<3, 64, 128>::smem_bytes : StGeom<3, 32, 128>::smem_bytes)
                      : (co_tile == 64 ? StGeom<1, 64, 128>::smem_bytes : StGeom<1, 32, 128>::smem_bytes);
    return k == 3 ? (co_tile == 64 ? StGeom<3, 64>::smem_bytes : StGeom<3, 32>::smem_bytes)
                  : (co_tile == 64 ? StGeom<1, 64>::smem_bytes : StGeom<1, 32>::smem_bytes);
}

size_t st_filter_grad_smem_bytes(int k) { return k == 3 ? FgGeom<3>::smem_bytes : kF1SmemBytes; }

template <int T>
void launch_conv_t(const ConvRowsArgs& a, int k, int co_tile, int blocks, cudaStream_t st)
{
    if (k == 3 && co_tile == 64) launch_conv_vec<3, 64, T>(a, blocks, st);
    else if (k == 3) launch_conv_vec<3, 32, T>(a, blocks, st);
    else if (co_tile == 64) launch_conv_vec<1, 64, T>(a, blocks, st);
    else launch_conv_vec<1, 32, T>(a, blocks, st);
}

void st_launch_conv_rows(ConvRowsArgs& a, int k, int co_tile, int threads, int blocks, void* stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    a.rp_img = (a.H + 1) / 2; a.x_tiles = (a.W + kStCols - 1) / kStCols; a.co_tiles = (a.Cout + co_tile - 1) / co_tile;
    if (threads == 128) launch_conv_t<128>(a, k, co_tile, blocks, st);
    else launch_conv_t<256>(a, k, co_tile, blocks, st);
}

void st_launch_filter_grad_rows(FilterGradRowsArgs& a, int k, int blocks, void* stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    a.rp_img = (a.H + 1) / 2; a.x_tiles = (a.W + kStCols - 1) / kStCols;
    a.co_tiles = (a.Cout + kFgCo - 1) / kFgCo; a.ci_tiles = (a.Cin + kFgCi - 1) / kFgCi;
    if (k == 3) { filter_grad_rows_kernel<3><<<blocks, kStThreads, FgGeom<3>::smem_bytes, st>>>(a); return; }
    // 1 x 1: a contraction over the flat pixels of an image, 64 x 128 channel slices
    a.co_tiles = (a.Cout + kF1Co - 1) / kF1Co; a.ci_tiles = (a.Cin + kF1Ci - 1) / kF1Ci;
    filter_grad_1x1_kernel<<<blocks, kStThreads, kF1SmemBytes, st>>>(a);
}

void st_launch_delta_act(const float* dy, const float* y, const unsigned char* arg, float* dz, size_t count, int pooled_width,
                         float slope, int pool, void* stream)
{
    const int blocks = (int)std::min<size_t>((count + 255) / 256, (size_t)kSmCount * 16);
    delta_act_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(dy, y, arg, dz, count, pooled_width, slope, pool);
}

void st_launch_thin_bwd(const ThinBwdArgs& a, int blocks, void* stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (a.Cin) {
    case 1: thin_bwd_kernel<1><<<blocks, kStThreads, kThinSmemBytes, st>>>(a); break;
    case 2: thin_bwd_kernel<2><<<blocks, kStThreads, kThinSmemBytes, st>>>(a); break;
    case 3: thin_bwd_kernel<3><<<blocks, kStThreads, kThinSmemBytes, st>>>(a); break;
    default: thin_bwd_kernel<4><<<blocks, kStThreads, kThinSmemBytes, st>>>(a); break;
    }
}

}  // namespace ftp
