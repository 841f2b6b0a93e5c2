// Arguments and host-side launchers of the weight-stationary kernels (stationary.cuh), for the entry points.
#pragma once

#include <cstddef>

#include "plan.hpp"

namespace ftp {

struct ConvRowsArgs {
    const float* in;        // [N][Cin][H][W]
    const float* w;         // [Cin][K*K][CoutPad]: per input channel and tap, the 8-padded output channels
    const float* bias;      // [Cout] or null
    float* out;             // [N][Cout][H][W], or the pooled map [N][Cout][H/2][W/2] when pool != 0
    unsigned char* arg;     // pool: arg-max (dy * 2 + dx, first maximum in row-major order) per pooled value
    int N, Cin, Cout, CoutPad, H, W;
    float slope;            // leaky-ReLU slope (act != 0)
    int act, pool;          // act == 0: plain sums (input delta)
    int rp_img;             // row pairs per image = ceil(H / 2)
    int x_tiles, co_tiles;  // blockIdx.x = (rp_tile * x_tiles + x_tile) * co_tiles + co_tile
};

struct FilterGradRowsArgs {
    const float* dz;        // [N][Cout][H][W]: delta in front of the activation
    const float* x;         // [N][Cin][H][W]: the layer's input
    float* partial;         // [splits][set_floats]; the layer's filter [Cout][Cin][K][K] at filter_off, its bias at bias_off
    long long set_floats, filter_off, bias_off;
    int N, Cin, Cout, H, W;
    int rp_img, x_tiles;    // row pairs per image, column tiles
    int stages;             // (row-pair tiles) x (column tiles) over the whole batch
    int splits;             // shares of the stages; gridDim.x = co_tiles * ci_tiles * splits
    int co_tiles, ci_tiles;
};

struct ThinBwdArgs {
    const float* dyp;           // [N][Cout][OH][OW] delta at the pooled map
    const float* yp;            // [N][Cout][OH][OW] pooled output (sign of the activation at the arg-max)
    const unsigned char* arg;   // [N][Cout][OH][OW]
    const float* x;             // [N][Cin][2 OH][2 OW]
    const float* filter;        // [Cout][Cin][3][3]
    float* dx;                  // [N][Cin][2 OH][2 OW] or null
    float* partial;             // [gridDim.x][set_floats]
    long long set_floats, filter_off, bias_off;
    int N, Cin, Cout, OH, OW;
    int tiles_y, tiles_x;       // tiles per image
    float slope;
};

// Launchers (stationary.cu); `stream` is a cudaStream_t.  They fill in the tiling fields of the arguments.
bool st_prepare_device();                                                   // opt-in shared-memory sizes; once per device
void st_launch_conv_rows(ConvRowsArgs& a, int k, int co_tile, int threads, int blocks, void* stream);   // threads: 256 or 128
void st_launch_filter_grad_rows(FilterGradRowsArgs& a, int k, int blocks, void* stream);
void st_launch_delta_act(const float* dy, const float* y, const unsigned char* arg, float* dz, size_t count, int pooled_width,
                         float slope, int pool, void* stream);
void st_launch_thin_bwd(const ThinBwdArgs& a, int blocks, void* stream);
size_t st_conv_smem_bytes(int k, int co_tile, int threads);
size_t st_filter_grad_smem_bytes(int k);

}  // namespace ftp
