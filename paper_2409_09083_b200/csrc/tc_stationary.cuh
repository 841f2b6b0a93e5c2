// bf16 path, executed groups of one conv layer (with its pool): the filter gradient by a weight-stationary
// tensor-core kernel, the forward pass and the input delta by a banded tensor-core convolution (further down),
// and their helpers (dz planes, window unroll / fold for the first layer).
//
// Filter gradient.  In the fused tile-stack kernel every sub-tile adds its whole partial filter gradient (K*K*cout*cin fp32) to
// the block's partial set, because tensor memory cannot keep the accumulators of a wide layer across sub-tiles.
// For layers with hundreds of channels that flush costs several times the MMAs.  Here the roles are turned
// round: a block owns a slice of the FILTER GRADIENT (64 or 128 output channels x up to 48 input channels x all
// window positions; K*K accumulators of `ncols` columns each, plus 16 columns for the bias gradient) and keeps
// it in tensor memory while bands of rows of the whole batch stream past it, so the gradient leaves the SM
// once.  The pixels are dealt out in `shares`; a share is one partial gradient set of Section 4.1, summed by
// the same cross-tile reduction as the sets of the fused kernels.
//
// A band is R rows x Cw columns (Cw = W, or a column chunk of at most 126 columns of a wider map) of one image at
// the conv's resolution.  The delta in front of the activation (dz, bf16 planes, written by the input-delta
// kernel of the layer above or by delta_act_planes_kernel) and the layer's saved input map arrive by TMA tensor
// copies into tiles of the same pitch Wp = Cw + K - 1: dz at columns 0 .. Cw-1 with zeros behind them (beyond
// the edge of the chunk's tensor map), the input shifted by the padding.  With equal pitches one run of 16 consecutive tile entries
// is a K step of both operands (MN-major, 8 pixels x 8 channels per core matrix), and window position (ky, kx)
// only moves the start of the input operand by ky * Wp + kx entries.  Two stages: the copies of the next band
// run behind the MMAs of the current one.
#pragma once

#include <algorithm>

#include "kernels_tc.cuh"

namespace ftp {

// Tensor maps of bf16 planes [N x C16/8][H][W][8] as the TMA engine sees them here: 3-dimensional, rows of 2 W
// eight-byte elements (a pixel's 8 channels = two elements), so that a box row is one contiguous run of Wp pixels
// instead of Wp separate 16-byte pieces; a box row holds at most 256 elements, i.e. Wp <= 128 pixels.
struct TcFilterGradArgs {
    // dz planes, one map per column chunk: the chunk's columns only (base moved to its first column, extent = its
    // width), so that the box (Wp pixels x R rows) reads zeros behind the chunk's last column
    alignas(64) unsigned char tmap_dz[kTcMaxColChunks][128];
    alignas(64) unsigned char tmap_x[128];    // the layer's input planes, box = Wp pixels x (R + K - 1) rows
    float* partial;                           // partial sets of the group
    long long set_floats, tgp_off;            // floats per set, offset of this layer inside a set
    int* error;
    int N, K, cout16, cin16;
    int Ms, slices;                           // output channels per block (64 or 128) and number of such slices
    int ncols, nci;                           // input channels per block (multiple of 16) and number of such slices
    int R, Wp, bands_img, bands, shares;      // rows per band, tile pitch, bands per image / in the batch, pixel shares
    int ncc, Cw;                              // column chunks per row band and their width (Wp = Cw + K - 1)
    int dz_plane, x_plane, stage_bytes;       // bytes between planes of the two tiles, bytes of one stage
};

struct DeltaActPlanesArgs {
    const void* dmap; int dmap_planes;        // delta at the layer's output: bf16 planes, or fp32 NCHW (dmap_planes = 0)
    const uint4* y; const unsigned long long* arg;   // saved output (planes) and, for a fused pool, its arg-max bytes
    uint4* dz;                                // out: planes at the conv's resolution
    int N, cout, cout16, out_H, out_W, pool;
    float slope;
};

// dz = delta * act'(y), routed through the arg-max of a fused pool (zeros at the three other positions of a
// window): the same arithmetic and roundings as the fused backward kernel applies when it fills its dz tile.
__global__ void delta_act_planes_kernel(const __grid_constant__ DeltaActPlanesArgs A)
{
    const int planes = A.cout16 / 8;
    const size_t total = (size_t)A.N * planes * A.out_H * A.out_W;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const int x = (int)(e % A.out_W); size_t t = e / A.out_W;
        const int y = (int)(t % A.out_H); t /= A.out_H;
        const int pl = (int)(t % planes); const int n = (int)(t / planes);
        float v[8], yv[8];
        if (A.dmap_planes) {
            tcd::unpack8(__ldg(static_cast<const uint4*>(A.dmap) + e), v);
        } else {
            const float* d = static_cast<const float*>(A.dmap);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int ch = pl * 8 + c;
                v[c] = ch < A.cout ? __ldg(d + (((size_t)n * A.cout + ch) * A.out_H + y) * A.out_W + x) : 0.f;
            }
        }
        tcd::unpack8(__ldg(A.y + e), yv);
#pragma unroll
        for (int c = 0; c < 8; ++c) v[c] *= yv[c] > 0.f ? 1.f : A.slope;
        if (!A.pool) { A.dz[e] = tcd::pack8(v); continue; }
        const unsigned long long am = A.arg[e];
        const int W2 = 2 * A.out_W;
        uint4* o = A.dz + (((size_t)n * planes + pl) * (2 * A.out_H) + 2 * y) * W2 + 2 * x;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            float z[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) z[c] = (int)((am >> (c * 8)) & 3ull) == w ? v[c] : 0.f;
            o[(w >> 1) * W2 + (w & 1)] = tcd::pack8(z);
        }
    }
}

// First layer: the fp32 network input [N][C][H][W] -> window-unrolled bf16 planes [N][C16'/8][H][W][8] with channel
// ci * 9 + ky * 3 + kx of pixel (y, x) = input(ci, y + ky - 1, x + kx - 1) (zero outside the map and beyond 9 C).
// One thread per pixel: it reads the 9 C values of its window once and writes its entry of every plane (the
// channel -> (ci, ky, kx) arithmetic is resolved at compile time).
template <int C>
__global__ void unroll_windows_kernel(const float* __restrict__ x, uint4* __restrict__ col, int N, int H, int W)
{
    constexpr int planes = (9 * C + 15) / 16 * 2;
    const size_t HW = (size_t)H * W, total = (size_t)N * HW;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const int px = (int)(e % W); size_t t = e / W;
        const int py = (int)(t % H); const int n = (int)(t / H);
        float v[planes * 8];
        const float* ctr = x + (size_t)n * C * HW + (size_t)py * W + px;       // this pixel in channel 0
        if (py > 0 && py < H - 1 && px > 0 && px < W - 1) {                    // the whole window lies inside the map
#pragma unroll
            for (int j = 0; j < planes * 8; ++j) {
                const int ci = j / 9, tap = j - ci * 9, ky = tap / 3, kx = tap - ky * 3;
                v[j] = ci < C ? __ldg(ctr + (size_t)ci * HW + (ky - 1) * W + (kx - 1)) : 0.f;
            }
        } else {
#pragma unroll
            for (int j = 0; j < planes * 8; ++j) {
                const int ci = j / 9, tap = j - ci * 9, ky = tap / 3, kx = tap - ky * 3;
                const int yy = py + ky - 1, xx = px + kx - 1;
                v[j] = (ci < C && yy >= 0 && yy < H && xx >= 0 && xx < W) ? __ldg(ctr + (size_t)ci * HW + (ky - 1) * W + (kx - 1)) : 0.f;
            }
        }
#pragma unroll
        for (int pl = 0; pl < planes; ++pl) col[((size_t)n * planes + pl) * HW + (size_t)py * W + px] = tcd::pack8(v + 8 * pl);
    }
}

// ... and back: the delta at the network input, fp32 NCHW, as the sum over the window positions of the delta planes of
// the unrolled input: dx(ci, y, x) = sum over (ky, kx) of dcol(ci * 9 + ky * 3 + kx, y - ky + 1, x - kx + 1), in the
// order of the window positions.  One thread per pixel and all its channels: of the neighbour at window position
// (ky, kx) it needs channel ci * 9 + ky * 3 + kx for every ci.
template <int C>
__global__ void fold_windows_kernel(const __nv_bfloat16* __restrict__ dcol, float* __restrict__ dx, int N, int H, int W)
{
    constexpr int planes = (9 * C + 15) / 16 * 2;
    const size_t HW = (size_t)H * W, total = (size_t)N * HW;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const int px = (int)(e % W); size_t t = e / W;
        const int py = (int)(t % H); const int n = (int)(t / H);
        float s[C];
#pragma unroll
        for (int ci = 0; ci < C; ++ci) s[ci] = 0.f;
#pragma unroll
        for (int tap = 0; tap < 9; ++tap) {
            const int ky = tap / 3, kx = tap - ky * 3, yy = py - ky + 1, xx = px - kx + 1;
            if (yy >= 0 && yy < H && xx >= 0 && xx < W) {
                const __nv_bfloat16* src = dcol + ((size_t)n * planes * HW + (size_t)yy * W + xx) * 8;
#pragma unroll
                for (int ci = 0; ci < C; ++ci) {
                    const int j = ci * 9 + tap;
                    s[ci] += __bfloat162float(__ldg(src + (size_t)(j >> 3) * HW * 8 + (j & 7)));
                }
            }
        }
#pragma unroll
        for (int ci = 0; ci < C; ++ci) dx[((size_t)n * C + ci) * HW + (size_t)py * W + px] = s[ci];
    }
}

// the two kernels for the channel counts the route takes (9 C <= 64)
inline void launch_unroll_windows(const float* x, uint4* col, int N, int C, int H, int W, cudaStream_t st)
{
    const int blocks = (int)std::min<size_t>(((size_t)N * H * W + 255) / 256, (size_t)kSmCount * 16);
    switch (C) {
        case 1: unroll_windows_kernel<1><<<blocks, 256, 0, st>>>(x, col, N, H, W); break;
        case 2: unroll_windows_kernel<2><<<blocks, 256, 0, st>>>(x, col, N, H, W); break;
        case 3: unroll_windows_kernel<3><<<blocks, 256, 0, st>>>(x, col, N, H, W); break;
        case 4: unroll_windows_kernel<4><<<blocks, 256, 0, st>>>(x, col, N, H, W); break;
        case 5: unroll_windows_kernel<5><<<blocks, 256, 0, st>>>(x, col, N, H, W); break;
        case 6: unroll_windows_kernel<6><<<blocks, 256, 0, st>>>(x, col, N, H, W); break;
        default: unroll_windows_kernel<7><<<blocks, 256, 0, st>>>(x, col, N, H, W); break;
    }
}
inline void launch_fold_windows(const __nv_bfloat16* dcol, float* dx, int N, int C, int H, int W, cudaStream_t st)
{
    const int blocks = (int)std::min<size_t>(((size_t)N * H * W + 255) / 256, (size_t)kSmCount * 16);
    switch (C) {
        case 1: fold_windows_kernel<1><<<blocks, 256, 0, st>>>(dcol, dx, N, H, W); break;
        case 2: fold_windows_kernel<2><<<blocks, 256, 0, st>>>(dcol, dx, N, H, W); break;
        case 3: fold_windows_kernel<3><<<blocks, 256, 0, st>>>(dcol, dx, N, H, W); break;
        case 4: fold_windows_kernel<4><<<blocks, 256, 0, st>>>(dcol, dx, N, H, W); break;
        case 5: fold_windows_kernel<5><<<blocks, 256, 0, st>>>(dcol, dx, N, H, W); break;
        case 6: fold_windows_kernel<6><<<blocks, 256, 0, st>>>(dcol, dx, N, H, W); break;
        default: fold_windows_kernel<7><<<blocks, 256, 0, st>>>(dcol, dx, N, H, W); break;
    }
}

constexpr int kTcFgThreads = 256;

__global__ void __launch_bounds__(kTcFgThreads, 1) filter_grad_tc_rows_kernel(const __grid_constant__ TcFilterGradArgs A)
{
    using namespace tc;
    extern __shared__ __align__(1024) unsigned char fg_smem[];
    struct Hdr {
        unsigned long long full[2], empty[2], done;
        uint32_t tmem_base;
        volatile int failed;
        __align__(16) __nv_bfloat16 ones[64];
    };
    static_assert(sizeof(Hdr) <= kTcFgHeader, "header does not fit");
    Hdr* H = reinterpret_cast<Hdr*>(fg_smem);
    unsigned char* stages = fg_smem + kTcFgHeader;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int K = A.K, KK = K * K;

    // this block's slice of the gradient and share of the bands
    const int nroles = A.slices * A.nci;
    const int role = (int)blockIdx.x % nroles, share = (int)blockIdx.x / nroles;
    const int slice = role / A.nci, cs = role - slice * A.nci;
    const int ci0 = cs * A.ncols, cols = min(A.ncols, A.cin16 - ci0);
    const int mp = A.Ms / 8;                                            // dz planes of a full slice
    const int nd = min(mp, A.cout16 / 8 - slice * mp), np = cols / 8;   // planes this block copies per band
    const bool bias = cs == 0;
    const int b_lo = (int)((long long)share * A.bands / A.shares), b_hi = (int)((long long)(share + 1) * A.bands / A.shares);
    const int nb = b_hi - b_lo;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&H->full[s]), 1); mbar_init(smem_u32(&H->empty[s]), kTcIssuers); }
        mbar_init(smem_u32(&H->done), kTcIssuers);
        H->failed = 0;
        fence_mbar_init();
    }
    if (warp == 0) { __syncwarp(); tmem_alloc(smem_u32(&H->tmem_base), (uint32_t)kTcTmemCols); }
    // tails, planes that are never copied and everything else the tensor core may read: zeros from here on
    tcd::zero_bytes(stages, 2 * (size_t)A.stage_bytes);
    for (int i = threadIdx.x; i < 64; i += blockDim.x) H->ones[i] = __float2bfloat16(1.0f);
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = H->tmem_base;

    auto wait = [&](unsigned long long* bar, uint32_t parity, unsigned sleep_ns = 0) {
        if (H->failed) return false;
        if (mbar_wait(smem_u32(bar), parity, kWaitLimitCycles, sleep_ns)) return true;
        H->failed = 1;
        atomicExch(A.error, 1);
        return false;
    };
    if ((smem_u32(fg_smem) & 127u) != 0) {                  // tensor copies want 128-byte aligned destinations
        if (threadIdx.x == 0) { H->failed = 1; atomicExch(A.error, 1); }
        __syncthreads();
    }

    if (warp == kTcIssuers && lane == 0) {
        // producer: the two tiles of a band, one tensor copy per plane
        int issued[2] = {0, 0};
        for (int i = 0; i < nb; ++i) {
            const int s = i & 1;
            if (!wait(&H->empty[s], ((uint32_t)(i >> 1) & 1u) ^ 1u)) break;
            const int b = b_lo + i, n = b / A.bands_img, bi = b - n * A.bands_img;
            const int cc = bi % A.ncc, y0 = (bi / A.ncc) * A.R, x0 = cc * A.Cw;
            unsigned char* dzs = stages + (size_t)s * A.stage_bytes;
            unsigned char* xs = dzs + (size_t)mp * A.dz_plane;
            const uint32_t bar = smem_u32(&H->full[s]);
            mbar_expect_tx(bar, (uint32_t)((nd * A.R + np * (A.R + K - 1)) * A.Wp) * 16u);
            for (int pl = 0; pl < nd; ++pl)
                tma_load_3d(smem_u32(dzs + (size_t)pl * A.dz_plane), A.tmap_dz[cc], 0, y0, n * (A.cout16 / 8) + slice * mp + pl, bar);
            for (int pl = 0; pl < np; ++pl)
                tma_load_3d(smem_u32(xs + (size_t)pl * A.x_plane), A.tmap_x, 2 * (x0 - K / 2), y0 - K / 2, n * (A.cin16 / 8) + ci0 / 8 + pl, bar);
            ++issued[s];
        }
        if (H->failed)       // gave up somewhere: let the copies already under way land before the block leaves
            for (int s = 0; s < 2; ++s)
                if (issued[s] > 0) mbar_wait(smem_u32(&H->full[s]), (uint32_t)(issued[s] - 1) & 1u, 200000000ll);
    } else if (warp < kTcIssuers && lane == 0) {
        // MMA issue: every issuer takes every kTcIssuers-th accumulator (window positions, then the bias)
        const uint32_t a_hi = desc_hi((uint32_t)A.dz_plane), x_hi = desc_hi((uint32_t)A.x_plane);
        const uint32_t idesc = make_idesc(A.Ms, cols, true, true), idb = make_idesc(A.Ms, 16, true, true);
        const uint64_t ones_d = make_desc(smem_u32(H->ones), 0, 0);
        const int nunits = KK + (bias ? 1 : 0);
        const int nk = (A.R * A.Wp + 15) >> 4;
        for (int i = 0; i < nb; ++i) {
            const int s = i & 1;
            if (!wait(&H->full[s], (uint32_t)(i >> 1) & 1u)) break;
            fence_after_sync();
            const uint32_t dz_addr = smem_u32(stages + (size_t)s * A.stage_bytes);
            const uint32_t dz_lo0 = desc_lo(dz_addr, 128), x_lo0 = desc_lo(dz_addr + (uint32_t)(mp * A.dz_plane), 128);
            for (int u = warp; u < nunits; u += kTcIssuers) {
                uint32_t a_lo = dz_lo0;
                if (u < KK) {
                    const int ky = u / K, kx = u - ky * K;
                    uint32_t x_lo = x_lo0 + (uint32_t)(ky * A.Wp + kx);
                    const uint32_t col = tmem + (uint32_t)(u * A.ncols);
                    for (int ks = 0; ks < nk; ++ks) {
                        mma_bf16(col, desc64(a_hi, a_lo), desc64(x_hi, x_lo), idesc, (i | ks) != 0);
                        a_lo += 16; x_lo += 16;
                    }
                } else {
                    const uint32_t col = tmem + (uint32_t)(KK * A.ncols);
                    for (int ks = 0; ks < nk; ++ks) { mma_bf16(col, desc64(a_hi, a_lo), ones_d, idb, (i | ks) != 0); a_lo += 16; }
                }
            }
            mma_commit(smem_u32(&H->empty[s]));
        }
        mma_commit(smem_u32(&H->done));
    }
    __syncwarp();
    const bool have = nb > 0 && wait(&H->done, 0, 256);        // (asleep between polls: the issuers share the schedulers)
    if (!have && nb > 0) mbar_wait(smem_u32(&H->done), 0, 200000000ll);   // gave up: the MMAs under way still end first
    fence_after_sync();

    // tensor memory -> this share's partial set; lane quarter q holds rows 32q.. (Ms = 128) or rows 16q.. in its
    // first 16 lanes (Ms = 64).  The slices of the blocks are disjoint: plain stores.
    const int q = warp & 3, half = warp >> 2;
    const int row = A.Ms == 128 ? q * 32 + lane : q * 16 + lane;
    const bool row_ok = (A.Ms == 128 || lane < 16) && slice * A.Ms + row < A.cout16;
    const int co = slice * A.Ms + row;
    float* gset = A.partial + (size_t)share * A.set_floats + A.tgp_off;
    for (int u = 0; u < KK; ++u)
        for (int c0 = half * 16; c0 < cols; c0 += 32) {
            float v[16];
            if (have) tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(u * A.ncols + c0), v);
            else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = 0.f;
            }
            if (row_ok) {
                float* g = gset + ((size_t)u * A.cout16 + co) * A.cin16 + ci0 + c0;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    *reinterpret_cast<float4*>(g + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            }
        }
    if (bias && half == 0) {
        float v[16];
        if (have) tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(KK * A.ncols), v);
        else v[0] = 0.f;
        if (row_ok) gset[(size_t)KK * A.cout16 * A.cin16 + co] = v[0];
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)kTcTmemCols);
}

// ---------------------------------------------------------------------------------------------
// Convolution of a one-conv group over bands of rows (forward pass, and the input delta as the convolution of dz
// with the rotated filters).  A work item is a band of R rows x Cw columns of one image x a slice of Ns output
// channels: up to 512 / Ns accumulator blocks of 128 consecutive tile entries (pitch Wp = Cw + K - 1, so the entries
// of a block are pixels of consecutive rows with K - 1 discarded positions between them) stay in tensor memory
// while the input channels stream past in chunks: per chunk one tile of `kpc` 8-channel planes of the band (with
// its K - 1 halo rows, TMA tensor copies) and the filters of those channels for the slice (one bulk copy),
// through a ring of stages.  Window position (ky, kx) moves the A operand by ky * Wp + kx entries.  Against the
// fused sub-tile kernel, whose sub-tiles follow the tile grid (64 pixels a tile on the deepest maps) and which
// streams all filters of the layer once per 128 pixels, the filters read per pixel shrink by the number of
// accumulator blocks and the pixels per block no longer depend on the grid.
//
// Persistent blocks (one per SM) walk over the items; the warps have fixed roles: warps 0-7 read the accumulators
// back (bias, leaky ReLU, bf16 planes; with a fused 2x2 pool through a small staging area, 16 channels or more at
// a time, first maximum in window order, with the arg-max bytes the backward pass routes deltas by), lane 0 of
// warps 8-11 issues the MMAs (each for its own accumulator blocks), lane 0 of warp 12 issues the copies and runs
// ahead into the next item while the accumulators of the current one are read back.
// ---------------------------------------------------------------------------------------------
struct TcConvRowsArgs {
    alignas(64) unsigned char tmap_x[128];    // input planes (rows of 2 W eight-byte elements): box = Wp pixels x (R + K - 1) rows
    const __nv_bfloat16* w;                   // filters of the layer, [slice][chunk][window position][kpc][Ns][8]: the
                                              //   filters a block needs for one chunk are one contiguous run
    const float* bias;                        // cout floats, or null
    uint4* out;                               // output planes [N][cout16/8][OH][OW] (OH = H / 2 with the pool)
    unsigned long long* arg;                  // pool: arg-max bytes in the same arrangement
    int* error;
    int N, K, cin16, cout16, cout, H, W, pool;
    float slope;
    int Ns, slices;                           // output channels per item, number of slices
    int R, Wp, bands_img, nblk;               // rows per band, tile pitch, bands per image, accumulator blocks of a full band
    int ncc, Cw;                              // column chunks per row band and their width (even with the pool; Wp = Cw + K - 1)
    int kpc;                                  // 8-channel planes per chunk (3x3: 2, or 4 with narrow slices; 1x1: up to 8)
    int x_plane, stage_bytes, stages;
    int items;                                // N * bands_img * slices
    int pool_planes;                          // pool: 8-channel planes the staging area holds (even)
    // input delta only: when the layer below is a one-conv group too, the delta goes straight into ITS dz planes (`out`;
    // at twice the resolution if it ends with a pool): prev_y = that layer's saved output (= this conv's output shape),
    // prev_arg = its pool's arg-max bytes or null, prev_slope = its leaky slope.  prev_y null: plain delta planes.
    const uint4* prev_y; const unsigned long long* prev_arg; float prev_slope;
    int nbuf;                                 // accumulator buffers (2: items of at most 256 columns alternate between the halves
                                              //   of the tensor memory, so the MMAs of one run while the other is read back)
};

constexpr int kTcConvMaxStages = 4;
constexpr int kTcConvEpiWarps = 16;           // four per lane quarter of the tensor memory
constexpr int kTcConvEpiThreads = kTcConvEpiWarps * 32;
constexpr int kTcConvThreads = (kTcConvEpiWarps + kTcIssuers + 1) * 32;

__global__ void __launch_bounds__(kTcConvThreads, 1) conv_tc_rows_kernel(const __grid_constant__ TcConvRowsArgs A)
{
    using namespace tc;
    extern __shared__ __align__(1024) unsigned char cv_smem[];
    struct Hdr {
        unsigned long long full[kTcConvMaxStages], empty[kTcConvMaxStages];
        unsigned long long done[2];     // the MMAs of an item have completed (one commit per issuer), per accumulator buffer
        unsigned long long tfree[2];    // its accumulators have been read back (one arrival per epilogue warp)
        unsigned long long drain;       // all MMAs of the block have completed
        uint32_t tmem_base;
        volatile int failed;
        volatile int epi_stop[2];       // the epilogue warps' common view of `failed` (they meet at named barriers), items in turn
        float bias[128];
    };
    static_assert(sizeof(Hdr) <= kTcFgHeader, "header does not fit");
    Hdr* H = reinterpret_cast<Hdr*>(cv_smem);
    unsigned char* stages = cv_smem + kTcFgHeader;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int K = A.K, KK = K * K;
    const int kplanes = A.cin16 / 8, nchunks = (kplanes + A.kpc - 1) / A.kpc;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcConvMaxStages; ++s) { mbar_init(smem_u32(&H->full[s]), 1); mbar_init(smem_u32(&H->empty[s]), kTcIssuers); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&H->done[i]), kTcIssuers); mbar_init(smem_u32(&H->tfree[i]), kTcConvEpiWarps); }
        mbar_init(smem_u32(&H->drain), kTcIssuers);
        H->failed = 0;
        fence_mbar_init();
    }
    if (warp == 0) { __syncwarp(); tmem_alloc(smem_u32(&H->tmem_base), (uint32_t)kTcTmemCols); }
    tcd::zero_bytes(stages, (size_t)A.stages * A.stage_bytes);       // what the copies never write is read as zeros
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = H->tmem_base;

    auto wait = [&](unsigned long long* bar, uint32_t parity, unsigned sleep_ns = 0) {
        if (H->failed) return false;
        if (mbar_wait(smem_u32(bar), parity, kWaitLimitCycles, sleep_ns)) return true;
        H->failed = 1;
        atomicExch(A.error, 1);
        return false;
    };
    if ((smem_u32(cv_smem) & 127u) != 0) {                  // tensor copies want 128-byte aligned destinations
        if (threadIdx.x == 0) { H->failed = 1; atomicExch(A.error, 1); }
        __syncthreads();
    }
    // item -> (slice, image, band origin); every role walks the same sequence of items
    struct Item { int slice, n, y0, x0, rows, cw, co0, cols, nblk; };
    auto item_of = [&](int it) {
        Item I;
        I.slice = it % A.slices;
        const int band = it / A.slices;
        I.n = band / A.bands_img;
        const int bi = band - I.n * A.bands_img;
        I.y0 = (bi / A.ncc) * A.R; I.x0 = (bi % A.ncc) * A.Cw;
        I.rows = min(A.R, A.H - I.y0); I.cw = min(A.Cw, A.W - I.x0);
        I.co0 = I.slice * A.Ns; I.cols = min(A.Ns, A.cout16 - I.co0);
        I.nblk = (I.rows * A.Wp + 127) >> 7;
        return I;
    };
    const uint32_t w_tap = (uint32_t)A.kpc * (uint32_t)A.Ns * 16u;                      // filter bytes of one window position
    const uint32_t w_chunk = (uint32_t)KK * w_tap;

    if (warp == kTcConvEpiWarps + kTcIssuers) {
        if (lane == 0) {
            // producer
            int issued[kTcConvMaxStages] = {0, 0, 0, 0};
            uint32_t g = 0;                                                             // chunks issued so far
            for (int it = blockIdx.x; it < A.items && !H->failed; it += gridDim.x) {
                const Item I = item_of(it);
                for (int c = 0; c < nchunks; ++c, ++g) {
                    const int s = (int)(g % (uint32_t)A.stages);
                    if (!wait(&H->empty[s], ((g / (uint32_t)A.stages) & 1u) ^ 1u)) break;
                    const int kp0 = c * A.kpc, np = min(A.kpc, kplanes - kp0);
                    unsigned char* xs = stages + (size_t)s * A.stage_bytes;
                    unsigned char* ws = xs + (size_t)A.kpc * A.x_plane;
                    const uint32_t bar = smem_u32(&H->full[s]);
                    mbar_expect_tx(bar, (uint32_t)(np * (A.R + K - 1) * A.Wp) * 16u + w_chunk);
                    for (int pl = 0; pl < np; ++pl)
                        tma_load_3d(smem_u32(xs + (size_t)pl * A.x_plane), A.tmap_x, 2 * (I.x0 - K / 2), I.y0 - K / 2,
                                    I.n * kplanes + kp0 + pl, bar);
                    bulk_g2s(smem_u32(ws), A.w + ((size_t)I.slice * nchunks + c) * (w_chunk / 2), w_chunk, bar);
                    ++issued[s];
                }
            }
            if (H->failed)       // gave up somewhere: let the copies already under way land before the block leaves
                for (int s = 0; s < A.stages; ++s)
                    if (issued[s] > 0) mbar_wait(smem_u32(&H->full[s]), (uint32_t)(issued[s] - 1) & 1u, 200000000ll);
        }
    } else if (warp >= kTcConvEpiWarps) {
        if (lane == 0) {
            // MMA issue: every issuer takes every kTcIssuers-th accumulator block; K-major operands: 8 pixels (or 8
            // output channels) x 16 bytes per core matrix, the next 8 rows 128 bytes on, the next 8 channels one plane on
            const int iw = warp - kTcConvEpiWarps;
            const uint32_t a_hi = desc_hi(128), b_hi = desc_hi(128);
            const uint32_t xstep = 2u * ((uint32_t)A.x_plane >> 4), wstep = 2u * (uint32_t)A.Ns;   // one K step, 16-byte units
            const uint32_t w_tap16 = w_tap >> 4;
            uint32_t g = 0, k = 0;
            for (int it = blockIdx.x; it < A.items && !H->failed; it += gridDim.x, ++k) {
                const Item I = item_of(it);
                const uint32_t idesc = make_idesc(128, I.cols, false, false);
                const uint32_t buf = k % (uint32_t)A.nbuf, use = k / (uint32_t)A.nbuf;  // accumulator buffer and how often it was used
                if (use > 0 && !wait(&H->tfree[buf], (use - 1) & 1u)) break;            // its accumulators have been read back
                fence_after_sync();
                for (int c = 0; c < nchunks; ++c, ++g) {
                    const int s = (int)(g % (uint32_t)A.stages);
                    if (!wait(&H->full[s], (g / (uint32_t)A.stages) & 1u)) break;
                    fence_after_sync();
                    const int nks = min(A.kpc, kplanes - c * A.kpc) >> 1;
                    const uint32_t xaddr = smem_u32(stages + (size_t)s * A.stage_bytes), waddr = xaddr + (uint32_t)(A.kpc * A.x_plane);
                    const uint32_t b_lo0 = desc_lo(waddr, (uint32_t)A.Ns * 16u);
                    // (the thread that issues is the bottleneck of a narrow MMA: descriptors advance by adds only)
                    for (int b = iw; b < I.nblk; b += kTcIssuers) {
                        const uint32_t tcol = tmem + buf * 256u + (uint32_t)(b * A.Ns);
                        const uint32_t a0 = desc_lo(xaddr + (uint32_t)b * 2048u, (uint32_t)A.x_plane);
                        if (K == 3) {
                            // nine MMAs per K step, one per window position, written out: the issuing thread runs a few dozen
                            // instructions per MMA if it has to loop, and then it, not the tensor core, sets the pace
                            // (measured: an MMA every 100 cycles with the loops, every 40-64 with straight-line code)
                            const uint32_t wp = (uint32_t)A.Wp;
                            uint32_t a = a0, w0 = b_lo0;
                            for (int ks = 0; ks < nks; ++ks, a += xstep, w0 += wstep) {
                                mma_bf16(tcol, desc64(a_hi, a), desc64(b_hi, w0), idesc, (c | ks) != 0);
                                mma_bf16(tcol, desc64(a_hi, a + 1), desc64(b_hi, w0 + w_tap16), idesc, true);
                                mma_bf16(tcol, desc64(a_hi, a + 2), desc64(b_hi, w0 + 2 * w_tap16), idesc, true);
                                mma_bf16(tcol, desc64(a_hi, a + wp), desc64(b_hi, w0 + 3 * w_tap16), idesc, true);
                                mma_bf16(tcol, desc64(a_hi, a + wp + 1), desc64(b_hi, w0 + 4 * w_tap16), idesc, true);
                                mma_bf16(tcol, desc64(a_hi, a + wp + 2), desc64(b_hi, w0 + 5 * w_tap16), idesc, true);
                                mma_bf16(tcol, desc64(a_hi, a + 2 * wp), desc64(b_hi, w0 + 6 * w_tap16), idesc, true);
                                mma_bf16(tcol, desc64(a_hi, a + 2 * wp + 1), desc64(b_hi, w0 + 7 * w_tap16), idesc, true);
                                mma_bf16(tcol, desc64(a_hi, a + 2 * wp + 2), desc64(b_hi, w0 + 8 * w_tap16), idesc, true);
                            }
                        } else {
                            uint32_t a_lo = a0, b_lo = b_lo0;
                            bool acc = c > 0;
                            for (int ks = 0; ks < nks; ++ks) {
                                mma_bf16(tcol, desc64(a_hi, a_lo), desc64(b_hi, b_lo), idesc, acc);
                                acc = true; a_lo += xstep; b_lo += wstep;
                            }
                        }
                    }
                    mma_commit(smem_u32(&H->empty[s]));
                }
                mma_commit(smem_u32(&H->done[buf]));
            }
            mma_commit(smem_u32(&H->drain));
        }
    } else {
        // epilogue warps: lane quarter q = warp % 4 of every accumulator block; the two warps of a quarter take
        // alternate blocks
        const int q = warp & 3, part = warp >> 2;                  // the warps of a quarter share its (block, 16 columns) units
        constexpr int kParts = kTcConvEpiWarps / 4;
        const int oplanes = A.cout16 / 8;
        const float slope = A.slope;
        const int E = A.nblk * 128;                                   // entries per plane of the pooling layout
        uint4* S = reinterpret_cast<uint4*>(stages + (size_t)A.stages * A.stage_bytes);
        const int et = threadIdx.x;                                   // 0 .. kTcConvEpiThreads - 1
        uint32_t k = 0;
        // one slice of output channels: its bias is fetched once, and an item costs the epilogue warps one barrier (the
        // stop word of item k is written before that barrier and read behind it; its slot is written again two items
        // on, behind the barrier of the item between, at which every thread has read it)
        const bool one_slice = A.slices == 1;
        if (one_slice)
            for (int c = et; c < A.Ns; c += kTcConvEpiThreads) H->bias[c] = (A.bias && c < A.cout) ? __ldg(A.bias + c) : 0.f;
        for (int it = blockIdx.x; it < A.items; it += gridDim.x, ++k) {
            const Item I = item_of(it);
            if (!one_slice) {
                asm volatile("bar.sync 1, %0;" :: "n"(kTcConvEpiThreads) : "memory");        // every warp is through with the bias of the item before
                for (int c = et; c < A.Ns; c += kTcConvEpiThreads) H->bias[c] = (A.bias && I.co0 + c < A.cout) ? __ldg(A.bias + I.co0 + c) : 0.f;
            }
            if (et == 0) H->epi_stop[k & 1u] = H->failed;
            asm volatile("bar.sync 1, %0;" :: "n"(kTcConvEpiThreads) : "memory");
            if (H->epi_stop[k & 1u]) break;                           // the same answer for all epilogue threads: they leave together
            const uint32_t buf = k % (uint32_t)A.nbuf, use = k / (uint32_t)A.nbuf;
            const uint32_t tbuf = tmem + buf * 256u;
            wait(&H->done[buf], use & 1u, 128);                       // asleep between polls; (ran out: the item is written from
                                                                      // whatever is there; the error word is set)
            fence_after_sync();
            if (!A.pool) {
                const int nc = I.cols >> 4, nunits = I.nblk * nc;
                const size_t gstep = (size_t)A.H * A.W;
                // where unit u (accumulator block b, channels c0 .. c0 + 15) of this thread lies in the output planes
                auto place = [&](int u, int& b, int& c0, size_t& g0) {
                    b = u / nc; c0 = (u - b * nc) << 4;
                    const int p = b * 128 + q * 32 + lane;
                    const int r = p / A.Wp, c = p - r * A.Wp;
                    g0 = (((size_t)I.n * oplanes + ((I.co0 + c0) >> 3)) * A.H + I.y0 + r) * A.W + I.x0 + c;
                    return r < I.rows && c < I.cw;
                };
                for (int u = part; u < nunits; u += kParts) {
                    int b, c0; size_t g0;
                    const bool valid = place(u, b, c0, g0);
                    // what the fused dz step reads of the layer below is requested before the accumulators, so that the
                    // latencies overlap (requested a whole unit ahead, even for the launches through a pool only, the
                    // kernel was measured slower)
                    uint4 yq[2] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
                    unsigned long long amq[2] = {0ull, 0ull};
                    if (A.prev_y && valid) {
                        yq[0] = __ldg(A.prev_y + g0); yq[1] = __ldg(A.prev_y + g0 + gstep);
                        if (A.prev_arg) { amq[0] = __ldg(A.prev_arg + g0); amq[1] = __ldg(A.prev_arg + g0 + gstep); }
                    }
                    float v[16];
                    tmem_ld16(tbuf + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * A.Ns + c0), v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) { const float z = v[j] + H->bias[c0 + j]; v[j] = z > 0.f ? z : slope * z; }
                    if (valid && !A.prev_y) {
                        A.out[g0] = tcd::pack8(v);
                        A.out[g0 + gstep] = tcd::pack8(v + 8);
                    } else if (valid) {
                        // input delta straight into the dz planes of the layer below: rounded as a stored delta
                        // would be, times the derivative of that layer's activation, through its pool's arg-max
                        const int p = b * 128 + q * 32 + lane;
                        const int r = p / A.Wp, c = p - r * A.Wp;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            float d[8], yv[8];
                            tcd::unpack8(tcd::pack8(v + 8 * h), d);
                            tcd::unpack8(yq[h], yv);
#pragma unroll
                            for (int j = 0; j < 8; ++j) d[j] *= yv[j] > 0.f ? 1.f : A.prev_slope;
                            const uint4 dq = tcd::pack8(d);
                            if (!A.prev_arg) { A.out[g0 + h * gstep] = dq; continue; }
                            // the four members of every channel's pool window: the delta where the arg-max byte names the
                            // member, zero elsewhere (byte masks widened to the bf16 halves)
                            const uint32_t alo = (uint32_t)amq[h] & 0x03030303u, ahi = (uint32_t)(amq[h] >> 32) & 0x03030303u;
                            const int W2 = 2 * A.W;
                            uint4* o2 = A.out + (((size_t)I.n * oplanes + ((I.co0 + c0) >> 3) + h) * (2 * A.H) + 2 * (I.y0 + r)) * W2 + 2 * (I.x0 + c);
#pragma unroll
                            for (int w = 0; w < 4; ++w) {
                                const uint32_t ml = __vcmpeq4(alo, (uint32_t)w * 0x01010101u), mh = __vcmpeq4(ahi, (uint32_t)w * 0x01010101u);
                                o2[(w >> 1) * W2 + (w & 1)] = make_uint4(dq.x & __byte_perm(ml, 0u, 0x1100), dq.y & __byte_perm(ml, 0u, 0x3322),
                                                                         dq.z & __byte_perm(mh, 0u, 0x1100), dq.w & __byte_perm(mh, 0u, 0x3322));
                            }
                        }
                    }
                }
            } else {
                const int OH = A.H / 2, OW = A.W / 2, prs = I.rows / 2, pcs = I.cw / 2;
                for (int pl0 = 0; pl0 < (I.cols >> 3); pl0 += A.pool_planes) {
                    const int npl = min(A.pool_planes, (I.cols >> 3) - pl0);
                    // the band as it would be stored, planes pl0 .. pl0 + npl - 1
                    const int nc = npl >> 1;
                    for (int u = part; u < I.nblk * nc; u += kParts) {
                        const int b = u / nc, c0 = pl0 * 8 + ((u - b * nc) << 4);
                        const int p = b * 128 + q * 32 + lane;
                        {
                            float v[16];
                            tmem_ld16(tbuf + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * A.Ns + c0), v);
#pragma unroll
                            for (int j = 0; j < 16; ++j) { const float z = v[j] + H->bias[c0 + j]; v[j] = z > 0.f ? z : slope * z; }
                            S[(size_t)((c0 >> 3) - pl0) * E + p] = tcd::pack8(v);
                            S[(size_t)((c0 >> 3) - pl0 + 1) * E + p] = tcd::pack8(v + 8);
                        }
                    }
                    asm volatile("bar.sync 1, %0;" :: "n"(kTcConvEpiThreads) : "memory");
                    // one thread per pooled pixel and plane; the four window members are compared as stored, two
                    // channels (a bf16 pair) per instruction: a later member wins only if it is greater
                    const int npix = prs * pcs, total = npl * npix;
                    for (int e = et; e < total; e += kTcConvEpiThreads) {
                        const int pl = e / npix, pix = e - pl * npix, pr = pix / pcs, pc = pix - pr * pcs;
                        const uint4* s4 = S + (size_t)pl * E + (size_t)(2 * pr) * A.Wp + 2 * pc;
                        const uint4 m0 = s4[0], m1 = s4[1], m2 = s4[A.Wp], m3 = s4[A.Wp + 1];
                        const uint32_t* w0 = &m0.x; const uint32_t* w1 = &m1.x; const uint32_t* w2 = &m2.x; const uint32_t* w3 = &m3.x;
                        uint32_t best[4], code[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t m = w0[j], a = 0u;
                            const uint32_t cand[3] = {w1[j], w2[j], w3[j]};
#pragma unroll
                            for (int w = 0; w < 3; ++w) {
                                const uint32_t gt = __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&cand[w]),
                                                                *reinterpret_cast<const __nv_bfloat162*>(&m));
                                m = (cand[w] & gt) | (m & ~gt);
                                a = (((uint32_t)(w + 1) * 0x00010001u) & gt) | (a & ~gt);
                            }
                            best[j] = m; code[j] = a;
                        }
                        // arg-max bytes: channel 2j in the low half of code[j], channel 2j + 1 in the high half
                        const unsigned long long am = (unsigned long long)__byte_perm(code[0], code[1], 0x6420) |
                                                      ((unsigned long long)__byte_perm(code[2], code[3], 0x6420) << 32);
                        const size_t gi = (((size_t)I.n * oplanes + (I.co0 >> 3) + pl0 + pl) * OH + (I.y0 >> 1) + pr) * OW + (I.x0 >> 1) + pc;
                        A.out[gi] = make_uint4(best[0], best[1], best[2], best[3]);
                        A.arg[gi] = am;
                    }
                    asm volatile("bar.sync 1, %0;" :: "n"(kTcConvEpiThreads) : "memory");    // the staging area is free for the next planes
                }
            }
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&H->tfree[buf]));
        }
    }
    __syncthreads();
    // every MMA of the block has completed before the tensor memory goes back (also when a wait gave up)
    if (warp == 0) {
        if (lane == 0) mbar_wait(smem_u32(&H->drain), 0, 200000000ll);
        __syncwarp();
        fence_after_sync();
        tmem_dealloc(tmem, (uint32_t)kTcTmemCols);
    }
}

}  // namespace ftp
