// Fused tile-stack kernels of the bf16 path: every convolution is an implicit GEMM on the
// tcgen05 tensor cores with fp32 accumulators in tensor memory.
//
// A map tile lives in shared memory as 8-channel planes [channel/8][row][col][8] bf16 (16 bytes per
// pixel and plane; channel counts are padded to 16 with zeros).  For a K x K convolution the A
// operand of one MMA is a block of 16 rows x 8 columns of output pixels: the window position
// (ky, kx) only moves the start address of the block inside the input tile, so no im2col copy is
// ever made.  The B operand (filters of one window position, [cout][cin] K-major) is streamed from
// global memory through a small ring of stages with bulk (TMA) copies.  The saved maps in global
// memory use the same plane arrangement, [n][C16/8][H][W][8] bf16.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "plan.hpp"
#include "tc.cuh"

namespace ftp {

struct TcGroupArgs {
    int n_ops, R, Q, N;
    OpDesc op[kMaxOps];
    const void* map[kMaxOps + 1];        // map[0] = group input (bf16 planes; fp32 NCHW when in_f32), map[m] = output of op m-1
    __nv_bfloat16* map_out[kMaxOps + 1]; // forward: writable aliases of map[1..]
    unsigned char* arg[kMaxOps];         // arg-max bytes of op i's pooled output map (fused conv+pool), same arrangement
    int in_f32, in_C;                    // the group input is the network input X_1 (fp32 NCHW with in_C channels)
    const int *yspan, *xspan, *ycell, *xcell;
    const __nv_bfloat16* wpk;            // packed filters (forward or rotated arrangement)
    const float* params;
    int* error;                          // set to 1 when a bounded wait ran out
    // Tensor maps (128 bytes each, CUtensorMap) of the bf16 maps that tiles are copied from by TMA: [0] the group
    // input (forward), [i] the input map of op i (backward); use_tma bit i says whether entry i is valid.
    // A map is seen as the 4-dimensional tensor [image x plane][row][column][8 channels]; a box is one plane of
    // a tile (rows x columns of the tile's pitch), positions outside the map arrive as zeros (the padding).
    alignas(64) unsigned char tmap[kMaxOps][128];
    unsigned use_tma;
    // backward only
    const void*  dmap_out;               // delta at the group's output map: fp32 NCHW (from the caller / the loss), or
    int          dmap_planes;            //   bf16 planes written by halo_sum_planes_kernel (dmap_planes = 1)
    float*       scratch;                // per-sub-tile deltas at the group input: fp32 [c][h][w] blocks for the first
                                         //   group (network input), else fp32 [c/8][h][w][8] blocks of the padded channels
    const int *yoff, *xoff, *ytile, *xtile;
    float*       partial;
    long long    set_floats;
    int need_dx;
};

namespace tcd {

using namespace tc;

// Fixed part of the dynamic shared memory (kTcHeader bytes), then the weight ring, then the tiles.
struct Header {
    int hdr[(kMaxOps + 1) * 8];                  // spans / cells of the current sub-tile
    unsigned long long full[kTcMaxStages];          // weight stage filled (transaction bytes)
    unsigned long long empty[kTcMaxStages];         // weight stage consumed (tcgen05.commit)
    unsigned long long done;                     // all MMAs of a pass completed
    unsigned long long tile_bar;                 // a tile copied by TMA has arrived (transaction bytes)
    uint32_t tmem_base;
    int stage_mask, stage_shift;                 // filter ring: stages - 1 and log2(stages)
    int tmem_cols;                               // columns this block allocated (512, or 256 with two blocks per SM)
    volatile int failed;                         // a wait ran out: skip every later wait
    int dw_nw, dw_nbias;                         // entries of dw_unit / dw_bias in the current pass
    __align__(16) __nv_bfloat16 ones[64];        // one core matrix of 1.0: operand of the bias-gradient contraction
    __align__(16) uint4 dw_unit[kTcMaxUnits + 4];  // filter gradient: MMAs of the current pass {a_lo, x_lo, idesc, column}
    uint2 dw_bias[kTcMaxUnits];                  //                  bias MMAs {a_lo, column}
    float bias[kTcTmemCols];
};
static_assert(sizeof(Header) <= kTcHeader, "header does not fit");

// Per-thread view of the pipeline state.  The producer thread, the MMA thread and the epilogue
// threads each advance the counters they use; all of them see the same sequence of passes and stages.
struct Pipe {
    Header* h;
    uint32_t ring;          // shared-memory address of the weight ring
    uint32_t stages_done;   // weight stages produced / consumed so far by this thread's role
    uint32_t passes_done;   // passes completed so far
    uint32_t tiles_done;    // tiles received by TMA so far
    int* error;
};

__device__ __forceinline__ bool wait_or_fail(Pipe& p, unsigned long long* bar, uint32_t parity, unsigned sleep_ns = 0)
{
    if (p.h->failed) return false;
    if (mbar_wait(smem_u32(bar), parity, kWaitLimitCycles, sleep_ns)) return true;
    p.h->failed = 1;
    if (p.error) atomicExch(p.error, 1);
    return false;
}

// Exercises the give-up path of the bounded waits on its own: one thread sets up a barrier that nothing ever
// arrives on and waits on it through the same routine as the tile kernels, with a limit of `limit_cycles`
// instead of seconds; the wait runs out, the error word is set and the kernel returns.
__global__ void wait_probe_kernel(int* error, long long limit_cycles)
{
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
        if (!mbar_wait(smem_u32(&bar), 0, limit_cycles)) atomicExch(error, 1);
    }
}

__device__ __forceinline__ uint4 pack8(const float* v)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
    uint4 r;
    r.x = *reinterpret_cast<uint32_t*>(&a); r.y = *reinterpret_cast<uint32_t*>(&b);
    r.z = *reinterpret_cast<uint32_t*>(&c); r.w = *reinterpret_cast<uint32_t*>(&d);
    return r;
}

__device__ __forceinline__ void unpack8(const uint4& r, float* v)
{
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 f = __bfloat1622float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
}

// Implicit-GEMM convolution on a shared-memory tile.
//   a_base  shared address such that output pixel (y, x) of the region reads tile entry
//           a_base + ((y + ky) * a_Wp + x + kx) * 16 of every plane for window position (ky, kx)
//   kplanes input channel planes (cin16 / 8), N output channels (cout16 <= 512)
//   w       packed filters [ky*K+kx][kplanes][N][8] bf16
//   rows x cols: extent of the output region; it is covered by blocks of 16 x 8 pixels
// The accumulator block of each pixel block takes N tensor-memory columns; as many blocks as fit are
// in flight per pass, and the filter stages are streamed once per pass.  After each pass every warp
// calls epi(by, bx, q, lane, c0, v[16]) for its lane quarter q and 16-channel chunks c0.
template <class Epi>
__device__ __forceinline__ void conv_mma(Pipe& p, uint32_t a_base, int a_Wp, uint32_t a_plane, int kplanes, int K,
                                         int N, const __nv_bfloat16* __restrict__ w, int rows, int cols, Epi epi)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nby = (rows + 15) >> 4, nbx = (cols + 7) >> 3, nblocks = nby * nbx;
    const int in_flight = p.h->tmem_cols / N;
    const int planes = K * K * kplanes;                               // even
    int spp = (kTcStageBytes / (N * 16)) & ~1;                        // planes per stage, even, >= 2
    if (spp > planes) spp = planes;
    const int nstages = (planes + spp - 1) / spp;
    const uint32_t plane_bytes = (uint32_t)N * 16;
    const uint32_t tmem = p.h->tmem_base;

    for (int b0 = 0; b0 < nblocks; b0 += in_flight) {
        const int nb = min(in_flight, nblocks - b0);
        if (warp == kTcIssuers && lane == 0) {
            // producer: one bulk copy per stage
            for (int s = 0; s < nstages; ++s) {
                const uint32_t q = p.stages_done + s, slot = q & (uint32_t)p.h->stage_mask, par = (q >> p.h->stage_shift) & 1;
                if (!wait_or_fail(p, &p.h->empty[slot], par ^ 1)) break;
                const int pl = min(spp, planes - s * spp);
                const uint32_t bytes = (uint32_t)pl * plane_bytes;
                mbar_expect_tx(smem_u32(&p.h->full[slot]), bytes);
                bulk_g2s(p.ring + slot * kTcStageBytes, w + (size_t)s * spp * N * 8, bytes, smem_u32(&p.h->full[slot]));
            }
        } else if (warp < kTcIssuers && lane == 0) {
            // MMA issue.  A single thread cannot keep the tensor core busy (an MMA of this size takes it
            // about 45 cycles, the thread needs well over 100 to prepare the next one), so lane 0 of the
            // first kTcIssuers warps each issue the MMAs of every kTcIssuers-th pixel block; their
            // accumulators are disjoint, so no order between the issuers is needed.  Descriptor halves
            // are advanced with adds only.
            const uint32_t a_hi = desc_hi((uint32_t)a_Wp * 16), b_hi = desc_hi(128);
            const uint32_t plane16 = a_plane >> 4, bplane16 = plane_bytes >> 4;
            const uint32_t idesc_full = make_idesc(128, min(N, 256), false, false);
            const uint32_t idesc_rest = N > 256 ? make_idesc(128, N - 256, false, false) : 0u;
            int gp0 = 0;                                            // first plane of the stage
            for (int s = 0; s < nstages; ++s) {
                const uint32_t q = p.stages_done + s, slot = q & (uint32_t)p.h->stage_mask, par = (q >> p.h->stage_shift) & 1;
                if (!wait_or_fail(p, &p.h->full[slot], par)) break;
                fence_after_sync();
                const int pl = min(spp, planes - gp0);
                const uint32_t b_lo0 = desc_lo(p.ring + slot * kTcStageBytes, plane_bytes);
                // window position and channel plane at which the stage starts (once per stage)
                const int tap0 = gp0 / kplanes, kc0 = gp0 - tap0 * kplanes, ky0 = tap0 / K, kx0 = tap0 - ky0 * K;
                const uint32_t off0 = (uint32_t)kc0 * plane16 + (uint32_t)(ky0 * a_Wp + kx0);
                for (int bi = warp; bi < nb; bi += kTcIssuers) {
                    const int b = b0 + bi, by = b / nbx, bx = b - by * nbx;
                    const uint32_t tcol = tmem + (uint32_t)(bi * N);
                    const uint32_t a_lo0 = desc_lo(a_base + (uint32_t)((by * 16) * a_Wp + bx * 8) * 16, a_plane);
                    uint32_t off = off0, b_lo = b_lo0;
                    int kc = kc0, kx = kx0;
                    bool acc = gp0 > 0;
                    for (int pp = 0; pp < pl; pp += 2) {
                        const uint64_t ad = desc64(a_hi, a_lo0 + off);
                        mma_bf16(tcol, ad, desc64(b_hi, b_lo), idesc_full, acc);
                        if (N > 256) mma_bf16(tcol + 256, ad, desc64(b_hi, b_lo + 256), idesc_rest, acc);
                        acc = true;
                        b_lo += 2 * bplane16;
                        kc += 2; off += 2 * plane16;
                        if (kc == kplanes) {                        // next window position
                            kc = 0; off -= (uint32_t)kplanes * plane16;
                            ++kx; ++off;
                            if (kx == K) { kx = 0; off += (uint32_t)(a_Wp - K); }
                        }
                    }
                }
                mma_commit(smem_u32(&p.h->empty[slot]));
                gp0 += pl;
            }
            mma_commit(smem_u32(&p.h->done));
        }
        p.stages_done += nstages;
        __syncwarp();
        wait_or_fail(p, &p.h->done, p.passes_done & 1, 128);   // every thread waits here: asleep between polls
        p.passes_done++;
        fence_after_sync();
        const int q = warp & 3;
        for (int bi = 0; bi < nb; ++bi) {
            const int b = b0 + bi, by = b / nbx, bx = b % nbx;
            for (int c0 = (warp >> 2) * 16; c0 < N; c0 += (int)(blockDim.x >> 7) * 16) {
                float v[16];
                tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(bi * N + c0), v);
                epi(by, bx, q, lane, c0, v);
            }
        }
        fence_before_sync();
        __syncthreads();          // accumulators are free again; tile writes of the epilogue are visible
        fence_after_sync();
    }
}

// A shared-memory tile: planes of Hp x Wp entries (16 bytes = 8 channels of one pixel) plus a tail.
struct Tile {
    unsigned char* base; int planes, Hp, Wp; uint32_t plane;      // plane = bytes between planes
    __device__ __forceinline__ uint4* at(int pl, int y, int x) const
    {
        return reinterpret_cast<uint4*>(base + (size_t)pl * plane + ((size_t)y * Wp + x) * 16);
    }
};
__device__ __forceinline__ Tile make_tile(unsigned char* tiles, int off, int planes, int Hp, int Wp)
{
    return Tile{tiles + off, planes, Hp, Wp, (uint32_t)tc_plane_bytes(Hp, Wp)};
}

// Load the header of sub-tile (r, q): spans and owned cells at every map of the group.
__device__ __forceinline__ void load_header(int* hdr, const TcGroupArgs& A, int r, int q, bool cells)
{
    for (int m = threadIdx.x; m <= A.n_ops; m += blockDim.x) {
        hdr[m * 8 + 0] = A.yspan[(m * A.R + r) * 2 + 0];
        hdr[m * 8 + 1] = A.yspan[(m * A.R + r) * 2 + 1];
        hdr[m * 8 + 2] = A.xspan[(m * A.Q + q) * 2 + 0];
        hdr[m * 8 + 3] = A.xspan[(m * A.Q + q) * 2 + 1];
        if (cells) {
            hdr[m * 8 + 4] = A.ycell[(m * A.R + r) * 2 + 0];
            hdr[m * 8 + 5] = A.ycell[(m * A.R + r) * 2 + 1];
            hdr[m * 8 + 6] = A.xcell[(m * A.Q + q) * 2 + 0];
            hdr[m * 8 + 7] = A.xcell[(m * A.Q + q) * 2 + 1];
        }
    }
}

// Fill rows [0, bh) x cols [0, fill_w) of a tile with the part of a global map that starts at map
// position (oy, ox): columns >= bw and positions outside the map are zero.
__device__ __forceinline__ void load_tile(const Tile& T, int bh, int bw, int fill_w, const void* __restrict__ src, bool f32,
                                          int C, int n, int H, int W, int oy, int ox)
{
    const int total = T.planes * bh * fill_w;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int xx = e % fill_w, t = e / fill_w, yy = t % bh, pl = t / bh;
        const int gy = oy + yy, gx = ox + xx;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (xx < bw && gy >= 0 && gy < H && gx >= 0 && gx < W) {
            if (f32) {
                float f[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int ch = pl * 8 + c;
                    f[c] = ch < C ? __ldg(static_cast<const float*>(src) + (((size_t)n * C + ch) * H + gy) * W + gx) : 0.f;
                }
                v = pack8(f);
            } else {
                v = __ldg(static_cast<const uint4*>(src) + (((size_t)n * T.planes + pl) * H + gy) * W + gx);
            }
        }
        *T.at(pl, yy, xx) = v;
    }
}

// The same fill by TMA for a map stored as bf16 planes: one box of Hp x Wp entries per plane, starting at map
// position (oy, ox) of image n (negative and beyond-the-edge positions arrive as zeros: the padding).  Columns
// beyond the sub-tile's own width then hold the map's neighbouring values instead of zeros; they only meet
// accumulator rows that are discarded, or zeros of the other operand, like the tile's tail.  One thread issues
// the copies; every thread waits (bounded) for the bytes to arrive.  All threads must make the call.
__device__ __forceinline__ void load_tile_tma(Pipe& p, const Tile& T, const void* tmap, int n, int oy, int ox)
{
    fence_async_smem();           // earlier writes of this block to the tile's area are ordered before the copies
    __syncthreads();
    const uint32_t bar = smem_u32(&p.h->tile_bar);
    if (threadIdx.x == 0) {
        mbar_expect_tx(bar, (uint32_t)T.planes * (uint32_t)(T.Hp * T.Wp) * 16u);
        for (int pl = 0; pl < T.planes; ++pl)
            tma_load_4d(smem_u32(T.base + (size_t)pl * T.plane), tmap, 0, ox, oy, n * T.planes + pl, bar);
    }
    wait_or_fail(p, &p.h->tile_bar, p.tiles_done & 1);
    p.tiles_done++;
}

// Zero every entry of rows [0, bh) x cols [0, bw) of a tile outside the rectangle [y0,y1] x [x0,x1].
__device__ __forceinline__ void zero_outside(const Tile& T, int bh, int bw, int y0, int y1, int x0, int x1)
{
    if (y0 <= 0 && x0 <= 0 && y1 >= bh - 1 && x1 >= bw - 1) return;
    const int total = T.planes * bh * bw;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int xx = e % bw, t = e / bw, yy = t % bh, pl = t / bh;
        if (yy < y0 || yy > y1 || xx < x0 || xx > x1) *T.at(pl, yy, xx) = make_uint4(0, 0, 0, 0);
    }
}

// Zero `bytes` (multiple of 16) of shared memory.
__device__ __forceinline__ void zero_bytes(unsigned char* p, size_t bytes)
{
    for (size_t e = (size_t)threadIdx.x * 16; e < bytes; e += (size_t)blockDim.x * 16)
        *reinterpret_cast<uint4*>(p + e) = make_uint4(0, 0, 0, 0);
}

__device__ __forceinline__ void setup(Header* h, Pipe& p, unsigned char* smem, int* error, size_t tile_bytes, int tmem_cols,
                                      int stages)
{
    if (threadIdx.x == 0) {
        h->tmem_cols = tmem_cols;
        h->stage_mask = stages - 1; h->stage_shift = stages == 4 ? 2 : 1;
        for (int s = 0; s < kTcMaxStages; ++s) { mbar_init(smem_u32(&h->full[s]), 1); mbar_init(smem_u32(&h->empty[s]), kTcIssuers); }
        mbar_init(smem_u32(&h->done), kTcIssuers);
        mbar_init(smem_u32(&h->tile_bar), 1);
        h->failed = 0;
        fence_mbar_init();
    }
    if (threadIdx.x < 32) { __syncwarp(); tmem_alloc(smem_u32(&h->tmem_base), (uint32_t)tmem_cols); }
    // every byte the tensor core may ever read is a finite bf16 from here on
    zero_bytes(smem + (kTcHeader + stages * kTcStageBytes), tile_bytes);
    for (int i = threadIdx.x; i < 64; i += blockDim.x) h->ones[i] = __float2bfloat16(1.0f);
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    p.h = h; p.ring = smem_u32(smem + kTcHeader); p.stages_done = 0; p.passes_done = 0; p.tiles_done = 0; p.error = error;
}

__device__ __forceinline__ void teardown(Header* h)
{
    fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(h->tmem_base, (uint32_t)h->tmem_cols);
}

// Partial filter gradient of one sub-tile on the tensor core (Section 4.1: the feature-map tile
// convolved with the delta tile): for every window position t = (ky, kx)
//   G_t[co][ci] = sum over pixels p of dz[p][co] * x[p + ky * Wp + kx][ci],
// a GEMM whose contraction runs over the pixels.  Both tiles have the same pitch Wp, so one run of
// 16 consecutive tile entries is one K step for both operands (MN-major: 8 pixels x 8 channels per
// core matrix); the zero apron and tail of dz make the entries between the rows of the region and
// after its end contribute nothing.  The bias gradient is the same contraction against a tile of
// ones.  Accumulators ("units"): per 64- or 128-channel slice of cout one unit of N = cin16 columns
// per window position and 16 columns for the bias; as many units as fit in tensor memory per pass.
// With at most 8 input channels (the first layer) the K window positions of one filter row share a
// unit instead: N-chunk j of the x operand is the same plane moved by j pixels (stride 16 bytes),
// so one MMA yields G for kx = 0..K-1 and the layer needs K + 1 MMAs per K step instead of K*K + 1
// (an MMA costs the tensor core about 45 cycles however narrow it is).
// The result is added to (first: stored into) this block's partial set, arranged per layer as
// [t][cout16][cin16] followed by [cout16] bias entries.
__device__ __forceinline__ void filter_grad_mma(Pipe& p, uint32_t dz_run /*address of the region's first pixel*/,
                                                uint32_t dz_plane, uint32_t x_base, uint32_t x_plane, int Wp, int K,
                                                int cout16, int cin16, int cin, int run /*entries from first to last pixel*/,
                                                float* __restrict__ gset, bool first)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KK = K * K;
    const int Ms = cout16 <= 64 ? 64 : 128;
    const int nslices = cout16 <= 64 ? 1 : (cout16 + 127) / 128;
    const bool folded = cin <= 8;
    const int T = folded ? K : KK;                       // window units per slice
    const int ucols = folded ? (8 * K + 15) / 16 * 16 : cin16;
    const int nunits = nslices * (T + 1);
    const int nk = (run + 15) >> 4;
    const uint32_t tmem = p.h->tmem_base;
    Header* H = p.h;

    int u0 = 0;
    while (u0 < nunits) {
        // units of this pass: as many as fit in the tensor-memory columns
        int u1 = u0, cols = 0;
        while (u1 < nunits && u1 - u0 < kTcMaxUnits) {
            const int c = (u1 % (T + 1)) == T ? 16 : ucols;
            if (cols + c > H->tmem_cols) break;
            cols += c; ++u1;
        }
        const uint32_t a_hi = desc_hi(dz_plane);
        const uint32_t x_hi = desc_hi(folded ? 16u : x_plane);
        if (warp == 0 && lane == 0) {
            // Table of this pass's MMAs (operand descriptor halves, instruction descriptor, accumulator
            // column), built once; the K loops below then only add the step to the descriptors.
            const uint32_t a_lo0 = desc_lo(dz_run, 128), x_lo0 = desc_lo(x_base, 128);
            const uint32_t slice16 = 16u * (dz_plane >> 4), xhalf16 = 32u * (x_plane >> 4);
            const uint32_t id0 = make_idesc(Ms, min(ucols, 256), true, true);
            const uint32_t id1 = ucols > 256 ? make_idesc(Ms, ucols - 256, true, true) : 0u;
            int nw = 0, nbias = 0;
            const int s0 = u0 / (T + 1);
            int t = u0 - s0 * (T + 1), ky = folded ? t : t / K, kx = folded ? 0 : t - ky * K;
            uint32_t a_lo = a_lo0 + (uint32_t)s0 * slice16, col = tmem;
            for (int u = u0; u < u1; ++u) {
                if (t == T) {
                    H->dw_bias[nbias++] = make_uint2(a_lo, col);
                    col += 16; t = 0; ky = 0; kx = 0; a_lo += slice16;
                } else {
                    const uint32_t x_lo = x_lo0 + (uint32_t)(ky * Wp + kx);
                    H->dw_unit[nw] = make_uint4(a_lo, x_lo, id0, col); ++nw;
                    if (ucols > 256) { H->dw_unit[nw] = make_uint4(a_lo, x_lo + xhalf16, id1, col + 256); ++nw; }
                    col += (uint32_t)ucols; ++t;
                    if (folded) ++ky; else if (++kx == K) { kx = 0; ++ky; }
                }
            }
            H->dw_nw = nw; H->dw_nbias = nbias;
        }
        __syncthreads();
        if (warp < kTcIssuers && lane == 0) {
            // every issuer takes every kTcIssuers-th accumulator of the pass (see conv_mma)
            const int nw = H->dw_nw, nbias = H->dw_nbias;
            const uint32_t idb = make_idesc(Ms, 16, true, true);
            const uint64_t ones_d = make_desc(smem_u32(H->ones), 0, 0);
            for (int e = warp; e < nw; e += kTcIssuers) {
                const uint4 d = H->dw_unit[e];
                uint32_t a_lo = d.x, x_lo = d.y;
                for (int ks = 0; ks < nk; ++ks) {
                    mma_bf16(d.w, desc64(a_hi, a_lo), desc64(x_hi, x_lo), d.z, ks > 0);
                    a_lo += 16; x_lo += 16;
                }
            }
            for (int e = warp; e < nbias; e += kTcIssuers) {
                const uint2 d = H->dw_bias[e];
                uint32_t a_lo = d.x;
                for (int ks = 0; ks < nk; ++ks) { mma_bf16(d.y, desc64(a_hi, a_lo), ones_d, idb, ks > 0); a_lo += 16; }
            }
            mma_commit(smem_u32(&p.h->done));
        }
        __syncwarp();
        wait_or_fail(p, &p.h->done, p.passes_done & 1, 128);   // every thread waits here: asleep between polls
        p.passes_done++;
        fence_after_sync();
        // flush: lane quarter q holds rows 32q.. (M = 128) or rows 16q..16q+15 in its first 16 lanes (M = 64)
        const int q = warp & 3;
        const int row = Ms == 128 ? q * 32 + lane : q * 16 + lane;
        const bool row_ok = Ms == 128 || lane < 16;
        int col = 0;
        for (int u = u0; u < u1; ++u) {
            const int slice = u / (T + 1), t = u % (T + 1);
            const int co = slice * 128 + row;
            const int ncols = t == T ? 16 : ucols;
            for (int c0 = (warp >> 2) * 16; c0 < ncols; c0 += (int)(blockDim.x >> 7) * 16) {
                float v[16];
                tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(col + c0), v);
                if (row_ok && co < cout16) {
                    if (t == T) {
                        float* g = gset + (size_t)KK * cout16 * cin16 + co;
                        if (first) *g = v[0]; else atomicAdd(g, v[0]);
                    } else if (folded) {
                        // columns c0 .. c0+15 of filter row t: window columns kx = c0/8 and c0/8 + 1, channels 0..7
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int kx = (c0 >> 3) + h;
                            if (kx < K) {
                                float* g = gset + ((size_t)(t * K + kx) * cout16 + co) * cin16;
#pragma unroll
                                for (int j = 0; j < 2; ++j) {
                                    const float* w4 = v + 8 * h + 4 * j;
                                    if (first) *reinterpret_cast<float4*>(g + 4 * j) = make_float4(w4[0], w4[1], w4[2], w4[3]);
                                    else red_add_v4(g + 4 * j, w4[0], w4[1], w4[2], w4[3]);
                                }
                            }
                        }
                    } else {
                        float* g = gset + ((size_t)t * cout16 + co) * cin16 + c0;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (first) *reinterpret_cast<float4*>(g + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                            else red_add_v4(g + 4 * j, v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        }
                    }
                }
            }
            col += ncols;
        }
        fence_before_sync();
        __syncthreads();
        fence_after_sync();
        u0 = u1;
    }
}

}  // namespace tcd

// ---------------------------------------------------------------------------------------------
// Fused forward of one group, bf16: persistent blocks walk over the (image, sub-tile) stacks.
// ---------------------------------------------------------------------------------------------
template <int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 2 : 1) fwd_group_tc_kernel(const __grid_constant__ TcGroupArgs A, int tile_bytes, int tmem_cols, int stages)
{
    using namespace tcd;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Header* H = reinterpret_cast<Header*>(smem_raw);
    unsigned char* tiles = smem_raw + (kTcHeader + stages * kTcStageBytes);
    Pipe pipe;
    setup(H, pipe, smem_raw, A.error, (size_t)tile_bytes, tmem_cols, stages);
    const bool tma_ok = (smem_u32(smem_raw) & 127u) == 0;       // tensor copies want 128-byte aligned destinations
    int* hdr = H->hdr;
    const int items = A.N * A.R * A.Q;

    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int n = item / (A.R * A.Q), rq = item % (A.R * A.Q), r = rq / A.Q, q = rq % A.Q;
        load_header(hdr, A, r, q, true);
        __syncthreads();
        {   // group input -> input tile of the first op (halo comes from the neighbours' part of the map)
            const OpDesc& op = A.op[0];
            const int oh = hdr[8 + 1] - hdr[8 + 0] + 1, ow = hdr[8 + 3] - hdr[8 + 2] + 1;
            const int bh = (oh - 1) * op.S + op.keff, bw = (ow - 1) * op.S + op.keff;
            const Tile IN = make_tile(tiles, op.t_in_off, op.cin16 / 8, op.t_in_Hp, op.t_in_Wp);
            if ((A.use_tma & 1u) && tma_ok) load_tile_tma(pipe, IN, A.tmap[0], n, hdr[8 + 0] * op.S - op.pad, hdr[8 + 2] * op.S - op.pad);
            else load_tile(IN, bh, bw, bw, A.map[0], A.in_f32 != 0, A.in_C, n, op.in_H, op.in_W, hdr[8 + 0] * op.S - op.pad,
                           hdr[8 + 2] * op.S - op.pad);
        }
        for (int i = 0; i < A.n_ops; ++i) {
            const OpDesc& op = A.op[i];
            const int* ho = hdr + (i + 1) * 8;
            const int oy1 = ho[0], ox1 = ho[2];
            const int oh = ho[1] - ho[0] + 1, ow = ho[3] - ho[2] + 1;
            const int cy1 = ho[4], cy2 = ho[5], cx1 = ho[6], cx2 = ho[7];
            const bool last = i == A.n_ops - 1;
            Tile NT{}; int noy = 0, nox = 0;
            if (!last) {
                const OpDesc& nx = A.op[i + 1];
                const int* hn = hdr + (i + 2) * 8;
                NT = make_tile(tiles, nx.t_in_off, nx.cin16 / 8, nx.t_in_Hp, nx.t_in_Wp);
                noy = hn[0] * nx.S - nx.pad; nox = hn[2] * nx.S - nx.pad;
                const int nbh = (hn[1] - hn[0]) * nx.S + nx.keff, nbw = (hn[3] - hn[2]) * nx.S + nx.keff;
                zero_outside(NT, nbh, nbw, oy1 - noy, oy1 - noy + oh - 1, ox1 - nox, ox1 - nox + ow - 1);
            }
            __nv_bfloat16* gout = A.map_out[i + 1];
            unsigned char* garg = A.arg[i];
            const int OH = op.out_H, OW = op.out_W, oplanes = op.cout16 / 8;
            // one 16-byte entry (8 channels of plane pl) of the op's output at span position (ly, lx)
            auto emit = [&](int pl, int ly, int lx, const uint4& v, unsigned long long am, bool has_arg) {
                const int y = oy1 + ly, x = ox1 + lx;
                if (!last) *NT.at(pl, y - noy, x - nox) = v;
                if (y >= cy1 && y <= cy2 && x >= cx1 && x <= cx2) {
                    const size_t gi = (((size_t)n * oplanes + pl) * OH + y) * OW + x;
                    reinterpret_cast<uint4*>(gout)[gi] = v;
                    if (has_arg) reinterpret_cast<unsigned long long*>(garg)[gi] = am;
                }
            };
            const Tile IT = make_tile(tiles, op.t_in_off, op.cin16 / 8, op.t_in_Hp, op.t_in_Wp);
            if (op.kind == kOpPool) {
                __syncthreads();
                const int total = oplanes * oh * ow;
                for (int e = threadIdx.x; e < total; e += blockDim.x) {
                    const int lx = e % ow, t = e / ow, ly = t % oh, pl = t / oh;
                    const uint4* s = IT.at(pl, 2 * ly, 2 * lx);
                    float a[8], b[8];
                    unpack8(s[0], a);
                    unpack8(s[1], b);
#pragma unroll
                    for (int c = 0; c < 8; ++c) a[c] = b[c] > a[c] ? b[c] : a[c];
                    unpack8(s[IT.Wp], b);
#pragma unroll
                    for (int c = 0; c < 8; ++c) a[c] = b[c] > a[c] ? b[c] : a[c];
                    unpack8(s[IT.Wp + 1], b);
#pragma unroll
                    for (int c = 0; c < 8; ++c) a[c] = b[c] > a[c] ? b[c] : a[c];
                    emit(pl, ly, lx, pack8(a), 0ull, false);
                }
                __syncthreads();
                continue;
            }
            // bias of this op -> shared memory (zero for the padded channels; no parameters: a convolution without bias)
            const float* bias = A.params ? A.params + op.p_off + (size_t)op.cout * op.cin * op.k * op.k : nullptr;
            for (int c = threadIdx.x; c < op.cout16; c += blockDim.x) H->bias[c] = (bias && c < op.cout) ? __ldg(bias + c) : 0.f;
            tc::fence_async_smem();      // tile written with ordinary stores, read by the tensor core
            __syncthreads();
            const float slope = op.slope;
            const bool pooled = op.kind == kOpConvPool;
            const int coh = op.S * oh, cow = op.S * ow;
            conv_mma(pipe, tc::smem_u32(IT.base), IT.Wp, IT.plane, op.cin16 / 8, op.k, op.cout16,
                     A.wpk + op.twf_off, coh, cow,
                     [&](int by, int bx, int qq, int lane, int c0, float (&v)[16]) {
                const int py = by * 16 + qq * 4 + (lane >> 3), px = bx * 8 + (lane & 7);
#pragma unroll
                for (int c = 0; c < 16; ++c) { const float z = v[c] + H->bias[c0 + c]; v[c] = z > 0.f ? z : slope * z; }
                if (!pooled) {
                    if (py < coh && px < cow) {
                        emit(c0 / 8, py, px, pack8(v), 0ull, false);
                        emit(c0 / 8 + 1, py, px, pack8(v + 8), 0ull, false);
                    }
                } else {
                    // the pool and its arg-max act on the values as they are stored (bf16)
                    unsigned long long am[2] = {0ull, 0ull};
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        v[c] = __bfloat162float(__float2bfloat16(v[c]));
                        const float v01 = __shfl_xor_sync(0xffffffffu, v[c], 1);
                        const float v10 = __shfl_xor_sync(0xffffffffu, v[c], 8);
                        const float v11 = __shfl_xor_sync(0xffffffffu, v[c], 9);
                        float best = v[c]; unsigned a = 0;
                        if (v01 > best) { best = v01; a = 1; }
                        if (v10 > best) { best = v10; a = 2; }
                        if (v11 > best) { best = v11; a = 3; }
                        v[c] = best;
                        am[c >> 3] |= (unsigned long long)a << ((c & 7) * 8);
                    }
                    if (((lane & 1) | ((lane >> 3) & 1)) == 0 && py < coh && px < cow) {
                        emit(c0 / 8, py >> 1, px >> 1, pack8(v), am[0], true);
                        emit(c0 / 8 + 1, py >> 1, px >> 1, pack8(v + 8), am[1], true);
                    }
                }
            });
        }
        __syncthreads();
    }
    teardown(H);
}

// ---------------------------------------------------------------------------------------------
// Fused backward of one group, bf16 (adjoint form): each block owns one partial gradient set and
// walks through its share of the (image, sub-tile) stacks of one user tile in a fixed order.
// ---------------------------------------------------------------------------------------------
template <int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 2 : 1) bwd_group_tc_kernel(const __grid_constant__ TcGroupArgs A, int tile_bytes, int tmem_cols, int stages)
{
    using namespace tcd;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Header* H = reinterpret_cast<Header*>(smem_raw);
    unsigned char* tiles = smem_raw + (kTcHeader + stages * kTcStageBytes);
    Pipe pipe;
    setup(H, pipe, smem_raw, A.error, (size_t)tile_bytes, tmem_cols, stages);
    const bool tma_ok = (smem_u32(smem_raw) & 127u) == 0;       // tensor copies want 128-byte aligned destinations
    int* hdr = H->hdr;

    // The sub-tile stacks of the whole batch, image by image and row by row, are dealt out evenly to
    // the blocks; each block adds the filter gradients of its stacks into its own partial set.
    const int slot = blockIdx.x;
    const int items = A.N * A.R * A.Q;
    const int lo = (int)((long long)slot * items / (int)gridDim.x), hi = (int)((long long)(slot + 1) * items / (int)gridDim.x);
    float* myset = A.partial + (size_t)slot * A.set_floats;
    const int nops = A.n_ops;

    // Write 8 channels (plane pl) of a delta at position (ly, lx) of op j's output span into op j's dz tile:
    // directly (conv: inside the apron; pool: as is) or through the arg-max of the fused pool.
    auto put_dz = [&](const OpDesc& oj, const Tile& DZ, int pl, int ly, int lx, const float* v, unsigned long long am) {
        if (oj.kind == kOpConvPool) {
            const int a = oj.k - 1;
            float z[8];
#pragma unroll
            for (int w = 0; w < 4; ++w) {
#pragma unroll
                for (int c = 0; c < 8; ++c) z[c] = (int)((am >> (c * 8)) & 3ull) == w ? v[c] : 0.f;
                *DZ.at(pl, a + 2 * ly + (w >> 1), a + 2 * lx + (w & 1)) = pack8(z);
            }
        } else {
            const int a = oj.kind == kOpConv ? oj.k - 1 : 0;
            *DZ.at(pl, a + ly, a + lx) = pack8(v);
        }
    };

    for (int item = lo; item < hi; ++item) {
        const bool first = item == lo;
        const int n = item / (A.R * A.Q), r = (item / A.Q) % A.R, q = item % A.Q;
        __syncthreads();
        load_header(hdr, A, r, q, false);
        __syncthreads();

        {   // delta at the group's output map over this sub-tile's cut -> dz tile of the last op
            const OpDesc& op = A.op[nops - 1];
            const int* ho = hdr + nops * 8;
            const int oh = ho[1] - ho[0] + 1, ow = ho[3] - ho[2] + 1;
            const Tile DZ = make_tile(tiles, op.t_dz_off, op.t_dz_planes, op.t_dz_Hp, op.t_dz_Wp);
            zero_bytes(DZ.base, (size_t)DZ.planes * DZ.plane);
            __syncthreads();
            const bool act = op.kind != kOpPool;
            const int oplanes = op.cout16 / 8;
            const uint4* ysrc = static_cast<const uint4*>(A.map[nops]);
            const unsigned long long* asrc = reinterpret_cast<const unsigned long long*>(A.arg[nops - 1]);
            const int total = oplanes * oh * ow;
            for (int e = threadIdx.x; e < total; e += blockDim.x) {
                const int lx = e % ow, t = e / ow, ly = t % oh, pl = t / oh;
                const int y = ho[0] + ly, x = ho[2] + lx;
                float v[8];
                const size_t gi = (((size_t)n * oplanes + pl) * op.out_H + y) * op.out_W + x;
                if (A.dmap_planes) {
                    unpack8(__ldg(static_cast<const uint4*>(A.dmap_out) + gi), v);
                } else {
                    const float* dsrc = static_cast<const float*>(A.dmap_out);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int ch = pl * 8 + c;
                        v[c] = ch < op.cout ? __ldg(dsrc + (((size_t)n * op.cout + ch) * op.out_H + y) * op.out_W + x) : 0.f;
                    }
                }
                if (act) {
                    float yv[8];
                    unpack8(__ldg(ysrc + gi), yv);
#pragma unroll
                    for (int c = 0; c < 8; ++c) v[c] *= yv[c] > 0.f ? 1.f : op.slope;
                }
                put_dz(op, DZ, pl, ly, lx, v, op.kind == kOpConvPool ? asrc[gi] : 0ull);
            }
        }

        for (int i = nops - 1; i >= 0; --i) {
            const OpDesc& op = A.op[i];
            const int* ho = hdr + (i + 1) * 8;     // span at this op's output map
            const int* hi_ = hdr + i * 8;          // span at its input map
            const int oh = ho[1] - ho[0] + 1, ow = ho[3] - ho[2] + 1;
            const int oy = ho[0] * op.S - op.pad, ox = ho[2] * op.S - op.pad;   // map position of the X tile's (0,0)
            const int bh = (oh - 1) * op.S + op.keff, bw = (ow - 1) * op.S + op.keff;
            const int ih = hi_[1] - hi_[0] + 1, iw = hi_[3] - hi_[2] + 1;       // valid input span
            const int vy0 = hi_[0] - oy, vx0 = hi_[2] - ox;                     // its offset inside the X tile
            const Tile X = make_tile(tiles, op.t_x_off, op.cin16 / 8, op.t_x_Hp, op.t_x_Wp);
            const Tile DZ = make_tile(tiles, op.t_dz_off, op.t_dz_planes, op.t_dz_Hp, op.t_dz_Wp);
            if (((A.use_tma >> i) & 1u) && tma_ok) load_tile_tma(pipe, X, A.tmap[i], n, oy, ox);
            else load_tile(X, bh, bw, X.Wp, A.map[i], i == 0 && A.in_f32, A.in_C, n, op.in_H, op.in_W, oy, ox);
            const bool to_scratch = i == 0;
            Tile PD{};
            const OpDesc& pv = A.op[i > 0 ? i - 1 : 0];
            if (!to_scratch) {
                PD = make_tile(tiles, pv.t_dz_off, pv.t_dz_planes, pv.t_dz_Hp, pv.t_dz_Wp);
                zero_bytes(PD.base, (size_t)PD.planes * PD.plane);
            }
            float* sdst = nullptr;
            const bool scratch_planes = !A.in_f32;
            if (to_scratch) {
                const int Wtot = A.xoff[A.Q], Htot = A.yoff[A.R];
                const int sc = scratch_planes ? op.cin16 : op.cin;
                sdst = A.scratch + (size_t)n * sc * Htot * Wtot + (size_t)sc * ((size_t)A.yoff[r] * Wtot + (size_t)ih * A.xoff[q]);
            }
            const unsigned long long* parg = (!to_scratch && pv.kind == kOpConvPool)
                                                 ? reinterpret_cast<const unsigned long long*>(A.arg[i - 1]) : nullptr;
            const int pplanes = op.cin16 / 8;
            tc::fence_async_smem();
            __syncthreads();   // X loaded, dz complete, producer tile zeroed

            const float pslope = op.prev_has_act ? pv.slope : 1.f;
            const bool pact = op.prev_has_act != 0;
            const bool need_in_delta = !to_scratch || A.need_dx;
            // 8 channels (plane pl) of the delta at input-span position (uy, ux): through the producer's
            // activation, then into the producer's dz tile or the scratch block of this sub-tile
            auto put_in = [&](int pl, int uy, int ux, float* v) {
                if (pact) {
                    float xv[8];
                    unpack8(*X.at(pl, vy0 + uy, vx0 + ux), xv);
#pragma unroll
                    for (int c = 0; c < 8; ++c) v[c] *= xv[c] > 0.f ? 1.f : pslope;
                }
                if (to_scratch && scratch_planes) {
                    float4* o = reinterpret_cast<float4*>(sdst + (((size_t)pl * ih + uy) * iw + ux) * 8);
                    o[0] = make_float4(v[0], v[1], v[2], v[3]);
                    o[1] = make_float4(v[4], v[5], v[6], v[7]);
                } else if (to_scratch) {
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        if (pl * 8 + c < op.cin) sdst[((size_t)(pl * 8 + c) * ih + uy) * iw + ux] = v[c];
                } else {
                    unsigned long long am = 0ull;
                    if (parg) am = parg[(((size_t)n * pplanes + pl) * op.in_H + hi_[0] + uy) * op.in_W + hi_[2] + ux];
                    put_dz(pv, PD, pl, uy, ux, v, am);
                }
            };

            if (op.kind == kOpPool) {
                if (need_in_delta) {
                    const int total = pplanes * oh * ow;
                    for (int e = threadIdx.x; e < total; e += blockDim.x) {
                        const int lx = e % ow, t = e / ow, ly = t % oh, pl = t / oh;
                        const uint4* s = X.at(pl, 2 * ly, 2 * lx);
                        float w4[4][8], d[8];
                        unpack8(s[0], w4[0]); unpack8(s[1], w4[1]); unpack8(s[X.Wp], w4[2]); unpack8(s[X.Wp + 1], w4[3]);
                        unpack8(*DZ.at(pl, ly, lx), d);
                        float o[4][8];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            float best = w4[0][c]; int am = 0;
                            if (w4[1][c] > best) { best = w4[1][c]; am = 1; }
                            if (w4[2][c] > best) { best = w4[2][c]; am = 2; }
                            if (w4[3][c] > best) { best = w4[3][c]; am = 3; }
#pragma unroll
                            for (int w = 0; w < 4; ++w) o[w][c] = am == w ? d[c] : 0.f;
                        }
#pragma unroll
                        for (int w = 0; w < 4; ++w) put_in(pl, 2 * ly + (w >> 1), 2 * lx + (w & 1), o[w]);
                    }
                }
            } else {
                const int a = op.k - 1, coh = op.S * oh, cow = op.S * ow;
                filter_grad_mma(pipe, tc::smem_u32(DZ.at(0, a, a)), DZ.plane, tc::smem_u32(X.base), X.plane, DZ.Wp, op.k,
                                op.cout16, op.cin16, op.cin, (coh - 1) * DZ.Wp + cow, myset + op.tgp_off, first);
                if (need_in_delta)
                    conv_mma(pipe, tc::smem_u32(DZ.at(0, vy0, vx0)), DZ.Wp, DZ.plane, op.cout16 / 8, op.k, op.cin16,
                             A.wpk + op.twb_off, ih, iw,
                             [&](int by, int bx, int qq, int lane, int c0, float (&v)[16]) {
                        const int py = by * 16 + qq * 4 + (lane >> 3), px = bx * 8 + (lane & 7);
                        if (py < ih && px < iw) {
                            put_in(c0 / 8, py, px, v);
                            put_in(c0 / 8 + 1, py, px, v + 8);
                        }
                    });
            }
            __syncthreads();
        }
    }
    teardown(H);
}

// Backward boundary exchange of the tensor-core path for every group but the first: sum of the
// overlapping per-sub-tile deltas (fp32 [c/8][h][w][8] blocks) in a fixed (row, column) order, written
// as the bf16 planes the previous group's backward reads.  One warp per row (n, plane, y).
__global__ void halo_sum_planes_kernel(const __grid_constant__ HaloSumArgs A)
{
    extern __shared__ int halo_tab[];
    int* xcover = halo_tab;              int* xspan = xcover + 2 * A.W;   int* xoff = xspan + 2 * A.Q;
    int* ycover = xoff + A.Q + 1;        int* yspan = ycover + 2 * A.H;   int* yoff = yspan + 2 * A.R;
    for (int i = threadIdx.x; i < 2 * A.W; i += blockDim.x) xcover[i] = A.xcover[i];
    for (int i = threadIdx.x; i < 2 * A.H; i += blockDim.x) ycover[i] = A.ycover[i];
    for (int i = threadIdx.x; i < 2 * A.Q; i += blockDim.x) xspan[i] = A.xspan[i];
    for (int i = threadIdx.x; i < 2 * A.R; i += blockDim.x) yspan[i] = A.yspan[i];
    for (int i = threadIdx.x; i <= A.Q; i += blockDim.x) xoff[i] = A.xoff[i];
    for (int i = threadIdx.x; i <= A.R; i += blockDim.x) yoff[i] = A.yoff[i];
    __syncthreads();
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const int planes = A.C / 8;                                   // A.C = padded channel count
    const long long rows = (long long)A.N * planes * A.H;
    uint4* out = reinterpret_cast<uint4*>(A.out);
    for (long long row = (long long)blockIdx.x * wpb + (threadIdx.x >> 5); row < rows; row += (long long)gridDim.x * wpb) {
        const int y = (int)(row % A.H); long long t = row / A.H;
        const int pl = (int)(t % planes); const int n = (int)(t / planes);
        const int r0 = ycover[2 * y], nr = ycover[2 * y + 1] - r0 + 1;       // the first four covering rows are prepared, the rest walked
        int base[4], ch[4], dr[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int r = min(r0 + k, A.R - 1);
            const int y1 = yspan[2 * r], h = yspan[2 * r + 1] - y1 + 1;
            base[k] = A.C * yoff[r] * A.Wtot; ch[k] = A.C * h; dr[k] = pl * h + (y - y1);
        }
        const float* img = A.scratch + (size_t)n * A.C * A.Htot * A.Wtot;
        for (int x = lane; x < A.W; x += 32) {
            const int q0 = xcover[2 * x], q1 = xcover[2 * x + 1];
            float s[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            // the first two covering sub-tile columns are handled without a loop, so that the loads of
            // up to 4 x 2 blocks are in flight together (same order of the sums as the plain loops)
            const int qb = min(q0 + 1, A.Q - 1);
            const int xa1 = xspan[2 * q0], wa = xspan[2 * q0 + 1] - xa1 + 1, oa = xoff[q0];
            const int xb1 = xspan[2 * qb], wb = xspan[2 * qb + 1] - xb1 + 1, ob = xoff[qb];
            const bool two = q1 > q0;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < nr) {
                    {
                        const float4* e = reinterpret_cast<const float4*>(img + base[k] + oa * ch[k] + (dr[k] * wa + (x - xa1)) * 8);
                        const float4 a = e[0], b = e[1];
                        s[0] += a.x; s[1] += a.y; s[2] += a.z; s[3] += a.w; s[4] += b.x; s[5] += b.y; s[6] += b.z; s[7] += b.w;
                    }
                    if (two) {
                        const float4* e = reinterpret_cast<const float4*>(img + base[k] + ob * ch[k] + (dr[k] * wb + (x - xb1)) * 8);
                        const float4 a = e[0], b = e[1];
                        s[0] += a.x; s[1] += a.y; s[2] += a.z; s[3] += a.w; s[4] += b.x; s[5] += b.y; s[6] += b.z; s[7] += b.w;
                    }
                    for (int q = q0 + 2; q <= q1; ++q) {
                        const int x1 = xspan[2 * q], w = xspan[2 * q + 1] - x1 + 1;
                        const float4* e = reinterpret_cast<const float4*>(img + base[k] + xoff[q] * ch[k] + (dr[k] * w + (x - x1)) * 8);
                        const float4 a = e[0], b = e[1];
                        s[0] += a.x; s[1] += a.y; s[2] += a.z; s[3] += a.w; s[4] += b.x; s[5] += b.y; s[6] += b.z; s[7] += b.w;
                    }
                }
            for (int k = 4; k < nr; ++k) {                 // very fine splits: same order, offsets worked out on the spot
                const int r = r0 + k, y1 = yspan[2 * r], h = yspan[2 * r + 1] - y1 + 1;
                for (int q = q0; q <= q1; ++q) {
                    const int x1 = xspan[2 * q], w = xspan[2 * q + 1] - x1 + 1;
                    const float4* e = reinterpret_cast<const float4*>(img + A.C * yoff[r] * A.Wtot + xoff[q] * (A.C * h) +
                                                                      ((pl * h + (y - y1)) * w + (x - x1)) * 8);
                    const float4 a = e[0], b = e[1];
                    s[0] += a.x; s[1] += a.y; s[2] += a.z; s[3] += a.w; s[4] += b.x; s[5] += b.y; s[6] += b.z; s[7] += b.w;
                }
            }
            out[row * A.W + x] = tcd::pack8(s);
        }
    }
}

// Cross-tile reduction of the partial gradient sets of the tensor-core path in a fixed order, fused
// with the update.  A set holds each layer as [window position][cout16][cin16] + [cout16] bias.
struct TcReduceLayer { long long p_off; const float* partial; long long set_floats, tgp_off; int sets, cin, cout, k, cin16, cout16; };
struct TcReduceArgs { int n; TcReduceLayer l[kMaxOps * 2]; };

__global__ void reduce_sgd_tc_kernel(const __grid_constant__ TcReduceArgs A, float* __restrict__ params, float lr,
                                     float* __restrict__ grad_out)
{
    // Threads walk the set's own arrangement, so the reads of every set are coalesced (the sets are the
    // bulk of the traffic); the one write per parameter goes to its place in the caller's arrangement.
    const TcReduceLayer L = A.l[blockIdx.y];
    const int KK = L.k * L.k;
    const long long nf = (long long)KK * L.cout16 * L.cin16, total = nf + L.cout16;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        long long dst;
        if (e < nf) {
            const int ci = (int)(e % L.cin16); long long t = e / L.cin16;
            const int co = (int)(t % L.cout16); const int tap = (int)(t / L.cout16);
            if (ci >= L.cin || co >= L.cout) continue;
            dst = L.p_off + ((long long)co * L.cin + ci) * KK + tap;
        } else {
            const int co = (int)(e - nf);
            if (co >= L.cout) continue;
            dst = L.p_off + (long long)L.cout * L.cin * KK + co;
        }
        const float* src = L.partial + L.tgp_off + e;
        float s = 0.f;
#pragma unroll 16
        for (int k = 0; k < L.sets; ++k) s += src[(size_t)k * L.set_floats];
        if (grad_out) grad_out[dst] = s;
        if (params) params[dst] = params[dst] - lr * s;
    }
}

// fp32 NCHW view of a saved bf16 map (the network output handed back to the caller).
__global__ void planes_to_nchw_kernel(const __nv_bfloat16* __restrict__ src, float* __restrict__ dst, int N, int C, int C16,
                                      int H, int W)
{
    const size_t total = (size_t)N * C * H * W;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const int x = (int)(e % W); size_t t = e / W;
        const int y = (int)(t % H); t /= H;
        const int c = (int)(t % C); const int n = (int)(t / C);
        dst[e] = __bfloat162float(src[((((size_t)n * (C16 / 8) + c / 8) * H + y) * W + x) * 8 + (c & 7)]);
    }
}

// Filters -> the two packed bf16 arrangements of the tensor-core kernels:
//   wf[tap][cin16/8][cout16][8]   B operand of the forward pass   (rows = cout, K = cin)
//   wb[tap'][cout16/8][cin16][8]  B operand of the delta pass, tap' = K*K-1-tap (rotated 180 degrees; rows = cin, K = cout)
// Layers run by the banded kernels (sliced != 0) get instead, per pass, the arrangement in which the filters one block
// needs for one chunk of input channels are contiguous (one bulk copy):
//   wf[slice][chunk][tap][kpc_f][ns_f][8]    rows = output channels slice*ns_f .., K = input channels (chunk*kpc_f + j)*8 ..
//   wb[slice][chunk][tap'][kpc_d][ns_d][8]   rows = input channels slice*ns_d ..,  K = output channels (chunk*kpc_d + j)*8 ..
// with zeros beyond the layer's channel counts.
struct TcPackLayer { long long p_off, w_off; int cin, cout, k, cin16, cout16; int sliced, ns_f, kpc_f, ns_d, kpc_d; };
struct TcPackArgs { int n; TcPackLayer l[kMaxOps * 2]; };

__global__ void pack_filters_tc_kernel(const __grid_constant__ TcPackArgs A, const float* __restrict__ params,
                                       __nv_bfloat16* __restrict__ wf, __nv_bfloat16* __restrict__ wb)
{
    const TcPackLayer L = A.l[blockIdx.y];
    const int KK = L.k * L.k;
    if (L.sliced) {
        const int nch_f = (L.cin16 / 8 + L.kpc_f - 1) / L.kpc_f, nch_d = (L.cout16 / 8 + L.kpc_d - 1) / L.kpc_d;
        const long long per_f = (long long)((L.cout16 + L.ns_f - 1) / L.ns_f) * nch_f * KK * L.kpc_f * L.ns_f * 8;
        const long long per_d = (long long)((L.cin16 + L.ns_d - 1) / L.ns_d) * nch_d * KK * L.kpc_d * L.ns_d * 8;
        // one thread per 16-byte entry (8 contraction channels of one row): the position is worked out once per entry
        const long long ent_f = per_f / 8, ent_d = per_d / 8;
        for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < ent_f + ent_d; e += (long long)gridDim.x * blockDim.x) {
            const bool fwd = e < ent_f;
            const int ns = fwd ? L.ns_f : L.ns_d, kpc = fwd ? L.kpc_f : L.kpc_d, nch = fwd ? nch_f : nch_d;
            long long t = fwd ? e : e - ent_f;
            const int r = (int)(t % ns); t /= ns;
            const int j = (int)(t % kpc); t /= kpc;
            const int tap = (int)(t % KK); t /= KK;
            const int c = (int)(t % nch); const int sl = (int)(t / nch);
            const int row = sl * ns + r, k0 = (c * kpc + j) * 8;                  // output row of the GEMM, first contraction channel
            const int ptap = fwd ? tap : KK - 1 - tap;
            float v[8];
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
                const int co = fwd ? row : k0 + c8, ci = fwd ? k0 + c8 : row;
                v[c8] = (co < L.cout && ci < L.cin) ? __ldg(params + L.p_off + ((long long)co * L.cin + ci) * KK + ptap) : 0.f;
            }
            uint4* dst = reinterpret_cast<uint4*>(fwd ? wf + L.w_off : wb + L.w_off) + (fwd ? e : e - ent_f);
            *dst = tcd::pack8(v);
        }
        return;
    }
    const long long per = (long long)KK * L.cin16 * L.cout16;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < 2 * per; e += (long long)gridDim.x * blockDim.x) {
        if (e < per) {
            const int c8 = (int)(e % 8); long long t = e / 8;
            const int co = (int)(t % L.cout16); t /= L.cout16;
            const int cp = (int)(t % (L.cin16 / 8)); const int tap = (int)(t / (L.cin16 / 8));
            const int ci = cp * 8 + c8;
            const float v = (co < L.cout && ci < L.cin) ? params[L.p_off + ((long long)co * L.cin + ci) * KK + tap] : 0.f;
            wf[L.w_off + e] = __float2bfloat16(v);
        } else {
            const long long f = e - per;
            const int c8 = (int)(f % 8); long long t = f / 8;
            const int ci = (int)(t % L.cin16); t /= L.cin16;
            const int cp = (int)(t % (L.cout16 / 8)); const int tapr = (int)(t / (L.cout16 / 8));
            const int co = cp * 8 + c8;
            const float v = (co < L.cout && ci < L.cin) ? params[L.p_off + ((long long)co * L.cin + ci) * KK + (KK - 1 - tapr)] : 0.f;
            wb[L.w_off + f] = __float2bfloat16(v);
        }
    }
}

}  // namespace ftp
