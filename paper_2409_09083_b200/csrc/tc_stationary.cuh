// bf16 path, one-conv groups: the filter gradient by a weight-stationary tensor-core kernel.
//
// In the fused tile-stack kernel every sub-tile adds its whole partial filter gradient (K*K*cout*cin fp32) to
// the block's partial set, because tensor memory cannot keep the accumulators of a wide layer across sub-tiles.
// For layers with hundreds of channels that flush costs several times the MMAs.  Here the roles are turned
// round: a block owns a slice of the FILTER GRADIENT (64 or 128 output channels x up to 48 input channels x all
// window positions; K*K accumulators of `ncols` columns each, plus 16 columns for the bias gradient) and keeps
// it in tensor memory while bands of rows of the whole batch stream past it, so the gradient leaves the SM
// once.  The pixels are dealt out in `shares`; a share is one partial gradient set of Section 4.1, summed by
// the same cross-tile reduction as the sets of the fused kernels.
//
// A band is R rows of one image at the conv's resolution.  The delta in front of the activation (dz, bf16
// planes, written by delta_act_planes_kernel) and the layer's saved input map arrive by TMA tensor copies
// into tiles of the same pitch Wp = W + K - 1: dz at columns 0 .. W-1 with zeros behind them (beyond the
// tensor's edge), the input shifted by the padding.  With equal pitches one run of 16 consecutive tile entries
// is a K step of both operands (MN-major, 8 pixels x 8 channels per core matrix), and window position (ky, kx)
// only moves the start of the input operand by ky * Wp + kx entries.  Two stages: the copies of the next band
// run behind the MMAs of the current one.
#pragma once

#include "kernels_tc.cuh"

namespace ftp {

struct TcFilterGradArgs {
    alignas(64) unsigned char tmap_dz[128];   // [N x cout16/8][H][W][8] bf16, box = 8 x Wp x R
    alignas(64) unsigned char tmap_x[128];    // [N x cin16/8][H][W][8] bf16,  box = 8 x Wp x (R + K - 1)
    float* partial;                           // partial sets of the group
    long long set_floats, tgp_off;            // floats per set, offset of this layer inside a set
    int* error;
    int N, K, cout16, cin16;
    int Ms, slices;                           // output channels per block (64 or 128) and number of such slices
    int ncols, nci;                           // input channels per block (multiple of 16) and number of such slices
    int R, Wp, bands_img, bands, shares;      // rows per band, tile pitch, bands per image / in the batch, pixel shares
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

    auto wait = [&](unsigned long long* bar, uint32_t parity) {
        if (H->failed) return false;
        if (mbar_wait(smem_u32(bar), parity)) return true;
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
            const int b = b_lo + i, n = b / A.bands_img, y0 = (b - n * A.bands_img) * A.R;
            unsigned char* dzs = stages + (size_t)s * A.stage_bytes;
            unsigned char* xs = dzs + (size_t)mp * A.dz_plane;
            const uint32_t bar = smem_u32(&H->full[s]);
            mbar_expect_tx(bar, (uint32_t)((nd * A.R + np * (A.R + K - 1)) * A.Wp) * 16u);
            for (int pl = 0; pl < nd; ++pl)
                tma_load_4d(smem_u32(dzs + (size_t)pl * A.dz_plane), A.tmap_dz, 0, 0, y0, n * (A.cout16 / 8) + slice * mp + pl, bar);
            for (int pl = 0; pl < np; ++pl)
                tma_load_4d(smem_u32(xs + (size_t)pl * A.x_plane), A.tmap_x, 0, -(K / 2), y0 - K / 2, n * (A.cin16 / 8) + ci0 / 8 + pl, bar);
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
    const bool have = nb > 0 && wait(&H->done, 0);
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

}  // namespace ftp
