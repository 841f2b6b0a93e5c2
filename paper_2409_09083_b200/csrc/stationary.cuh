// Weight-stationary kernels of the fp32 path for executed groups that hold one conv layer
// (optionally with the 2x2 max-pool after it).  The paper leaves weight-dominated layers to a
// weight partitioning it names as future work (Section 6); here such a layer is cut along its
// channels and its pixels instead of into fused stacks: a block keeps a slice of the filter
// (forward, input delta) or of the filter gradient (Section 4.1: feature-map tile convolved with the
// delta tile) on chip and streams pixel tiles through it.  The exchange with the neighbouring
// groups goes through the full maps in global memory, as at every group boundary (Section 3).
//
//   conv_rows_kernel         out = conv(in, w) (+ bias, leaky ReLU, optional fused 2x2 max-pool with
//                            arg-max): the forward convolution and, with the rotated filters, the
//                            input delta (Section 4.1)
//   filter_grad_rows_kernel  partial filter and bias gradients of a (64 output, 32 input) channel
//                            slice over a share of the pixels; the cross-tile reduction sums the shares
//   delta_act_kernel         the delta in front of the activation, dZ = dY * leaky'(Y), at the conv's
//                            resolution (routed through the arg-max where a pool follows)
//
// Rows are taken in pairs over the whole batch (image after image), so a tile of row pairs may span
// images and no rows are wasted on maps whose height is not a multiple of the tile; every row pair
// keeps its own K + 1 input rows in shared memory.  Columns are taken eight at a time.
// Each output value of the convolution is accumulated over input channels in ascending order and,
// per channel, over the window columns and then rows: the order of the fused stack kernels, so both
// give the same bits.
#pragma once

#include <cuda_runtime.h>

#include "plan.hpp"
#include "stationary_args.hpp"

namespace ftp {

// Shared-memory geometry of one input stage of the convolution, in floats.  Column 0 of a block's
// columns sits at offset 4 of a row (16-byte aligned for the 4-wide reads); the left halo uses offset
// 3 and the right halo the first, otherwise unused, slot of the next row.  The stride between row
// pairs is 8 or 24 modulo 32, so that the eight lanes of a quarter warp (two column quads of four row
// pairs) read 4-wide without bank conflicts.
// T = threads of a block: 256 (two blocks per SM), or 128 (four per SM, half the row pairs and half the channels per
// stage each) for launches with so few blocks that whole blocks would leave SMs idle in the last round.
template <int K, int CO, int T = kStThreads> struct StGeom {
    static constexpr int P = K / 2, RR = K + 1;
    static constexpr int npg = T * 8 / CO;                           // pixel groups (2 rows x 4 columns) per block: 32 or 64 (T = 256)
    static constexpr int row_pairs = npg / 2;                        // row pairs per block: 16 or 32 (T = 256)
    static constexpr int pitch = kStCols + (K > 1 ? 4 : 0);
    static constexpr int rp_stride = K == 3 ? 56 : 24;
    static constexpr int ci_stride = row_pairs * rp_stride;
    static constexpr int ci_chunk = (K == 3 ? 8 : 32) * CO / 64 * T / kStThreads;   // input channels per stage
    static constexpr int w_stage = ci_chunk * K * K * CO;            // floats
    static constexpr int in_stage = ci_chunk * ci_stride;
    static constexpr int smem_bytes = 2 * (w_stage + in_stage) * 4;
    static constexpr int cols = kStCols + 2 * P;
};

__device__ __forceinline__ void st_cp_async16(void* smem, const void* gmem, bool valid)
{
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    const int bytes = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(s), "l"(gmem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void st_cp_async4(void* smem, const void* gmem, bool valid)
{
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    const int bytes = valid ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" :: "r"(s), "l"(gmem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void st_cp_async8(void* smem, const void* gmem, bool valid)
{
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    const int bytes = valid ? 8 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" :: "r"(s), "l"(gmem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void st_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void st_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

// K = 1 or 3 (stride 1, padding K / 2); CO = 64 or 32 output channels per block (32 for layers with at most 32,
// which then take twice the row pairs).  Thread tile: 8 output channels x (2 rows x 4 columns).
// VEC = floats per copy of the input columns: 4 where the map's rows are 16-byte aligned (width a multiple of 4), else 2 or 1.
template <int K, int CO, int VEC, int T = kStThreads>
__global__ void __launch_bounds__(T, 512 / T) conv_rows_kernel(const __grid_constant__ ConvRowsArgs A)
{
    using G = StGeom<K, CO, T>;
    extern __shared__ __align__(16) float st_smem[];
    constexpr int KK = K * K, P = G::P, RR = G::RR;
    const int tid = threadIdx.x;
    const int cg = tid / G::npg, pg = tid % G::npg;          // a warp shares its 8 output channels: filter reads are broadcasts
    const int rp_l = pg >> 1, cq_l = pg & 1;
    const int co_t = blockIdx.x % A.co_tiles;
    const int xt = (blockIdx.x / A.co_tiles) % A.x_tiles;
    const int rt = blockIdx.x / (A.co_tiles * A.x_tiles);
    const int co0 = co_t * CO, x0 = xt * kStCols, rp0 = rt * G::row_pairs;
    float* sw = st_smem;                                     // two filter stages
    float* si = st_smem + 2 * G::w_stage;                    // two input stages
    const size_t plane = (size_t)A.H * A.W;

    // What this thread copies of the input in every stage.  A row of a row pair is copied as its left halo
    // column (3 x 3 only), its eight columns in pieces of VEC floats and its right halo column; piece i of the
    // block is (row pair, row, piece of the row).
    constexpr int vec = VEC;
    constexpr int per_row = kStCols / vec + 2 * P, nitems = G::row_pairs * RR * per_row;
    constexpr int max_items = (nitems + T - 1) / T;
    int it_s[max_items]; long long it_g[max_items]; unsigned it_ok = 0, it_halo = 0;
#pragma unroll
    for (int e = 0; e < max_items; ++e) {
        const int idx = tid + e * T;
        it_s[e] = -1; it_g[e] = 0;
        if (idx < nitems) {
            const int piece = idx % per_row, t = idx / per_row, r = t % RR, rl = t / RR;
            // column of the piece relative to the block's first column, and whether it is a single halo column
            int c; bool halo = false;
            if (P && piece == 0) { c = -1; halo = true; }
            else if (P && piece == per_row - 1) { c = kStCols; halo = true; }
            else c = (piece - P) * vec;
            const int rp = rp0 + rl;
            const int n = rp / A.rp_img, y = (rp - n * A.rp_img) * 2 + r - P, x = x0 + c;
            it_s[e] = rl * G::rp_stride + r * G::pitch + c + 4;
            if (halo) it_halo |= 1u << e;
            if (n < A.N && y >= 0 && y < A.H && x >= 0 && x < A.W) {     // a piece lies wholly inside or outside the row
                it_ok |= 1u << e;
                it_g[e] = (long long)n * A.Cin * plane + (long long)y * A.W + x;
            }
        }
    }
    auto load_stage = [&](int chunk) {
        const int ci0 = chunk * G::ci_chunk, nci = min(G::ci_chunk, A.Cin - ci0);
        float* dw = sw + (chunk & 1) * G::w_stage;
        float* di = si + (chunk & 1) * G::in_stage;
        // filters: a row of CO floats per (channel, tap)
        constexpr int q = CO / 4;
        for (int i = tid; i < nci * KK * q; i += T) {
            const int row = i / q, j = i - row * q;
            const int co = co0 + 4 * j;
            st_cp_async16(dw + row * CO + 4 * j, A.w + ((size_t)ci0 * KK + row) * A.CoutPad + min(co, A.CoutPad - 4), co < A.CoutPad);
        }
#pragma unroll
        for (int e = 0; e < max_items; ++e)
            if (it_s[e] >= 0) {
                const bool ok = (it_ok >> e) & 1u;
                const float* src = A.in + it_g[e] + (size_t)ci0 * plane;
                float* dst = di + it_s[e];
                const int w = ((it_halo >> e) & 1u) ? 1 : vec;
                if (w == 4) for (int ci = 0; ci < nci; ++ci) st_cp_async16(dst + ci * G::ci_stride, src + (size_t)ci * plane, ok);
                else if (w == 2) for (int ci = 0; ci < nci; ++ci) st_cp_async8(dst + ci * G::ci_stride, src + (size_t)ci * plane, ok);
                else for (int ci = 0; ci < nci; ++ci) st_cp_async4(dst + ci * G::ci_stride, src + (size_t)ci * plane, ok);
            }
        st_commit();
    };

    // Accumulators as pairs of neighbouring output channels: one packed multiply-add (two fp32 FMAs, each
    // rounded like a scalar one) updates both, which halves the instructions the FMA pipe has to be fed with.
    float2 acc[2][4][4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int co = co0 + cg * 8 + 2 * c;
        const float2 b = make_float2((A.bias != nullptr && co < A.Cout) ? __ldg(A.bias + co) : 0.f,
                                     (A.bias != nullptr && co + 1 < A.Cout) ? __ldg(A.bias + co + 1) : 0.f);
#pragma unroll
        for (int p = 0; p < 2; ++p)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[p][j][c] = b;
    }

    const int nchunks = (A.Cin + G::ci_chunk - 1) / G::ci_chunk;
    const int my_in = rp_l * G::rp_stride + cq_l * 4 + 4;    // column 0 of this thread's quad (16-byte aligned)
    load_stage(0);
    for (int chunk = 0; chunk < nchunks; ++chunk) {
        // one barrier per chunk: behind it every thread has left the previous chunk, whose buffer the next copies fill
        st_wait<0>();
        __syncthreads();
        if (chunk + 1 < nchunks) load_stage(chunk + 1);
        const int nci = min(G::ci_chunk, A.Cin - chunk * G::ci_chunk);
        const float* wc = sw + (chunk & 1) * G::w_stage + cg * 8;
        const float* ip = si + (chunk & 1) * G::in_stage + my_in;
#pragma unroll(K == 1 ? 4 : 1)
        for (int ci = 0; ci < nci; ++ci, wc += KK * CO, ip += G::ci_stride) {
            float v[RR][4 + 2 * P];
#pragma unroll
            for (int r = 0; r < RR; ++r) {
                const float4 m = *reinterpret_cast<const float4*>(ip + r * G::pitch);
                if constexpr (P > 0) v[r][0] = ip[r * G::pitch - 1];
                v[r][P] = m.x; v[r][P + 1] = m.y; v[r][P + 2] = m.z; v[r][P + 3] = m.w;
                if constexpr (P > 0) v[r][3 + 2 * P] = ip[r * G::pitch + 4];
            }
#pragma unroll
            for (int kx = 0; kx < K; ++kx)
#pragma unroll
                for (int ky = 0; ky < K; ++ky) {
                    const float4 wa = *reinterpret_cast<const float4*>(wc + (ky * K + kx) * CO);
                    const float4 wq = *reinterpret_cast<const float4*>(wc + (ky * K + kx) * CO + 4);
                    const float2 wv[4] = {make_float2(wa.x, wa.y), make_float2(wa.z, wa.w), make_float2(wq.x, wq.y), make_float2(wq.z, wq.w)};
#pragma unroll
                    for (int p = 0; p < 2; ++p)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float2 vv = make_float2(v[p + ky][j + kx], v[p + ky][j + kx]);
#pragma unroll
                            for (int c = 0; c < 4; ++c) acc[p][j][c] = __ffma2_rn(vv, wv[c], acc[p][j][c]);
                        }
                }
        }
    }

    // epilogue
    auto val = [&](int p, int j, int c) { return (c & 1) ? acc[p][j][c >> 1].y : acc[p][j][c >> 1].x; };
    const int rp = rp0 + rp_l;
    const int n = rp / A.rp_img, y = (rp - n * A.rp_img) * 2, x = x0 + cq_l * 4;
    if (n >= A.N || x >= A.W) return;
    if (!A.pool) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int co = co0 + cg * 8 + c;
            if (co >= A.Cout) break;
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                if (y + p >= A.H) break;
                float o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) { const float z = val(p, j, c); o[j] = A.act ? (z > 0.f ? z : A.slope * z) : z; }
                float* dst = A.out + (((size_t)n * A.Cout + co) * A.H + y + p) * A.W + x;
                if (x + 3 < A.W && (A.W & 3) == 0) *reinterpret_cast<float4*>(dst) = make_float4(o[0], o[1], o[2], o[3]);
                else
#pragma unroll
                    for (int j = 0; j < 4; ++j) if (x + j < A.W) dst[j] = o[j];
            }
        }
    } else {
        const int OH = A.H >> 1, OW = A.W >> 1;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int co = co0 + cg * 8 + c;
            if (co >= A.Cout) break;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (x + 2 * h >= A.W) break;
                float v00 = val(0, 2 * h, c), v01 = val(0, 2 * h + 1, c), v10 = val(1, 2 * h, c), v11 = val(1, 2 * h + 1, c);
                v00 = v00 > 0.f ? v00 : A.slope * v00; v01 = v01 > 0.f ? v01 : A.slope * v01;
                v10 = v10 > 0.f ? v10 : A.slope * v10; v11 = v11 > 0.f ? v11 : A.slope * v11;
                float best = v00; int am = 0;
                if (v01 > best) { best = v01; am = 1; }
                if (v10 > best) { best = v10; am = 2; }
                if (v11 > best) { best = v11; am = 3; }
                const size_t gi = (((size_t)n * A.Cout + co) * OH + (y >> 1)) * OW + (x >> 1) + h;
                A.out[gi] = best;
                if (A.arg) A.arg[gi] = (unsigned char)am;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Filter gradient.  Block: 64 output channels x 32 input channels; thread: 8 output channels x one
// input channel x K*K taps, all sums in registers over the block's share of the pixel tiles
// (4 row pairs x 8 columns each), in a fixed order.  The lanes of a warp hold consecutive input
// channels: delta reads are broadcasts, input reads hit distinct banks (odd channel stride).
// The sums of two neighbouring output channels share a register pair, and the delta is kept in shared
// memory with the output channels of a pixel side by side, so that one packed multiply-add (two fp32
// FMAs, each rounded like a scalar one) serves both channels.
// ---------------------------------------------------------------------------------------------
static_assert(2 * kFgRowPairs == kStThreads / 32, "one warp per delta row of a stage");
template <int K> struct FgGeom {
    static constexpr int P = K / 2, RR = K + 1;
    static constexpr int xpitch = kStCols + 2 * P;                       // input rows hold the columns -P .. 8 + P - 1
    static constexpr int x_rp = RR * xpitch;
    static constexpr int x_cs = (kFgRowPairs * x_rp) | 1;                // odd channel stride
    static constexpr int x_stage = kFgCi * x_cs;
    static constexpr int d_px = kFgCo + 4;                               // delta: [row pair][2 rows][8 columns][64 channels + 4]: the pad spreads
    static constexpr int d_rp = 2 * kStCols * d_px;                      //   the copies of 8 columns x 4 channels over all banks
    static constexpr int d_stage = kFgRowPairs * d_rp;
    static constexpr int smem_bytes = 2 * (x_stage + d_stage) * 4;
    static constexpr int xpos = kFgRowPairs * RR * xpitch;               // input positions per channel and stage
};

template <int K>
__global__ void __launch_bounds__(kStThreads, 2) filter_grad_rows_kernel(const __grid_constant__ FilterGradRowsArgs A)
{
    using G = FgGeom<K>;
    extern __shared__ __align__(16) float st_smem[];
    constexpr int KK = K * K, P = G::P, RR = G::RR;
    const int tid = threadIdx.x, lane = tid & 31, cg = tid >> 5;
    const int split = blockIdx.x % A.splits;
    const int ci_t = (blockIdx.x / A.splits) % A.ci_tiles;
    const int co_t = blockIdx.x / (A.splits * A.ci_tiles);
    const int co0 = co_t * kFgCo, ci0 = ci_t * kFgCi;
    const int s_lo = (int)((long long)split * A.stages / A.splits), s_hi = (int)((long long)(split + 1) * A.stages / A.splits);
    float* sx = st_smem;                       // two input stages
    float* sd = st_smem + 2 * G::x_stage;      // two delta stages
    const size_t plane = (size_t)A.H * A.W;

    // what this thread copies in every stage: one position of the input window (threads 0 .. xpos - 1, all 32
    // channels of it), and of the delta the column `dcol` of its warp's row for the channels dco, dco + 4, ...
    const int xe = tid < G::xpos ? tid : 0;
    const int xc = xe % G::xpitch, xr = (xe / G::xpitch) % RR, xrl = xe / (G::xpitch * RR);
    const int dcol = tid & 7, dco = (tid >> 3) & 3, dq = tid >> 5;       // warp dq copies row (dq >> 1, dq & 1): 8 columns x 4 channels at a time
    auto load_stage = [&](int s) {
        const int rt = s / A.x_tiles, xt = s - rt * A.x_tiles;
        const int rp0 = rt * kFgRowPairs, x0 = xt * kStCols;
        float* dx = sx + (s & 1) * G::x_stage;
        float* dd = sd + (s & 1) * G::d_stage;
        if (tid < G::xpos) {
            const int rp = rp0 + xrl, n = rp / A.rp_img, y = (rp - n * A.rp_img) * 2 + xr - P, x = x0 + xc - P;
            const bool ok = n < A.N && y >= 0 && y < A.H && x >= 0 && x < A.W;
            const float* src = ok ? A.x + ((size_t)n * A.Cin + ci0) * plane + (size_t)y * A.W + x : A.x;
            float* dst = dx + xe;
#pragma unroll 4
            for (int ci = 0; ci < kFgCi; ++ci) {
                const bool okc = ok && ci0 + ci < A.Cin;
                st_cp_async4(dst + ci * G::x_cs, okc ? src + (size_t)ci * plane : A.x, okc);
            }
        }
        {
            const int rp = rp0 + (dq >> 1), n = rp / A.rp_img, y = (rp - n * A.rp_img) * 2 + (dq & 1), x = x0 + dcol;
            const bool ok = n < A.N && y < A.H && x < A.W;
            const float* src = ok ? A.dz + ((size_t)n * A.Cout + co0) * plane + (size_t)y * A.W + x : A.dz;
            float* dst = dd + (dq * kStCols + dcol) * G::d_px;
#pragma unroll 4
            for (int co = dco; co < kFgCo; co += 4) {
                const bool okc = ok && co0 + co < A.Cout;
                st_cp_async4(dst + co, okc ? src + (size_t)co * plane : A.dz, okc);
            }
        }
        st_commit();
    };

    float2 acc[4][KK];                         // (channel 2c, channel 2c + 1) of the thread's eight
    float2 bsum[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        bsum[c] = make_float2(0.f, 0.f);
#pragma unroll
        for (int t = 0; t < KK; ++t) acc[c][t] = make_float2(0.f, 0.f);
    }
    const bool with_bias = ci_t == 0;          // one input-channel slice also sums the delta itself: the bias gradient

    if (s_lo < s_hi) load_stage(s_lo);
    for (int s = s_lo; s < s_hi; ++s) {
        st_wait<0>();
        __syncthreads();                      // also the release of the other buffer, which the next copies fill
        if (s + 1 < s_hi) load_stage(s + 1);
        const float* xb = sx + (s & 1) * G::x_stage + lane * G::x_cs;
        const float* db = sd + (s & 1) * G::d_stage + cg * 8;
#pragma unroll 1
        for (int rl = 0; rl < kFgRowPairs; ++rl)
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                float w[RR][4 + 2 * P];
#pragma unroll
                for (int r = 0; r < RR; ++r)
#pragma unroll
                    for (int c = 0; c < 4 + 2 * P; ++c) w[r][c] = xb[rl * G::x_rp + r * G::xpitch + 4 * q + c];
#pragma unroll
                for (int p = 0; p < 2; ++p)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float* dp = db + rl * G::d_rp + (p * kStCols + 4 * q + j) * G::d_px;
                        const float4 da = *reinterpret_cast<const float4*>(dp);
                        const float4 dq4 = *reinterpret_cast<const float4*>(dp + 4);
                        const float2 d[4] = {make_float2(da.x, da.y), make_float2(da.z, da.w), make_float2(dq4.x, dq4.y), make_float2(dq4.z, dq4.w)};
                        if (with_bias) {
#pragma unroll
                            for (int c = 0; c < 4; ++c) bsum[c] = __fadd2_rn(bsum[c], d[c]);
                        }
#pragma unroll
                        for (int ky = 0; ky < K; ++ky)
#pragma unroll
                            for (int kx = 0; kx < K; ++kx) {
                                const float2 ww = make_float2(w[p + ky][j + kx], w[p + ky][j + kx]);
#pragma unroll
                                for (int c = 0; c < 4; ++c) acc[c][ky * K + kx] = __ffma2_rn(d[c], ww, acc[c][ky * K + kx]);
                            }
                    }
            }
    }

    float* set = A.partial + (size_t)split * A.set_floats;
    const int ci = ci0 + lane;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const int co = co0 + cg * 8 + c;
        if (co >= A.Cout) break;
        if (ci < A.Cin) {
            float* dst = set + A.filter_off + ((size_t)co * A.Cin + ci) * KK;
#pragma unroll
            for (int t = 0; t < KK; ++t) dst[t] = (c & 1) ? acc[c >> 1][t].y : acc[c >> 1][t].x;
        }
        if (with_bias && lane == 0) set[A.bias_off + co] = (c & 1) ? bsum[c >> 1].y : bsum[c >> 1].x;
    }
}

// ---------------------------------------------------------------------------------------------
// Filter gradient of a 1 x 1 conv: a plain contraction over pixels, dW[co][ci] = sum_p dZ[co][p] X[ci][p].
// Block: 64 output x 128 input channels; thread: 4 output x 8 input channels (two groups of four, 64
// channels apart, so that the 16 lanes that differ in input channels read consecutive 16-byte pieces).
// A stage is 32 consecutive pixels of one image, kept in shared memory pixel-major ([pixel][channel],
// padded by 4) for both operands; the sums of two neighbouring input channels share a register pair.
// ---------------------------------------------------------------------------------------------
constexpr int kF1Co = kFg1Co, kF1Ci = kFg1Ci, kF1Px = kFg1Px;
constexpr int kF1Ds = kF1Co + 4, kF1Xs = kF1Ci + 4;                     // floats per pixel of the delta / input stage
constexpr int kF1Stage = kF1Px * (kF1Ds + kF1Xs);                       // floats
constexpr int kF1SmemBytes = 2 * kF1Stage * 4;

__global__ void __launch_bounds__(kStThreads, 3) filter_grad_1x1_kernel(const __grid_constant__ FilterGradRowsArgs A)
{
    extern __shared__ __align__(16) float st_smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int cig = tid & 15, cog = tid >> 4;              // a warp: 16 input-channel groups x 2 output-channel groups
    const int split = blockIdx.x % A.splits;
    const int ci_t = (blockIdx.x / A.splits) % A.ci_tiles;
    const int co_t = blockIdx.x / (A.splits * A.ci_tiles);
    const int co0 = co_t * kF1Co, ci0 = ci_t * kF1Ci;
    const int HW = A.H * A.W, per_img = (HW + kF1Px - 1) / kF1Px;     // stages = N * per_img (A.stages)
    const int s_lo = (int)((long long)split * A.stages / A.splits), s_hi = (int)((long long)(split + 1) * A.stages / A.splits);

    // copies: a warp takes 8 pixels x 4 channels at a time (conflict-free with the padded pixel stride)
    const int cpx = lane & 7, cch = lane >> 3, cw = tid >> 5;
    auto load_stage = [&](int s) {
        const int n = s / per_img, p0 = (s - n * per_img) * kF1Px;
        float* sd = st_smem + (s & 1) * kF1Stage;
        float* sx = sd + kF1Px * kF1Ds;
        const float* dsrc = A.dz + ((size_t)n * A.Cout + co0) * HW + p0;
        const float* xsrc = A.x + ((size_t)n * A.Cin + ci0) * HW + p0;
        // tasks: (pixel octet q of 4) x (channel quad): delta 4 x 16, input 4 x 32
        for (int t = cw; t < 4 * (kF1Co / 4); t += kStThreads / 32) {
            const int q = t & 3, ch = (t >> 2) * 4 + cch, p = q * 8 + cpx;
            const bool ok = p0 + p < HW && co0 + ch < A.Cout;
            st_cp_async4(sd + p * kF1Ds + ch, ok ? dsrc + (size_t)ch * HW + p : A.dz, ok);
        }
        for (int t = cw; t < 4 * (kF1Ci / 4); t += kStThreads / 32) {
            const int q = t & 3, ch = (t >> 2) * 4 + cch, p = q * 8 + cpx;
            const bool ok = p0 + p < HW && ci0 + ch < A.Cin;
            st_cp_async4(sx + p * kF1Xs + ch, ok ? xsrc + (size_t)ch * HW + p : A.x, ok);
        }
        st_commit();
    };

    float2 acc[4][4];                          // [output channel][pair of input channels]
    float bsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[c][i] = make_float2(0.f, 0.f);
    const bool with_bias = ci_t == 0 && cig == 0;

    if (s_lo < s_hi) load_stage(s_lo);
    for (int s = s_lo; s < s_hi; ++s) {
        st_wait<0>();
        __syncthreads();                      // also the release of the other buffer, which the next copies fill
        if (s + 1 < s_hi) load_stage(s + 1);
        const float* dp = st_smem + (s & 1) * kF1Stage + cog * 4;
        const float* xp = st_smem + (s & 1) * kF1Stage + kF1Px * kF1Ds + cig * 4;
#pragma unroll 4
        for (int p = 0; p < kF1Px; ++p) {
            const float4 d = *reinterpret_cast<const float4*>(dp + p * kF1Ds);
            const float4 xa = *reinterpret_cast<const float4*>(xp + p * kF1Xs);
            const float4 xb = *reinterpret_cast<const float4*>(xp + p * kF1Xs + 64);
            const float2 xv[4] = {make_float2(xa.x, xa.y), make_float2(xa.z, xa.w), make_float2(xb.x, xb.y), make_float2(xb.z, xb.w)};
            const float dv[4] = {d.x, d.y, d.z, d.w};
            if (with_bias) { bsum[0] += d.x; bsum[1] += d.y; bsum[2] += d.z; bsum[3] += d.w; }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float2 dd = make_float2(dv[c], dv[c]);
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[c][i] = __ffma2_rn(dd, xv[i], acc[c][i]);
            }
        }
    }

    float* set = A.partial + (size_t)split * A.set_floats;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int co = co0 + cog * 4 + c;
        if (co >= A.Cout) break;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int ci = ci0 + cig * 4 + (i >> 1) * 64 + (i & 1) * 2;
            float* dst = set + A.filter_off + (size_t)co * A.Cin + ci;
            if (ci < A.Cin) dst[0] = acc[c][i].x;
            if (ci + 1 < A.Cin) dst[1] = acc[c][i].y;
        }
        if (with_bias) set[A.bias_off + co] = bsum[c];
    }
}

// ---------------------------------------------------------------------------------------------
// dZ = dY * leaky'(Y) at the conv's resolution.  pool == 0: Y is the layer's output map, element by
// element.  pool != 0: dY and Y are the pooled maps; each pooled delta goes to the arg-max position
// of its 2x2 window and the other three positions get zero.
// ---------------------------------------------------------------------------------------------
__global__ void delta_act_kernel(const float* __restrict__ dy, const float* __restrict__ y, const unsigned char* __restrict__ arg,
                                 float* __restrict__ dz, size_t count /*elements of dy*/, int OW /*pooled width*/, float slope, int pool)
{
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x) {
        const float v = dy[e] * (y[e] > 0.f ? 1.f : slope);
        if (!pool) { dz[e] = v; continue; }
        const size_t row = e / OW; const int px = (int)(e - row * OW);
        const int am = arg[e];
        float* o = dz + (row * 2) * (size_t)(2 * OW) + 2 * px;
        *reinterpret_cast<float2*>(o) = make_float2(am == 0 ? v : 0.f, am == 1 ? v : 0.f);
        *reinterpret_cast<float2*>(o + 2 * OW) = make_float2(am == 2 ? v : 0.f, am == 3 ? v : 0.f);
    }
}

}  // namespace ftp

namespace ftp {

// ---------------------------------------------------------------------------------------------
// Backward of a thin-input conv3x3 + 2x2 max-pool group (at most 4 input and 32 output channels: the
// first layer of an image network).  The pooled delta is sparse at the conv's resolution -- one
// non-zero per 2x2 window, at the arg-max -- so the delta in front of the activation is never laid
// out in global memory: a block stages, for a tile of 8 x 32 pooled pixels and a ring of one pooled
// pixel around it, v = dY * leaky'(Y) and the arg-max of every output channel, plus the input patch
// under it, and then
//   filter gradient: lane = output channel; per pooled pixel the 3 x 3 x Cin input values around that
//     channel's arg-max position meet v (27 multiply-adds instead of the 108 of the zero-extended
//     delta); the warps of a block take the pixels of a tile in turn, and the block's sums over all its
//     tiles form one partial gradient set (Section 4.1);
//   input delta: thread = pooled pixel, i.e. 2 x 2 input pixels x Cin channels; per output channel
//     the 4 x 4 neighbourhood of the zero-extended delta is rebuilt from the nine surrounding pooled
//     values and meets the filter (correlation with the 180-degree-rotated filter written out as a
//     gather, Section 4.1).
// ---------------------------------------------------------------------------------------------
constexpr int kThinTH = kThinTileH, kThinTW = kThinTileW;   // pooled pixels per tile
constexpr int kThinPH = kThinTH + 2, kThinPW = kThinTW + 2;
constexpr int kThinVs = 33, kThinAs = 36;             // strides of the staged v (floats) and arg-max (bytes) per pooled pixel
constexpr int kThinXH = 2 * kThinTH + 2, kThinXW = 2 * kThinTW + 2, kThinXP = kThinXW + 1;   // input patch; odd pitch
constexpr int kThinMaxCin = 4, kThinMaxCout = 32;
constexpr int kThinSmemV = kThinPH * kThinPW * kThinVs;                  // floats
constexpr int kThinSmemX = kThinMaxCin * kThinXH * kThinXP;              // floats
constexpr int kThinSmemW = kThinMaxCout * 9 * 4;                         // floats: [co][tap][ci padded to 4]
constexpr int kThinSmemBytes = (kThinSmemV + kThinSmemX + kThinSmemW) * 4 + kThinPH * kThinPW * kThinAs;

template <int CIN>
__global__ void __launch_bounds__(kStThreads, 2) thin_bwd_kernel(const __grid_constant__ ThinBwdArgs A)
{
    extern __shared__ __align__(16) float st_smem[];
    float* sv = st_smem;                                   // [pooled pixel][33]: v per output channel
    float* sx = sv + kThinSmemV;                           // [ci][row][col]: input patch, global row 2 py0 - 1 at row 0
    float* swt = sx + kThinSmemX;                          // [co][tap][4]
    unsigned char* sa = reinterpret_cast<unsigned char*>(swt + kThinSmemW);   // [pooled pixel][36]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = 2 * A.OH, W = 2 * A.OW;
    const size_t pplane = (size_t)A.OH * A.OW, plane = (size_t)H * W;

    for (int i = tid; i < kThinMaxCout * 9 * 4; i += kStThreads) {
        const int ci = i & 3, tap = (i >> 2) % 9, co = i / 36;
        swt[i] = (co < A.Cout && ci < CIN) ? __ldg(A.filter + ((size_t)co * CIN + ci) * 9 + tap) : 0.f;
    }
    float acc[CIN][9];                                     // filter gradient of (output channel = lane, input channel, tap)
    float bsum = 0.f;
#pragma unroll
    for (int ci = 0; ci < CIN; ++ci)
#pragma unroll
        for (int t = 0; t < 9; ++t) acc[ci][t] = 0.f;

    const int tiles_img = A.tiles_y * A.tiles_x, tiles = A.N * tiles_img;
    const int t_lo = (int)((long long)blockIdx.x * tiles / gridDim.x), t_hi = (int)((long long)(blockIdx.x + 1) * tiles / gridDim.x);
    for (int tile = t_lo; tile < t_hi; ++tile) {
        const int n = tile / tiles_img, ty = (tile % tiles_img) / A.tiles_x, tx = tile % A.tiles_x;
        const int py0 = ty * kThinTH, px0 = tx * kThinTW;
        __syncthreads();                                   // the previous tile has been consumed
        // stage v and arg-max: one warp per output channel at a time, lanes along the 10 x 34 pooled pixels of the tile
        for (int co = warp; co < A.Cout; co += kStThreads / 32) {
            const size_t base = ((size_t)n * A.Cout + co) * pplane;
            // (all loads of a channel are issued before the first value is used: the loop is unrolled whole)
            constexpr int kIt = (kThinPH * kThinPW + 31) / 32;
            float dv[kIt], yv[kIt]; unsigned char av[kIt];
#pragma unroll
            for (int it = 0; it < kIt; ++it) {
                const int e = lane + 32 * it;
                const int ly = e / kThinPW, lx = e - ly * kThinPW;
                const int py = py0 + ly - 1, px = px0 + lx - 1;
                dv[it] = 0.f; yv[it] = 0.f; av[it] = 0;
                if (e < kThinPH * kThinPW && py >= 0 && py < A.OH && px >= 0 && px < A.OW) {
                    const size_t gi = base + (size_t)py * A.OW + px;
                    dv[it] = __ldg(A.dyp + gi); yv[it] = __ldg(A.yp + gi); av[it] = __ldg(A.arg + gi);
                }
            }
#pragma unroll
            for (int it = 0; it < kIt; ++it) {
                const int e = lane + 32 * it;
                if (e < kThinPH * kThinPW) {
                    sv[e * kThinVs + co] = dv[it] * (yv[it] > 0.f ? 1.f : A.slope);
                    sa[e * kThinAs + co] = av[it];
                }
            }
        }
        // stage the input patch
        for (int r = warp; r < CIN * kThinXH; r += kStThreads / 32) {
            const int ci = r / kThinXH, lr = r - ci * kThinXH, y = 2 * py0 - 1 + lr;
            const bool row_ok = y >= 0 && y < H;
            const float* src = A.x + ((size_t)n * CIN + ci) * plane + (size_t)(row_ok ? y : 0) * W;
            for (int lc = lane; lc < kThinXW; lc += 32) {
                const int xg = 2 * px0 - 1 + lc;
                sx[(ci * kThinXH + lr) * kThinXP + lc] = (row_ok && xg >= 0 && xg < W) ? __ldg(src + xg) : 0.f;
            }
        }
        __syncthreads();

        // filter gradient: lane = output channel, the warps take the tile's pooled pixels in turn
        if (lane < A.Cout) {
            for (int p = warp; p < kThinTH * kThinTW; p += kStThreads / 32) {
                const int wy = p >> 5, wx = p & 31;
                const int pi = (wy + 1) * kThinPW + wx + 1;
                const float v = sv[pi * kThinVs + lane];
                const int a = sa[pi * kThinAs + lane];
                bsum += v;
                // input position of tap (0, 0): rows 2 wy + ay (+ ky), columns 2 wx + ax (+ kx) of the patch
                const float* xp = sx + (2 * wy + (a >> 1)) * kThinXP + 2 * wx + (a & 1);
#pragma unroll
                for (int ci = 0; ci < CIN; ++ci)
#pragma unroll
                    for (int ky = 0; ky < 3; ++ky)
#pragma unroll
                        for (int kx = 0; kx < 3; ++kx)
                            acc[ci][ky * 3 + kx] = fmaf(v, xp[(ci * kThinXH + ky) * kThinXP + kx], acc[ci][ky * 3 + kx]);
            }
        }

        // input delta: thread = pooled pixel (wy, wx) = 2 x 2 input pixels
        if (A.dx) {
            const int wy = tid >> 5, wx = tid & 31;
            float o[CIN][2][2];
#pragma unroll
            for (int ci = 0; ci < CIN; ++ci) o[ci][0][0] = o[ci][0][1] = o[ci][1][0] = o[ci][1][1] = 0.f;
#pragma unroll 2
            for (int co = 0; co < A.Cout; ++co) {
                // the nine pooled values around the pixel and their arg-max
                float v9[3][3]; int a9[3][3];
#pragma unroll
                for (int dy = 0; dy < 3; ++dy)
#pragma unroll
                    for (int dx = 0; dx < 3; ++dx) {
                        const int pi = (wy + dy) * kThinPW + wx + dx;
                        v9[dy][dx] = sv[pi * kThinVs + co];
                        a9[dy][dx] = sa[pi * kThinAs + co];
                    }
                // zero-extended delta on rows 2 py - 1 .. 2 py + 2, columns 2 px - 1 .. 2 px + 2
                float dz[4][4];
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int wr = (r + 1) >> 1, wc = (c + 1) >> 1;              // 0, 1, 1, 2
                        const int want = (((r + 1) & 1) << 1) | ((c + 1) & 1);       // arg-max that puts the value there
                        dz[r][c] = a9[wr][wc] == want ? v9[wr][wc] : 0.f;
                    }
#pragma unroll
                for (int ky = 0; ky < 3; ++ky)
#pragma unroll
                    for (int kx = 0; kx < 3; ++kx) {
                        const float4 wv = *reinterpret_cast<const float4*>(swt + (co * 9 + ky * 3 + kx) * 4);
                        const float wc4[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                        for (int i = 0; i < 2; ++i)
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                const float d = dz[i - ky + 2][j - kx + 2];
#pragma unroll
                                for (int ci = 0; ci < CIN; ++ci) o[ci][i][j] = fmaf(wc4[ci], d, o[ci][i][j]);
                            }
                    }
            }
            const int py = py0 + wy, px = px0 + wx;
            if (py < A.OH && px < A.OW) {
#pragma unroll
                for (int ci = 0; ci < CIN; ++ci) {
                    float* dst = A.dx + ((size_t)n * CIN + ci) * plane + (size_t)(2 * py) * W + 2 * px;
                    *reinterpret_cast<float2*>(dst) = make_float2(o[ci][0][0], o[ci][0][1]);
                    *reinterpret_cast<float2*>(dst + W) = make_float2(o[ci][1][0], o[ci][1][1]);
                }
            }
        }
    }

    // the block's partial set: the eight warps' sums per (output channel, input channel, tap), added in warp order
    __syncthreads();
    float* red = st_smem;                                  // [warp][lane][40]
    {
        float* mine = red + (warp * 32 + lane) * 40;
#pragma unroll
        for (int ci = 0; ci < CIN; ++ci)
#pragma unroll
            for (int t = 0; t < 9; ++t) mine[ci * 9 + t] = acc[ci][t];
        mine[36] = bsum;
    }
    __syncthreads();
    float* set = A.partial + (size_t)blockIdx.x * A.set_floats;
    for (int e = tid; e < A.Cout * 37; e += kStThreads) {
        const int co = e / 37, k = e - co * 37;
        if (k < 36 && k >= CIN * 9) continue;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kStThreads / 32; ++w) s += red[(w * 32 + co) * 40 + k];
        if (k == 36) set[A.bias_off + co] = s;
        else set[A.filter_off + ((size_t)co * CIN + k / 9) * 9 + k % 9] = s;
    }
}

}  // namespace ftp
