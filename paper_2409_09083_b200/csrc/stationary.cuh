// Weight-stationary kernels of the fp32 path for executed groups that hold one conv layer
// (optionally with the 2x2 max-pool after it).  The paper leaves weight-dominated layers to a
// weight partitioning it names as future work (Section 6); here such a layer is cut along its
// output channels and its pixels instead of into fused stacks: a block keeps a slice of the filter
// (forward, input delta) or of the filter gradient (Section 4.1: feature-map tile convolved with the
// delta tile) on chip and streams pixel tiles through it.
//
//   conv_rows_kernel   out = conv(in, w) (+ bias, leaky ReLU, optional fused 2x2 max-pool with arg-max):
//                      the forward convolution and, with the rotated filters, the input delta
//   filter_grad_rows_kernel   partial filter and bias gradients of a slice of (output, input) channels
//                      over a share of the pixels; the shares are summed by the cross-tile reduction
//   delta_act_kernel   the delta in front of the activation, dZ = dY * leaky'(Y), at the conv's
//                      resolution (routed through the arg-max where a pool follows)
//
// Thread tile of the convolution: 8 output channels x (2 rows x 4 columns).  Rows are taken in
// pairs over the whole batch (image after image), so a tile of row pairs may span images and no
// rows are wasted on maps whose height is not a multiple of the tile; every row pair keeps its own
// four input rows in shared memory.  Each output value is accumulated over input channels in
// ascending order and, per channel, over the window columns and then rows, the order of the fused
// stack kernels, so both give the same bits.
#pragma once

#include <cuda_runtime.h>

namespace ftp {

struct ConvRowsArgs {
    const float* in;        // [N][Cin][H][W]
    const float* w;         // [Cin][K*K][CoutPad]: tap-major slices of 8-padded output channels
    const float* bias;      // [Cout] or null
    float* out;             // [N][Cout][H][W], or the pooled map [N][Cout][H/2][W/2] when pool != 0
    unsigned char* arg;     // pool: arg-max (dy * 2 + dx, first maximum in row-major order) per pooled value
    int N, Cin, Cout, CoutPad, H, W;
    float slope;            // leaky-ReLU slope; act == 0: no bias, no activation (input delta)
    int act, pool;
    int co_tile;            // output channels per block (multiple of 8)
    int prp, pcq;           // row pairs and column quads per block: (co_tile / 8) * prp * pcq threads
    int ci_chunk;           // input channels per shared-memory stage
    int rp_img;             // row pairs per image = ceil(H / 2)
    int x_tiles, co_tiles;  // blockIdx.x = (rp_tile * x_tiles + x_tile) * co_tiles + co_tile
    int in_pitch, rp_stride, ci_stride;   // shared-memory geometry of an input stage, in floats
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
__device__ __forceinline__ void st_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void st_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

constexpr int kStMaxPos = 6;   // input positions (row, column of a stage) a thread copies per channel

// K = 1 or 3 (stride 1, padding K/2).
template <int K>
__global__ void __launch_bounds__(256, 2) conv_rows_kernel(const __grid_constant__ ConvRowsArgs A)
{
    extern __shared__ __align__(16) float st_smem[];
    constexpr int KK = K * K, P = K / 2;
    constexpr int RR = K + 1;                      // input rows of a row pair
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int npg = A.prp * A.pcq;
    const int cg = tid / npg, pg = tid - cg * npg;
    const int rp_l = pg / A.pcq, cq_l = pg - rp_l * A.pcq;
    const int co_t = blockIdx.x % A.co_tiles;
    const int xt = (blockIdx.x / A.co_tiles) % A.x_tiles;
    const int rt = blockIdx.x / (A.co_tiles * A.x_tiles);
    const int co0 = co_t * A.co_tile, x0 = xt * A.pcq * 4, rp0 = rt * A.prp;
    const int TW = A.pcq * 4;
    const int w_stage = A.ci_chunk * KK * A.co_tile;            // floats
    const int in_stage = A.ci_chunk * A.ci_stride;
    float* sw = st_smem;                                        // two weight stages
    float* si = st_smem + 2 * w_stage;                          // two input stages
    const size_t plane = (size_t)A.H * A.W;

    // input positions this thread copies in every stage: (row pair, row, column) -> shared / global offsets
    int pos_s[kStMaxPos]; long long pos_g[kStMaxPos]; unsigned pos_ok = 0;
    const int cols = TW + 2 * P, npos = A.prp * RR * cols;
#pragma unroll
    for (int e = 0; e < kStMaxPos; ++e) {
        const int idx = tid + e * nthreads;
        pos_s[e] = -1; pos_g[e] = 0;
        if (idx < npos) {
            const int c = idx % cols, t = idx / cols, r = t % RR, rl = t / RR;
            const int rp = rp0 + rl;
            const int n = rp / A.rp_img, y = (rp - n * A.rp_img) * 2 + r - P, x = x0 + c - P;
            pos_s[e] = rl * A.rp_stride + r * A.in_pitch + c + (4 - P);
            if (n < A.N && y >= 0 && y < A.H && x >= 0 && x < A.W) {
                pos_ok |= 1u << e;
                pos_g[e] = (long long)n * A.Cin * plane + (long long)y * A.W + x;
            }
        }
    }
    auto load_stage = [&](int chunk) {
        const int ci0 = chunk * A.ci_chunk, nci = min(A.ci_chunk, A.Cin - ci0);
        float* dw = sw + (chunk & 1) * w_stage;
        float* di = si + (chunk & 1) * in_stage;
        // filters: rows of co_tile floats per (channel, tap)
        const int q = A.co_tile / 4, n16 = nci * KK * q;
        for (int i = tid; i < n16; i += nthreads) {
            const int row = i / q, j = i - row * q;
            const int co = co0 + 4 * j;
            st_cp_async16(dw + row * A.co_tile + 4 * j, A.w + ((size_t)ci0 * KK + row) * A.CoutPad + min(co, A.CoutPad - 4), co < A.CoutPad);
        }
#pragma unroll
        for (int e = 0; e < kStMaxPos; ++e)
            if (pos_s[e] >= 0) {
                const bool ok = (pos_ok >> e) & 1u;
                const float* src = A.in + pos_g[e] + (size_t)ci0 * plane;
                float* dst = di + pos_s[e];
                for (int ci = 0; ci < nci; ++ci) st_cp_async4(dst + ci * A.ci_stride, src + (size_t)ci * plane, ok);
            }
        st_commit();
    };

    float acc[2][4][8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const float b = (A.bias != nullptr && co0 + cg * 8 + c < A.Cout) ? __ldg(A.bias + co0 + cg * 8 + c) : 0.f;
#pragma unroll
        for (int p = 0; p < 2; ++p)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[p][j][c] = b;
    }

    const int nchunks = (A.Cin + A.ci_chunk - 1) / A.ci_chunk;
    const int my_in = rp_l * A.rp_stride + cq_l * 4 + 4;        // column 0 of this thread's quad (16-byte aligned)
    load_stage(0);
    for (int chunk = 0; chunk < nchunks; ++chunk) {
        if (chunk + 1 < nchunks) { load_stage(chunk + 1); st_wait<1>(); } else st_wait<0>();
        __syncthreads();
        const int nci = min(A.ci_chunk, A.Cin - chunk * A.ci_chunk);
        const float* wb = sw + (chunk & 1) * w_stage + cg * 8;
        const float* ib = si + (chunk & 1) * in_stage + my_in;
        for (int ci = 0; ci < nci; ++ci) {
            float v[RR][4 + 2 * P];
            const float* ip = ib + ci * A.ci_stride;
#pragma unroll
            for (int r = 0; r < RR; ++r) {
                const float4 m = *reinterpret_cast<const float4*>(ip + r * A.in_pitch);
                if constexpr (P > 0) v[r][0] = ip[r * A.in_pitch - 1];
                v[r][P] = m.x; v[r][P + 1] = m.y; v[r][P + 2] = m.z; v[r][P + 3] = m.w;
                if constexpr (P > 0) v[r][3 + 2 * P] = ip[r * A.in_pitch + 4];
            }
            const float* wc = wb + ci * KK * A.co_tile;
#pragma unroll
            for (int kx = 0; kx < K; ++kx)
#pragma unroll
                for (int ky = 0; ky < K; ++ky) {
                    const float4 wa = *reinterpret_cast<const float4*>(wc + (ky * K + kx) * A.co_tile);
                    const float4 wq = *reinterpret_cast<const float4*>(wc + (ky * K + kx) * A.co_tile + 4);
                    const float wv[8] = {wa.x, wa.y, wa.z, wa.w, wq.x, wq.y, wq.z, wq.w};
#pragma unroll
                    for (int p = 0; p < 2; ++p)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int c = 0; c < 8; ++c) acc[p][j][c] = fmaf(v[p + ky][j + kx], wv[c], acc[p][j][c]);
                }
        }
        __syncthreads();
    }

    // epilogue
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
                for (int j = 0; j < 4; ++j) { const float z = acc[p][j][c]; o[j] = A.act ? (z > 0.f ? z : A.slope * z) : z; }
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
                float v00 = acc[0][2 * h][c], v01 = acc[0][2 * h + 1][c], v10 = acc[1][2 * h][c], v11 = acc[1][2 * h + 1][c];
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

}  // namespace ftp
