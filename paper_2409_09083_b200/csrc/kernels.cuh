// Device code of the fused tile-stack kernels (fp32 path, CUDA cores).
//
// One thread block runs one sub-tile stack: every map of the group it touches lives in shared
// memory as [channel][row][col] planes; only the group input is read from HBM and only the owned
// cells of the layer outputs are written back (forward), resp. the saved layer outputs are read
// and the group-input delta contributions are written (backward).
#pragma once

#include <cuda_runtime.h>

#include "plan.hpp"

namespace ftp {

struct GroupArgs {
    int n_ops, R, Q, N;
    OpDesc op[kMaxOps];
    const float* map[kMaxOps + 1];     // map[0] = group input X_s, map[m] = output of op m-1
    float*       map_out[kMaxOps + 1]; // forward: writable aliases of map[1..]
    unsigned char* arg[kMaxOps];       // arg-max bytes of op i's pooled output map (fused conv+pool), else null
    const int *yspan, *xspan, *ycell, *xcell;
    const float* wpk;                  // packed filters (forward layout or rotated layout)
    const float* params;               // raw parameters (biases are read from here)
    // backward only
    const float* dmap_out;             // delta at the group's output map
    float*       scratch;              // per-sub-tile deltas at the group's input map
    const int *yoff, *xoff, *ytile, *xtile;
    float*       partial;              // [blocks][param_floats] partial gradient sets of this group
    long long    param_floats;
    int need_dx;
};

struct HaloSumArgs {
    const float* scratch; float* out;
    const int *yspan, *xspan, *yoff, *xoff, *ycover, *xcover;
    int N, C, H, W, R, Q, Htot, Wtot;
};

struct PackLayer { long long p_off, wf_off, wb_off; int cin, cout, k, cout_pad, cin_pad; };
struct PackArgs { int n; PackLayer l[kMaxOps * 2]; };

struct ReduceGroup { long long begin, floats; const float* partial; int sets; };
struct ReduceArgs { int n; ReduceGroup g[64]; };

__device__ __forceinline__ float leaky(float z, float slope) { return z > 0.f ? z : slope * z; }
// derivative of the leaky ReLU, decided from the activation's output (same sign as its input)
__device__ __forceinline__ float dleaky(float y, float slope) { return y > 0.f ? 1.f : slope; }

// Per-block header in shared memory: for every map m of the group the clamped span and the owned
// cell of this sub-tile: hdr[m*8 + {y1,y2,x1,x2, cy1,cy2,cx1,cx2}].
__device__ __forceinline__ void load_header(int* hdr, const GroupArgs& A, int r, int q, bool cells)
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

// Copy the part of a global NCHW map that an op reads into its shared-memory input buffer.
// The buffer's (0,0) is map position (oy, ox); positions outside the map are zero padding.
__device__ __forceinline__ void load_input(float* buf, int cs, int pitch, int bh, int bw, int C,
                                           const float* __restrict__ src, int n, int H, int W, int oy, int ox)
{
    if (bw < 24) {
        // narrow buffers: one element per thread and turn, whatever row it is in
        const int total = C * bh * bw;
        for (int e = threadIdx.x; e < total; e += blockDim.x) {
            int xx = e % bw, t = e / bw, yy = t % bh, c = t / bh;
            int gy = oy + yy, gx = ox + xx;
            float v = 0.f;
            if (gy >= 0 && gy < H && gx >= 0 && gx < W) v = __ldg(src + (((size_t)n * C + c) * H + gy) * W + gx);
            buf[c * cs + yy * pitch + xx] = v;
        }
        return;
    }
    // one warp per buffer row (c, yy), lanes along the row: coalesced reads and no division per
    // element; four rows are in flight per warp so that their loads overlap
    constexpr int U = 4;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int rows = C * bh;
    const float* img = src + (size_t)n * C * H * W;
    for (int r0 = warp * U; r0 < rows; r0 += nwarps * U) {
        const float* s[U]; float* d[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int r = min(r0 + u, rows - 1);
            const int c = r / bh, yy = r - c * bh, gy = oy + yy;
            d[u] = r0 + u < rows ? buf + c * cs + yy * pitch : nullptr;
            s[u] = (gy >= 0 && gy < H) ? img + ((size_t)c * H + gy) * W + ox : nullptr;
        }
        for (int xx = lane; xx < bw; xx += 32) {
            const bool in = ox + xx >= 0 && ox + xx < W;
            float v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) v[u] = (in && s[u]) ? __ldg(s[u] + xx) : 0.f;
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (d[u]) d[u][xx] = v[u];
        }
    }
}

// Zero everything of a [C][bh][bw] buffer outside the rectangle [y0,y1] x [x0,x1] (local coords).
__device__ __forceinline__ void zero_apron(float* buf, int cs, int pitch, int bh, int bw, int C,
                                           int y0, int y1, int x0, int x1)
{
    if (y0 == 0 && x0 == 0 && y1 == bh - 1 && x1 == bw - 1) return;
    const int total = C * bh * bw;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        int xx = e % bw, t = e / bw, yy = t % bh, c = t / bh;
        if (yy < y0 || yy > y1 || xx < x0 || xx > x1) buf[c * cs + yy * pitch + xx] = 0.f;
    }
}

// 16-byte asynchronous copy from global to shared memory (both 16-byte aligned), and its group bookkeeping.
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem)
{
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

// Direct convolution on a shared-memory tile: out(c, y, x) = init(c) + sum_{ci,ky,kx}
// w[ci][ky*K+kx][c] * in[ci][y+ky][x+kx] for y < oh, x < ow, c < cout.  A thread task is 8
// output channels x 4 rows at one column; lanes walk along x, so shared-memory reads are
// conflict free and all lanes of a warp read the same filter words (broadcast).  The same
// routine serves the forward pass (filters in [cin][tap][cout] layout) and the delta
// back-propagation (rotated filters in [cout][tap][cin] layout).
//   POOL_OUT: apply leaky ReLU and a 2x2/2 max-pool to the result in registers (fused conv+pool
//     forward); the epilogue gets (c, pooled y, pooled x, max, arg) with arg = dy*2+dx of the
//     first maximum in row-major window order.  oh and ow must be even.
//   MODE kInPlain:   `in` holds every position that is read (forward: halo and padding included).
//   MODE kInChecked: `in` is an in_rows x in_cols rectangle without apron; the read position
//     (y_base + y + ky, x_base + x + kx) may fall outside it and then counts as zero (delta
//     back-propagation: y_base = offset - (K-1)).
//   MODE kInExpand:  as kInChecked, but the rectangle is virtual: `in` is the delta of a pooled map
//     with its arg-max bytes, and the un-pooled delta at (vy, vx) is in[vy/2][vx/2] if the arg-max
//     of that window is (vy%2, vx%2), else 0.  in_rows/in_cols count un-pooled positions.
//   STAGED: the filter words come from shared memory instead of global memory.  The input
//     channels are taken w_ch at a time; the block copies the filters of the next w_ch channels
//     (contiguous in both filter layouts) into one half of `wst` with cp.async while it computes on
//     the other half, so the inner loop waits on shared-memory latency only.  All threads of the
//     block must make the call (it synchronises).
enum { kInPlain = 0, kInChecked = 1, kInExpand = 2 };

template <int K, bool POOL_OUT, int MODE, bool STAGED, class Epilogue>
__device__ __forceinline__ void conv_tile(const float* __restrict__ in, const unsigned char* __restrict__ arg,
                                          int in_cs, int in_pitch, int in_rows, int in_cols, int y_base, int x_base,
                                          const float* __restrict__ w, int cin, int cout_pad,
                                          const float* __restrict__ bias, int cout, float slope,
                                          int oh, int ow, float* __restrict__ wst, int w_ch, Epilogue epi)
{
    constexpr int TP = 4, TC = kCoutTile;
    const int ncob = cout_pad / TC, nyb = (oh + TP - 1) / TP;
    const int ntasks = ncob * nyb * ow;
    for (int t0 = 0; t0 < ntasks; t0 += blockDim.x) {
        const bool active = t0 + (int)threadIdx.x < ntasks;
        const int t = active ? t0 + (int)threadIdx.x : ntasks - 1;
        const int x = t % ow, rem = t / ow, yb = rem % nyb, cob = rem / nyb;
        const int y0 = yb * TP, c0 = cob * TC;
        float acc[TP][TC];
#pragma unroll
        for (int c = 0; c < TC; ++c) {
            float b = (bias != nullptr && c0 + c < cout) ? __ldg(bias + c0 + c) : 0.f;
#pragma unroll
            for (int p = 0; p < TP; ++p) acc[p][c] = b;
        }
        int rowoff[TP + K - 1];      // offset of the row inside a channel plane
        int coloff[K];               // kInChecked / kInExpand: column offset per kx
        unsigned okmask = 0;         // bit r: row r readable; bit 16 + kx: column readable
        unsigned parmask = 0;        // kInExpand: bit r: row parity; bit 16 + kx: column parity
#pragma unroll
        for (int r = 0; r < TP + K - 1; ++r) {
            const int vy = y_base + y0 + r;
            if (MODE == kInPlain) {
                rowoff[r] = min(vy, in_rows - 1) * in_pitch + x_base + x;
            } else {
                const int cy = min(max(vy, 0), in_rows - 1);
                if (vy == cy) okmask |= 1u << r;
                if (MODE == kInExpand) { rowoff[r] = (cy >> 1) * in_pitch; parmask |= (unsigned)(cy & 1) << r; }
                else rowoff[r] = cy * in_pitch;
            }
        }
        if (MODE != kInPlain) {
#pragma unroll
            for (int kx = 0; kx < K; ++kx) {
                const int vx = x_base + x + kx;
                const int cx = min(max(vx, 0), in_cols - 1);
                if (vx == cx) okmask |= 1u << (16 + kx);
                if (MODE == kInExpand) { coloff[kx] = cx >> 1; parmask |= (unsigned)(cx & 1) << (16 + kx); }
                else coloff[kx] = cx;
            }
        }
        const int per_ci = K * K * cout_pad;                  // filter words of one input channel
        const int step = STAGED ? w_ch : cin;
        auto stage = [&](int ci0) {                            // copy of the filters of channels ci0 .. ci0 + w_ch - 1
            const int n4 = min(w_ch, cin - ci0) * per_ci / 4;
            const float4* src = reinterpret_cast<const float4*>(w + (size_t)ci0 * per_ci);
            float4* dst = reinterpret_cast<float4*>(wst + ((ci0 / w_ch) & 1) * w_ch * per_ci);
            for (int i = threadIdx.x; i < n4; i += blockDim.x) cp_async16(dst + i, src + i);
            cp_async_commit();
        };
        if (STAGED) stage(0);
        for (int cb = 0; cb < cin; cb += step) {
        const int ce = min(cin, cb + step);
        const float* wp;
        if (STAGED) {
            if (ce < cin) { stage(ce); cp_async_wait<1>(); } else cp_async_wait<0>();
            __syncthreads();
            wp = wst + ((cb / w_ch) & 1) * w_ch * per_ci + c0 - (size_t)cb * per_ci;
        } else {
            wp = w + c0;
        }
        for (int ci = cb; ci < ce; ++ci) {
            const float* ip = in + ci * in_cs;
            const unsigned char* ap = MODE == kInExpand ? arg + ci * in_cs : nullptr;
            const float* wc = wp + (size_t)ci * per_ci;
#pragma unroll
            for (int kx = 0; kx < K; ++kx) {
                float wr[K][TC];
#pragma unroll
                for (int ky = 0; ky < K; ++ky) {
                    const float4* wq = reinterpret_cast<const float4*>(wc + (ky * K + kx) * cout_pad);
                    const float4 a = STAGED ? wq[0] : __ldg(wq);
                    const float4 b = STAGED ? wq[1] : __ldg(wq + 1);
                    wr[ky][0] = a.x; wr[ky][1] = a.y; wr[ky][2] = a.z; wr[ky][3] = a.w;
                    wr[ky][4] = b.x; wr[ky][5] = b.y; wr[ky][6] = b.z; wr[ky][7] = b.w;
                }
#pragma unroll
                for (int r = 0; r < TP + K - 1; ++r) {
                    float v;
                    if (MODE == kInPlain) {
                        v = ip[rowoff[r] + kx];
                    } else {
                        const bool ok = ((okmask >> r) & (okmask >> (16 + kx)) & 1u) != 0;
                        const int idx = rowoff[r] + coloff[kx];
                        v = ip[idx];
                        if (MODE == kInExpand) {
                            const int want = (int)(((parmask >> r) & 1u) << 1 | ((parmask >> (16 + kx)) & 1u));
                            v = (ok && (int)ap[idx] == want) ? v : 0.f;
                        } else {
                            v = ok ? v : 0.f;
                        }
                    }
#pragma unroll
                    for (int ky = 0; ky < K; ++ky) {
                        const int p = r - ky;
                        if (p >= 0 && p < TP) {
#pragma unroll
                            for (int c = 0; c < TC; ++c) acc[p][c] = fmaf(v, wr[ky][c], acc[p][c]);
                        }
                    }
                }
            }
        }
        if (STAGED) __syncthreads();                           // this half of wst may be overwritten now
        }
        if (POOL_OUT) {
#pragma unroll
            for (int p = 0; p < TP; p += 2) {
#pragma unroll
                for (int c = 0; c < TC; ++c) {
                    const float v00 = leaky(acc[p][c], slope), v10 = leaky(acc[p + 1][c], slope);
                    const float v01 = __shfl_xor_sync(0xffffffffu, v00, 1);
                    const float v11 = __shfl_xor_sync(0xffffffffu, v10, 1);
                    if (active && (x & 1) == 0 && y0 + p < oh && c0 + c < cout) {
                        float best = v00; int am = 0;
                        if (v01 > best) { best = v01; am = 1; }
                        if (v10 > best) { best = v10; am = 2; }
                        if (v11 > best) { best = v11; am = 3; }
                        epi(c0 + c, (y0 + p) >> 1, x >> 1, best, am);
                    }
                }
            }
        } else if (active) {
#pragma unroll
            for (int p = 0; p < TP; ++p)
                if (y0 + p < oh) {
#pragma unroll
                    for (int c = 0; c < TC; ++c)
                        if (c0 + c < cout) epi(c0 + c, y0 + p, x, acc[p][c], 0);
                }
        }
    }
}

// Input delta of a conv (or fused conv+pool) op with the output delta staged in shared memory:
// out[c][u] = sum_{d, ky, kx} w[d][ky][kx][c] * Z[d][vy0 + uy + ky - (K-1)][vx0 + ux + kx - (K-1)]
// for the ih x iw positions u of the op's input span, where Z is the zh x zw delta at the conv
// output (zero outside) and w the rotated filter.  Same thread tasks as conv_tile (4 rows x 8
// channels of one column).  The delta channels are taken `CH` at a time: all threads first write
// the window of Z the span needs, (ih + K - 1) x (iw + K - 1) values per channel, to `stage`, with
// the zeros of the border in place and, if `Darg` is given, the pooled delta D routed to the
// arg-max position of each 2 x 2 window (Z[zy][zx] = D[zy/2][zx/2] if arg = (zy%2)*2 + zx%2, else
// 0); the inner loop then reads it without any test, like the forward convolution.
// WST: the rotated filters of the CH channels are copied to `wst` (cp.async, overlapping the
// staging of the delta) and read from there.
template <int K, bool WST, class Epilogue>
__device__ __forceinline__ void delta_conv_staged(const float* __restrict__ D, const unsigned char* __restrict__ Darg,
                                                  int d_cs, int d_pitch, int zh, int zw, int vy0, int vx0,
                                                  float* __restrict__ stage, int CH, const float* __restrict__ w,
                                                  int nd /*delta channels*/, int cin_pad, int cin, int ih, int iw,
                                                  float* __restrict__ wst, Epilogue epi)
{
    constexpr int TP = 4, TC = kCoutTile;
    const int rows = ih + K - 1, pitch = iw + K - 1, cs = rows * pitch;
    const int ncob = cin_pad / TC, nyb = (ih + TP - 1) / TP;
    const int ntasks = ncob * nyb * iw;
    for (int t0 = 0; t0 < ntasks; t0 += blockDim.x) {
        const bool active = t0 + (int)threadIdx.x < ntasks;
        const int t = active ? t0 + (int)threadIdx.x : ntasks - 1;
        const int x = t % iw, rem = t / iw, yb = rem % nyb, cob = rem / nyb;
        const int y0 = yb * TP, c0 = cob * TC;
        float acc[TP][TC];
#pragma unroll
        for (int p = 0; p < TP; ++p)
#pragma unroll
            for (int c = 0; c < TC; ++c) acc[p][c] = 0.f;
        int rowoff[TP + K - 1];
#pragma unroll
        for (int r = 0; r < TP + K - 1; ++r) rowoff[r] = min(y0 + r, rows - 1) * pitch + x;
        for (int d0 = 0; d0 < nd; d0 += CH) {
            const int nch = min(CH, nd - d0);
            __syncthreads();                                   // the previous channels have been consumed
            if (WST) {
                const int n4 = nch * (K * K) * cin_pad / 4;
                const float4* src = reinterpret_cast<const float4*>(w + (size_t)d0 * (K * K) * cin_pad);
                float4* dst = reinterpret_cast<float4*>(wst);
                for (int i = threadIdx.x; i < n4; i += blockDim.x) cp_async16(dst + i, src + i);
                cp_async_commit();
            }
            for (int ch = 0; ch < nch; ++ch) {
                const float* dp = D + (d0 + ch) * d_cs;
                const unsigned char* ap = Darg ? Darg + (d0 + ch) * d_cs : nullptr;
                float* sp = stage + ch * cs;
                for (int e = threadIdx.x; e < cs; e += blockDim.x) {
                    const int a = e / pitch, b = e - a * pitch;
                    const int zy = vy0 + a - (K - 1), zx = vx0 + b - (K - 1);
                    float v = 0.f;
                    if (zy >= 0 && zy < zh && zx >= 0 && zx < zw) {
                        if (ap) {
                            const int idx = (zy >> 1) * d_pitch + (zx >> 1);
                            v = (int)ap[idx] == (((zy & 1) << 1) | (zx & 1)) ? dp[idx] : 0.f;
                        } else {
                            v = dp[zy * d_pitch + zx];
                        }
                    }
                    sp[e] = v;
                }
            }
            if (WST) cp_async_wait<0>();
            __syncthreads();
            if (active) {
                const float* wp = (WST ? wst : w + (size_t)d0 * (K * K) * cin_pad) + c0;
                for (int ci = 0; ci < nch; ++ci) {
                    const float* ip = stage + ci * cs;
                    const float* wc = wp + (size_t)ci * (K * K) * cin_pad;
#pragma unroll
                    for (int kx = 0; kx < K; ++kx) {
                        float wr[K][TC];
#pragma unroll
                        for (int ky = 0; ky < K; ++ky) {
                            const float4* wq = reinterpret_cast<const float4*>(wc + (ky * K + kx) * cin_pad);
                            const float4 a = WST ? wq[0] : __ldg(wq);
                            const float4 b = WST ? wq[1] : __ldg(wq + 1);
                            wr[ky][0] = a.x; wr[ky][1] = a.y; wr[ky][2] = a.z; wr[ky][3] = a.w;
                            wr[ky][4] = b.x; wr[ky][5] = b.y; wr[ky][6] = b.z; wr[ky][7] = b.w;
                        }
#pragma unroll
                        for (int r = 0; r < TP + K - 1; ++r) {
                            const float v = ip[rowoff[r] + kx];
#pragma unroll
                            for (int ky = 0; ky < K; ++ky) {
                                const int p = r - ky;
                                if (p >= 0 && p < TP) {
#pragma unroll
                                    for (int c = 0; c < TC; ++c) acc[p][c] = fmaf(v, wr[ky][c], acc[p][c]);
                                }
                            }
                        }
                    }
                }
            }
        }
        if (active) {
#pragma unroll
            for (int p = 0; p < TP; ++p)
                if (y0 + p < ih) {
#pragma unroll
                    for (int c = 0; c < TC; ++c)
                        if (c0 + c < cin) epi(c0 + c, y0 + p, x, acc[p][c], 0);
                }
        }
    }
}

template <int KMAX, class Epilogue>
__device__ __forceinline__ void delta_conv_staged_k(int K, const float* D, const unsigned char* Darg, int d_cs, int d_pitch,
                                                    int zh, int zw, int vy0, int vx0, float* stage, int CH, const float* w,
                                                    int nd, int cin_pad, int cin, int ih, int iw, float* wst, Epilogue epi)
{
#define FTP_DELTA_CONV(KK, WS) delta_conv_staged<KK, WS>(D, Darg, d_cs, d_pitch, zh, zw, vy0, vx0, stage, CH, w, nd, cin_pad, cin, \
                                                         ih, iw, wst, epi)
    if (wst) {
        switch (K) {
        case 1: FTP_DELTA_CONV(1, true); break;
        case 3: FTP_DELTA_CONV(3, true); break;
        default:
            if constexpr (KMAX > 3) { if (K == 5) FTP_DELTA_CONV(5, true); else FTP_DELTA_CONV(7, true); }
            break;
        }
    } else {
        switch (K) {
        case 1: FTP_DELTA_CONV(1, false); break;
        case 3: FTP_DELTA_CONV(3, false); break;
        default:
            if constexpr (KMAX > 3) { if (K == 5) FTP_DELTA_CONV(5, false); else FTP_DELTA_CONV(7, false); }
            break;
        }
    }
#undef FTP_DELTA_CONV
}

template <int KMAX, bool POOL_OUT, int MODE, class Epilogue>
__device__ __forceinline__ void conv_tile_k(int K, const float* in, const unsigned char* arg, int in_cs, int in_pitch,
                                            int in_rows, int in_cols, int y_base, int x_base, const float* w, int cin,
                                            int cout_pad, const float* bias, int cout, float slope, int oh, int ow,
                                            float* wst, int w_ch, Epilogue epi)
{
#define FTP_CONV_TILE(KK, ST) conv_tile<KK, POOL_OUT, MODE, ST>(in, arg, in_cs, in_pitch, in_rows, in_cols, y_base, x_base, w, cin, \
                                                                cout_pad, bias, cout, slope, oh, ow, wst, w_ch, epi)
    if (w_ch > 0) {
        switch (K) {
        case 1: FTP_CONV_TILE(1, true); break;
        case 3: FTP_CONV_TILE(3, true); break;
        default:
            if constexpr (KMAX > 3) { if (K == 5) FTP_CONV_TILE(5, true); else FTP_CONV_TILE(7, true); }
            break;
        }
    } else {
        switch (K) {
        case 1: FTP_CONV_TILE(1, false); break;
        case 3: FTP_CONV_TILE(3, false); break;
        default:
            if constexpr (KMAX > 3) { if (K == 5) FTP_CONV_TILE(5, false); else FTP_CONV_TILE(7, false); }
            break;
        }
    }
#undef FTP_CONV_TILE
}

// Partial filter gradient of one sub-tile (Section 4.1: feature-map tile convolved with the
// delta tile): g[co][ci][ky][kx] = sum_{y<oh, x<ow} d[co][y][x] * xin[ci][y+ky][x+kx].
// d points at the first data element of the delta buffer (inside its apron).  One warp per block
// of TCO x TCI filter planes; lanes split the pixels and are combined by a fixed butterfly, so the
// sum order never changes.  `first` selects store vs. accumulate into the block's own set.
//   POOLED: d is the delta of the pooled map and arg its arg-max bytes; only the arg-max position
//   of each 2x2 window carries a delta, so pixel (y, x) pairs with xin at (2y+ay+ky, 2x+ax+kx).
template <int K, int TCO, int TCI, bool POOLED>
__device__ __forceinline__ void filter_grad_tile(const float* __restrict__ d, const unsigned char* __restrict__ arg,
                                                 int d_cs, int d_pitch,
                                                 const float* __restrict__ xin, int in_cs, int in_pitch,
                                                 int cin, int cout, int oh, int ow, float* __restrict__ g, bool first)
{
    constexpr int KK = K * K, NACC = TCO * TCI * KK;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int ncob = (cout + TCO - 1) / TCO, ncib = (cin + TCI - 1) / TCI;
    const int npix = oh * ow;
    for (int t = warp; t < ncob * ncib; t += nwarps) {
        const int cob = t / ncib, cib = t % ncib;
        const int co0 = cob * TCO, ci0 = cib * TCI;
        float acc[NACC];
#pragma unroll
        for (int e = 0; e < NACC; ++e) acc[e] = 0.f;
        for (int p = lane; p < npix; p += 32) {
            const int ly = p / ow, lx = p % ow;
            float dv[TCO];
            int xo[TCO];
#pragma unroll
            for (int a = 0; a < TCO; ++a) {
                const int di = min(co0 + a, cout - 1) * d_cs + ly * d_pitch + lx;
                dv[a] = d[di];
                if (POOLED) {
                    const int am = arg[di];
                    xo[a] = (2 * ly + (am >> 1)) * in_pitch + 2 * lx + (am & 1);
                } else {
                    xo[a] = ly * in_pitch + lx;
                }
            }
#pragma unroll
            for (int b = 0; b < TCI; ++b) {
                const float* xp = xin + min(ci0 + b, cin - 1) * in_cs;
                if (POOLED) {
#pragma unroll
                    for (int a = 0; a < TCO; ++a)
#pragma unroll
                        for (int ky = 0; ky < K; ++ky)
#pragma unroll
                            for (int kx = 0; kx < K; ++kx)
                                acc[(a * TCI + b) * KK + ky * K + kx] =
                                    fmaf(dv[a], xp[xo[a] + ky * in_pitch + kx], acc[(a * TCI + b) * KK + ky * K + kx]);
                } else {
#pragma unroll
                    for (int ky = 0; ky < K; ++ky)
#pragma unroll
                        for (int kx = 0; kx < K; ++kx) {
                            const float xv = xp[xo[0] + ky * in_pitch + kx];
#pragma unroll
                            for (int a = 0; a < TCO; ++a)
                                acc[(a * TCI + b) * KK + ky * K + kx] = fmaf(dv[a], xv, acc[(a * TCI + b) * KK + ky * K + kx]);
                        }
                }
            }
        }
#pragma unroll
        for (int e = 0; e < NACC; ++e) {
#pragma unroll
            for (int s = 16; s >= 1; s >>= 1) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], s);
        }
        // lane l stores entries l, l+32, ...
#pragma unroll
        for (int base = 0; base < NACC; base += 32) {
            float mine = 0.f;
#pragma unroll
            for (int e = base; e < base + 32 && e < NACC; ++e)
                if (lane == e - base) mine = acc[e];
            const int me = base + lane;
            if (me < NACC) {
                const int a = me / (TCI * KK), b = (me / KK) % TCI, tap = me % KK;
                const int co = co0 + a, ci = ci0 + b;
                if (co < cout && ci < cin) {
                    float* dst = g + ((size_t)co * cin + ci) * KK + tap;
                    *dst = first ? mine : *dst + mine;
                }
            }
        }
    }
}

// Partial filter gradient, one thread per (block of TCO output channels, input channel): the thread
// keeps TCO x K x K sums in registers and walks over all delta pixels itself, so no cross-lane
// reduction is needed and the sum order is fixed.  Lanes of a warp hold consecutive input channels:
// the delta (and arg-max) reads are broadcasts, the input reads hit distinct banks because the
// channel stride of the input copy is odd.  Used when there are enough (channel block, channel)
// pairs to occupy the block; small layers take filter_grad_tile.
//   !POOLED: the K x K window of the input slides along the row in registers (K new values per pixel).
//   POOLED:  d is the delta of the pooled map; the arg-max of each 2x2 window (the same for all lanes)
//            picks which K x K part of the (K+1) x (K+1) input window the delta meets.
template <int K, int TCO, bool POOLED>
__device__ __forceinline__ void filter_grad_thread(const float* __restrict__ d, const unsigned char* __restrict__ arg,
                                                   int d_cs, int d_pitch, const float* __restrict__ xin, int in_cs,
                                                   int in_pitch, int cin, int cout, int oh, int ow,
                                                   float* __restrict__ g, bool first)
{
    constexpr int KK = K * K, WN = POOLED ? K + 1 : K;
    const int ncob = (cout + TCO - 1) / TCO;
    for (int task = threadIdx.x; task < ncob * cin; task += blockDim.x) {
        const int cob = task / cin, ci = task - cob * cin, co0 = cob * TCO;
        const float* xp = xin + ci * in_cs;
        int doff[TCO];
#pragma unroll
        for (int a = 0; a < TCO; ++a) doff[a] = min(co0 + a, cout - 1) * d_cs;
        float acc[TCO][KK];
#pragma unroll
        for (int a = 0; a < TCO; ++a)
#pragma unroll
            for (int e = 0; e < KK; ++e) acc[a][e] = 0.f;
        for (int y = 0; y < oh; ++y) {
            const float* xr = xp + (POOLED ? 2 * y : y) * in_pitch;
            float w[WN][WN];
#pragma unroll
            for (int r = 0; r < WN; ++r)
#pragma unroll
                for (int c = POOLED ? 2 : 1; c < WN; ++c) w[r][c] = xr[r * in_pitch + c - (POOLED ? 2 : 1)];
            for (int x = 0; x < ow; ++x) {
                // shift the window by one pixel (two input columns when pooled) and load the new columns
#pragma unroll
                for (int r = 0; r < WN; ++r) {
#pragma unroll
                    for (int c = 0; c + (POOLED ? 2 : 1) < WN; ++c) w[r][c] = w[r][c + (POOLED ? 2 : 1)];
                    if (POOLED) {
                        w[r][WN - 2] = xr[r * in_pitch + 2 * x + WN - 2];
                        w[r][WN - 1] = xr[r * in_pitch + 2 * x + WN - 1];
                    } else {
                        w[r][WN - 1] = xr[r * in_pitch + x + WN - 1];
                    }
                }
                const int dp = y * d_pitch + x;
#pragma unroll
                for (int a = 0; a < TCO; ++a) {
                    const float dv = d[doff[a] + dp];
                    if (POOLED) {
                        const int am = arg[doff[a] + dp];        // same for every lane: no divergence
                        if (am == 0) {
#pragma unroll
                            for (int ky = 0; ky < K; ++ky)
#pragma unroll
                                for (int kx = 0; kx < K; ++kx) acc[a][ky * K + kx] = fmaf(dv, w[ky][kx], acc[a][ky * K + kx]);
                        } else if (am == 1) {
#pragma unroll
                            for (int ky = 0; ky < K; ++ky)
#pragma unroll
                                for (int kx = 0; kx < K; ++kx) acc[a][ky * K + kx] = fmaf(dv, w[ky][kx + (POOLED ? 1 : 0)], acc[a][ky * K + kx]);
                        } else if (am == 2) {
#pragma unroll
                            for (int ky = 0; ky < K; ++ky)
#pragma unroll
                                for (int kx = 0; kx < K; ++kx) acc[a][ky * K + kx] = fmaf(dv, w[ky + (POOLED ? 1 : 0)][kx], acc[a][ky * K + kx]);
                        } else {
#pragma unroll
                            for (int ky = 0; ky < K; ++ky)
#pragma unroll
                                for (int kx = 0; kx < K; ++kx)
                                    acc[a][ky * K + kx] = fmaf(dv, w[ky + (POOLED ? 1 : 0)][kx + (POOLED ? 1 : 0)], acc[a][ky * K + kx]);
                        }
                    } else {
#pragma unroll
                        for (int ky = 0; ky < K; ++ky)
#pragma unroll
                            for (int kx = 0; kx < K; ++kx) acc[a][ky * K + kx] = fmaf(dv, w[ky][kx], acc[a][ky * K + kx]);
                    }
                }
            }
        }
#pragma unroll
        for (int a = 0; a < TCO; ++a)
            if (co0 + a < cout) {
                float* dst = g + ((size_t)(co0 + a) * cin + ci) * KK;
#pragma unroll
                for (int e = 0; e < KK; ++e) dst[e] = first ? acc[a][e] : dst[e] + acc[a][e];
            }
    }
}

template <int KMAX, bool POOLED>
__device__ __forceinline__ void filter_grad_k(int K, const float* d, const unsigned char* arg, int d_cs, int d_pitch,
                                              const float* xin, int in_cs, int in_pitch, int cin, int cout, int oh,
                                              int ow, float* g, bool first)
{
    // one thread per (channel block, channel) when that occupies at least half of the block's threads;
    // blocks of 8 output channels if that still fills the block, else blocks of 4
    if (K == 3) {
        const int t8 = ((cout + 7) / 8) * cin, t4 = ((cout + 3) / 4) * cin, nt = (int)blockDim.x;
        if (t8 >= nt || (t8 >= nt / 2 && t4 > 2 * nt)) {
            filter_grad_thread<3, 8, POOLED>(d, arg, d_cs, d_pitch, xin, in_cs, in_pitch, cin, cout, oh, ow, g, first);
            return;
        }
        if (t4 >= nt / 2) {
            filter_grad_thread<3, 4, POOLED>(d, arg, d_cs, d_pitch, xin, in_cs, in_pitch, cin, cout, oh, ow, g, first);
            return;
        }
    }
    switch (K) {
    case 1: filter_grad_tile<1, 4, 8, POOLED>(d, arg, d_cs, d_pitch, xin, in_cs, in_pitch, cin, cout, oh, ow, g, first); break;
    case 3: filter_grad_tile<3, 4, 2, POOLED>(d, arg, d_cs, d_pitch, xin, in_cs, in_pitch, cin, cout, oh, ow, g, first); break;
    default:
        if constexpr (KMAX > 3) {
            if (K == 5) filter_grad_tile<5, 2, 1, POOLED>(d, arg, d_cs, d_pitch, xin, in_cs, in_pitch, cin, cout, oh, ow, g, first);
            else filter_grad_tile<7, 1, 1, POOLED>(d, arg, d_cs, d_pitch, xin, in_cs, in_pitch, cin, cout, oh, ow, g, first);
        }
        break;
    }
}

// Partial bias gradient: gb[co] = sum over the sub-tile's delta pixels.
__device__ __forceinline__ void bias_grad_tile(const float* __restrict__ d, int d_cs, int d_pitch, int cout,
                                               int oh, int ow, float* __restrict__ gb, bool first)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int npix = oh * ow;
    // pixel p = lane, lane + 32, ... in row-major order; its (row, column) is stepped, not divided out
    const int y0 = lane / ow, x0 = lane - y0 * ow, dy = 32 / ow, dx = 32 - dy * ow;
    for (int co = warp; co < cout; co += nwarps) {
        const float* dc = d + co * d_cs;
        float s = 0.f;
        int y = y0, x = x0;
        for (int p = lane; p < npix; p += 32) {
            s += dc[y * d_pitch + x];
            x += dx; y += dy;
            if (x >= ow) { x -= ow; ++y; }
        }
#pragma unroll
        for (int k = 16; k >= 1; k >>= 1) s += __shfl_xor_sync(0xffffffffu, s, k);
        if (lane == 0) gb[co] = first ? s : gb[co] + s;
    }
}

// ---------------------------------------------------------------------------------------------
// Fused forward of one group: grid (R*Q, N), one sub-tile stack per block.
// ---------------------------------------------------------------------------------------------
// KMAX: largest conv window of the group (3: the 5x5 / 7x7 code paths are left out, which frees registers of the common ones).
template <int KMAX>
__global__ void __launch_bounds__(kThreads, 1) fwd_group_kernel(const __grid_constant__ GroupArgs A)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int* hdr = reinterpret_cast<int*>(smem_raw);
    float* sm = reinterpret_cast<float*>(smem_raw + kSmemHeader);
    const int q = blockIdx.x % A.Q, r = blockIdx.x / A.Q, n = blockIdx.y;
    load_header(hdr, A, r, q, true);
    __syncthreads();

    {   // group input -> input buffer of the first op (halo comes from the neighbours' part of the map)
        const OpDesc& op = A.op[0];
        const int oh = hdr[8 + 1] - hdr[8 + 0] + 1, ow = hdr[8 + 3] - hdr[8 + 2] + 1;
        const int bh = (oh - 1) * op.S + op.keff, bw = (ow - 1) * op.S + op.keff;
        load_input(sm + op.in_off, op.in_cs, op.in_pitch, bh, bw, op.cin, A.map[0], n, op.in_H, op.in_W,
                   hdr[8 + 0] * op.S - op.pad, hdr[8 + 2] * op.S - op.pad);
    }
    __syncthreads();

    for (int i = 0; i < A.n_ops; ++i) {
        const OpDesc& op = A.op[i];
        const int* ho = hdr + (i + 1) * 8;                    // span / cell at this op's output map
        const int oy1 = ho[0], ox1 = ho[2];
        const int oh = ho[1] - ho[0] + 1, ow = ho[3] - ho[2] + 1;
        const int cy1 = ho[4], cy2 = ho[5], cx1 = ho[6], cx2 = ho[7];
        const bool last = i == A.n_ops - 1;
        // geometry of the consumer's input buffer
        float* nb = nullptr; int ncs = 0, npitch = 0, noy = 0, nox = 0;
        if (!last) {
            const OpDesc& nx = A.op[i + 1];
            const int* hn = hdr + (i + 2) * 8;
            nb = sm + nx.in_off; ncs = nx.in_cs; npitch = nx.in_pitch;
            noy = hn[0] * nx.S - nx.pad; nox = hn[2] * nx.S - nx.pad;
            const int nbh = (hn[1] - hn[0]) * nx.S + nx.keff, nbw = (hn[3] - hn[2]) * nx.S + nx.keff;
            zero_apron(nb, ncs, npitch, nbh, nbw, nx.cin, oy1 - noy, oy1 - noy + oh - 1, ox1 - nox, ox1 - nox + ow - 1);
        }
        float* gout = A.map_out[i + 1];
        unsigned char* garg = A.arg[i];
        const int OH = op.out_H, OW = op.out_W, Cout = op.cout;
        auto emit = [&](int c, int ly, int lx, float v, int am) {
            const int y = oy1 + ly, x = ox1 + lx;
            if (!last) nb[c * ncs + (y - noy) * npitch + (x - nox)] = v;
            if (y >= cy1 && y <= cy2 && x >= cx1 && x <= cx2) {
                const size_t gi = (((size_t)n * Cout + c) * OH + y) * OW + x;
                gout[gi] = v;
                if (garg) garg[gi] = (unsigned char)am;
            }
        };
        const float* ib = sm + op.in_off;
        if (op.kind == kOpPool) {
            const int total = op.cout * oh * ow;
            for (int e = threadIdx.x; e < total; e += blockDim.x) {
                const int lx = e % ow, t = e / ow, ly = t % oh, c = t / oh;
                const float* p = ib + c * op.in_cs + 2 * ly * op.in_pitch + 2 * lx;
                float best = p[0];
                best = p[1] > best ? p[1] : best;
                best = p[op.in_pitch] > best ? p[op.in_pitch] : best;
                best = p[op.in_pitch + 1] > best ? p[op.in_pitch + 1] : best;
                emit(c, ly, lx, best, 0);
            }
        } else {
            const float slope = op.slope;
            const float* bias = A.params + op.p_off + (size_t)op.cout * op.cin * op.k * op.k;
            if (op.kind == kOpConv)
                conv_tile_k<KMAX, false, kInPlain>(op.k, ib, nullptr, op.in_cs, op.in_pitch, oh + op.k - 1, 0, 0, 0,
                                             A.wpk + op.wf_off, op.cin, op.cout_pad, bias, op.cout, slope, oh, ow,
                                             sm + op.w_off, op.w_ch,
                                             [&](int c, int ly, int lx, float z, int) { emit(c, ly, lx, leaky(z, slope), 0); });
            else
                conv_tile_k<KMAX, true, kInPlain>(op.k, ib, nullptr, op.in_cs, op.in_pitch, 2 * oh + op.k - 1, 0, 0, 0,
                                            A.wpk + op.wf_off, op.cin, op.cout_pad, bias, op.cout, slope, 2 * oh, 2 * ow,
                                            sm + op.w_off, op.w_ch, emit);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// Fused backward of one group (adjoint form): each block owns one partial gradient set and walks
// through its share of the (image, sub-tile) stacks of one user tile in a fixed order.
// ---------------------------------------------------------------------------------------------
template <int KMAX>
__global__ void __launch_bounds__(kThreads, 1) bwd_group_kernel(const __grid_constant__ GroupArgs A)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int* hdr = reinterpret_cast<int*>(smem_raw);
    unsigned char* smb = smem_raw + kSmemHeader;
    float* sm = reinterpret_cast<float*>(smb);

    // The sub-tile stacks of the whole batch, image by image and row by row, are dealt out evenly to
    // the blocks; each block adds the filter gradients of its stacks into its own partial set.
    const int slot = blockIdx.x;
    const int items = A.N * A.R * A.Q;
    const int lo = (int)((long long)slot * items / (int)gridDim.x), hi = (int)((long long)(slot + 1) * items / (int)gridDim.x);
    float* myset = A.partial + (size_t)slot * A.param_floats;
    const int nops = A.n_ops;

    for (int item = lo; item < hi; ++item) {
        const bool first = item == lo;
        const int n = item / (A.R * A.Q), r = (item / A.Q) % A.R, q = item % A.Q;
        load_header(hdr, A, r, q, false);
        __syncthreads();

        {   // delta at the group's output map, restricted to this sub-tile's owned cell
            const OpDesc& op = A.op[nops - 1];
            const int* ho = hdr + nops * 8;
            const int oh = ho[1] - ho[0] + 1, ow = ho[3] - ho[2] + 1;
            const bool act = op.kind != kOpPool;
            float* D = sm + op.d_off;
            unsigned char* Darg = smb + op.d_arg_off;
            const float* dsrc = A.dmap_out;
            const float* ysrc = A.map[nops];
            const unsigned char* asrc = op.kind == kOpConvPool ? A.arg[nops - 1] : nullptr;
            const int total = op.cout * oh * ow;
            for (int e = threadIdx.x; e < total; e += blockDim.x) {
                const int lx = e % ow, t = e / ow, ly = t % oh, c = t / oh;
                const size_t gi = (((size_t)n * op.cout + c) * op.out_H + ho[0] + ly) * op.out_W + ho[2] + lx;
                float v = __ldg(dsrc + gi);
                if (act) v *= dleaky(__ldg(ysrc + gi), op.slope);
                D[c * op.d_cs + ly * op.d_pitch + lx] = v;
                if (asrc) Darg[c * op.d_cs + ly * op.d_pitch + lx] = asrc[gi];
            }
        }

        for (int i = nops - 1; i >= 0; --i) {
            const OpDesc& op = A.op[i];
            const int* ho = hdr + (i + 1) * 8;     // span at this op's output map
            const int* hi_ = hdr + i * 8;          // span at its input map
            const int oh = ho[1] - ho[0] + 1, ow = ho[3] - ho[2] + 1;
            const int oy = ho[0] * op.S - op.pad, ox = ho[2] * op.S - op.pad;   // map position of the X buffer's (0,0)
            const int bh = (oh - 1) * op.S + op.keff, bw = (ow - 1) * op.S + op.keff;
            float* X = sm + op.in_off;
            float* D = sm + op.d_off;
            const unsigned char* Darg = smb + op.d_arg_off;
            load_input(X, op.in_cs, op.in_pitch, bh, bw, op.cin, A.map[i], n, op.in_H, op.in_W, oy, ox);

            // where this op's input delta goes: the producer's delta buffer, or the scratch block
            const int ih = hi_[1] - hi_[0] + 1, iw = hi_[3] - hi_[2] + 1;   // valid input span
            const int vy0 = hi_[0] - oy, vx0 = hi_[2] - ox;                 // its offset inside the X buffer
            float* dst; int dcs, dpitch;
            const bool to_scratch = i == 0;
            if (!to_scratch) {
                const OpDesc& pv = A.op[i - 1];
                dst = sm + pv.d_off; dcs = pv.d_cs; dpitch = pv.d_pitch;
                if (pv.kind == kOpConvPool) {       // arg-max of the producer's pooling windows over this span
                    unsigned char* parg = smb + pv.d_arg_off;
                    const unsigned char* asrc = A.arg[i - 1];
                    const int total = pv.cout * ih * iw;
                    for (int e = threadIdx.x; e < total; e += blockDim.x) {
                        const int xx = e % iw, t = e / iw, yy = t % ih, c = t / ih;
                        parg[c * dcs + yy * dpitch + xx] =
                            asrc[(((size_t)n * pv.cout + c) * pv.out_H + hi_[0] + yy) * pv.out_W + hi_[2] + xx];
                    }
                }
            } else {
                const int Wtot = A.xoff[A.Q];
                const int Htot = A.yoff[A.R];
                dst = A.scratch + (size_t)n * op.cin * Htot * Wtot +
                      (size_t)op.cin * ((size_t)A.yoff[r] * Wtot + (size_t)ih * A.xoff[q]);
                dcs = ih * iw; dpitch = iw;
            }
            __syncthreads();   // X loaded, D complete

            const float pslope = op.prev_has_act ? A.op[i - 1].slope : 1.f;
            const bool pact = op.prev_has_act != 0;
            const bool need_in_delta = !to_scratch || A.need_dx;
            if (op.kind != kOpPool) {
                float* gw = myset + op.gp_off;
                auto put = [&](int c, int uy, int ux, float v, int) {
                    if (pact) v *= dleaky(X[c * op.in_cs + (vy0 + uy) * op.in_pitch + vx0 + ux], pslope);
                    dst[c * dcs + uy * dpitch + ux] = v;
                };
                // input delta = correlation of the zero-extended output delta with the rotated filter:
                // position u of the X buffer reads delta rows u + ky' - (K-1)
                if (op.kind == kOpConv) {
                    filter_grad_k<KMAX, false>(op.k, D, nullptr, op.d_cs, op.d_pitch, X, op.in_cs, op.in_pitch, op.cin, op.cout,
                                         oh, ow, gw, first);
                    bias_grad_tile(D, op.d_cs, op.d_pitch, op.cout, oh, ow, gw + (size_t)op.cout * op.cin * op.k * op.k, first);
                    if (need_in_delta)
                        conv_tile_k<KMAX, false, kInChecked>(op.k, D, nullptr, op.d_cs, op.d_pitch, oh, ow, vy0 - (op.k - 1),
                                                       vx0 - (op.k - 1), A.wpk + op.wb_off, op.cout, op.cin_pad, nullptr,
                                                       op.cin, 0.f, ih, iw, sm + op.w_off, op.w_ch, put);
                } else {
                    filter_grad_k<KMAX, true>(op.k, D, Darg, op.d_cs, op.d_pitch, X, op.in_cs, op.in_pitch, op.cin, op.cout,
                                        oh, ow, gw, first);
                    bias_grad_tile(D, op.d_cs, op.d_pitch, op.cout, oh, ow, gw + (size_t)op.cout * op.cin * op.k * op.k, first);
                    if (need_in_delta && op.dz_ch > 0)
                        delta_conv_staged_k<KMAX>(op.k, D, Darg, op.d_cs, op.d_pitch, 2 * oh, 2 * ow, vy0, vx0, sm + op.dz_off, op.dz_ch,
                                            A.wpk + op.wb_off, op.cout, op.cin_pad, op.cin, ih, iw,
                                            op.w_ch > 0 ? sm + op.w_off : nullptr, put);
                    else if (need_in_delta)   // the pooled delta is expanded through the arg-max on the fly
                        conv_tile_k<KMAX, false, kInExpand>(op.k, D, Darg, op.d_cs, op.d_pitch, 2 * oh, 2 * ow, vy0 - (op.k - 1),
                                                      vx0 - (op.k - 1), A.wpk + op.wb_off, op.cout, op.cin_pad, nullptr,
                                                      op.cin, 0.f, ih, iw, nullptr, 0, put);
                }
            } else if (need_in_delta) {
                const int total = op.cout * oh * ow;
                for (int e = threadIdx.x; e < total; e += blockDim.x) {
                    const int lx = e % ow, t = e / ow, ly = t % oh, c = t / oh;
                    const float* p = X + c * op.in_cs + 2 * ly * op.in_pitch + 2 * lx;
                    const float v0 = p[0], v1 = p[1], v2 = p[op.in_pitch], v3 = p[op.in_pitch + 1];
                    float best = v0; int am = 0;
                    if (v1 > best) { best = v1; am = 1; }
                    if (v2 > best) { best = v2; am = 2; }
                    if (v3 > best) { best = v3; am = 3; }
                    float dv = D[c * op.d_cs + ly * op.d_pitch + lx];
                    if (pact) dv *= dleaky(best, pslope);
                    float* o = dst + c * dcs + 2 * ly * dpitch + 2 * lx;
                    o[0] = am == 0 ? dv : 0.f;
                    o[1] = am == 1 ? dv : 0.f;
                    o[dpitch] = am == 2 ? dv : 0.f;
                    o[dpitch + 1] = am == 3 ? dv : 0.f;
                }
            }
            __syncthreads();
        }
    }
}

// Sum of the overlapping group-input delta contributions of neighbouring sub-tiles, in a fixed
// (row, column) order: the backward boundary exchange at a group input.
__global__ void halo_sum_kernel(const __grid_constant__ HaloSumArgs A)
{
    // The cover / span / offset tables go to shared memory first: every output value walks through
    // three of them in a row, which from global memory is three dependent round trips.
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
    // one warp per map row (n, c, y): what depends on the covering sub-tile rows only is computed once
    // per row (32-bit offsets inside an image's scratch area), lanes walk along x
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const long long rows = (long long)A.N * A.C * A.H;
    for (long long row = (long long)blockIdx.x * wpb + (threadIdx.x >> 5); row < rows; row += (long long)gridDim.x * wpb) {
        const int y = (int)(row % A.H); long long t = row / A.H;
        const int c = (int)(t % A.C); const int n = (int)(t / A.C);
        const int r0 = ycover[2 * y], nr = ycover[2 * y + 1] - r0 + 1;
        int base[4], ch[4], dr[4];       // the first four covering sub-tile rows (more only with very fine splits)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int r = min(r0 + k, A.R - 1);
            const int y1 = yspan[2 * r], h = yspan[2 * r + 1] - y1 + 1;
            base[k] = A.C * yoff[r] * A.Wtot; ch[k] = A.C * h; dr[k] = c * h + (y - y1);
        }
        const float* img = A.scratch + (size_t)n * A.C * A.Htot * A.Wtot;
        float* orow = A.out + row * A.W;
        for (int x = lane; x < A.W; x += 32) {
            const int q0 = xcover[2 * x], q1 = xcover[2 * x + 1];
            float s = 0.f;
            // the first two covering sub-tile columns are handled without a loop, so that the loads of
            // up to 4 x 2 blocks are in flight together (same order of the sums as the plain loops)
            const int qb = min(q0 + 1, A.Q - 1);
            const int xa1 = xspan[2 * q0], wa = xspan[2 * q0 + 1] - xa1 + 1, oa = xoff[q0];
            const int xb1 = xspan[2 * qb], wb = xspan[2 * qb + 1] - xb1 + 1, ob = xoff[qb];
            const bool two = q1 > q0;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < nr) {
                    s += img[base[k] + oa * ch[k] + dr[k] * wa + (x - xa1)];
                    if (two) s += img[base[k] + ob * ch[k] + dr[k] * wb + (x - xb1)];
                    for (int q = q0 + 2; q <= q1; ++q) {
                        const int x1 = xspan[2 * q], w = xspan[2 * q + 1] - x1 + 1;
                        s += img[base[k] + xoff[q] * ch[k] + dr[k] * w + (x - x1)];
                    }
                }
            for (int k = 4; k < nr; ++k) {                 // same order, offsets worked out on the spot
                const int r = r0 + k, y1 = yspan[2 * r], h = yspan[2 * r + 1] - y1 + 1;
                for (int q = q0; q <= q1; ++q) {
                    const int x1 = xspan[2 * q], w = xspan[2 * q + 1] - x1 + 1;
                    s += img[A.C * yoff[r] * A.Wtot + xoff[q] * (A.C * h) + (c * h + (y - y1)) * w + (x - x1)];
                }
            }
            orow[x] = s;
        }
    }
}

// Filters -> the two packed layouts the tile kernels read:
//   wf[ci][tap][co_pad]           (forward)       wb[co][tap'][ci_pad] with tap' = K*K-1-tap (rotated 180 degrees)
__global__ void pack_filters_kernel(const __grid_constant__ PackArgs A, const float* __restrict__ params,
                                    float* __restrict__ wf, float* __restrict__ wb)
{
    const PackLayer L = A.l[blockIdx.y];
    const int KK = L.k * L.k;
    const long long nf = (long long)L.cin * KK * L.cout_pad, nb = (long long)L.cout * KK * L.cin_pad;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < nf + nb; e += (long long)gridDim.x * blockDim.x) {
        if (e < nf) {
            const int co = (int)(e % L.cout_pad); long long t = e / L.cout_pad;
            const int tap = (int)(t % KK); const int ci = (int)(t / KK);
            wf[L.wf_off + e] = co < L.cout ? params[L.p_off + ((long long)co * L.cin + ci) * KK + tap] : 0.f;
        } else {
            const long long f = e - nf;
            const int ci = (int)(f % L.cin_pad); long long t = f / L.cin_pad;
            const int tapr = (int)(t % KK); const int co = (int)(t / KK);
            wb[L.wb_off + f] = ci < L.cin ? params[L.p_off + ((long long)co * L.cin + ci) * KK + (KK - 1 - tapr)] : 0.f;
        }
    }
}

// Cross-tile reduction of the partial gradient sets in a fixed order, fused with the update
// (Section 4.1: the sets are summed once per batch and the result updates F_l).
__global__ void reduce_sgd_kernel(const __grid_constant__ ReduceArgs A, long long first, long long total, float* __restrict__ params,
                                  float lr, float* __restrict__ grad_out)
{
    // parameters first .. total - 1 (the groups of A cover them)
    for (long long e = first + blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        int g = 0;
        while (g + 1 < A.n && e >= A.g[g + 1].begin) ++g;
        const long long local = e - A.g[g].begin;
        const float* p = A.g[g].partial + local;
        float s = 0.f;
        for (int k = 0; k < A.g[g].sets; ++k) s += p[(size_t)k * A.g[g].floats];
        if (grad_out) grad_out[e] = s;
        if (params) params[e] = params[e] - lr * s;
    }
}

__global__ void sgd_kernel(float* __restrict__ params, const float* __restrict__ grad, size_t count, float lr)
{
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x)
        params[e] = params[e] - lr * grad[e];
}

// Mean-squared-error loss delta d = 2 (y - t) / M and per-block partial sums of (y - t)^2.
__global__ void mse_delta_kernel(const float* __restrict__ y, const float* __restrict__ t, float* __restrict__ d,
                                 size_t M, float* __restrict__ block_sums)
{
    __shared__ float red[256];
    const float scale = 2.0f / (float)M;
    float s = 0.f;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < M; e += (size_t)gridDim.x * blockDim.x) {
        const float diff = y[e] - t[e];
        d[e] = scale * diff;
        s += diff * diff;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int k = 128; k >= 1; k >>= 1) {
        if ((int)threadIdx.x < k) red[threadIdx.x] += red[threadIdx.x + k];
        __syncthreads();
    }
    if (threadIdx.x == 0) block_sums[blockIdx.x] = red[0];
}

// Sums the per-block partial sums in a fixed order (strided per thread, then a tree) and writes the mean.
__global__ void mse_finish_kernel(const float* __restrict__ block_sums, int n, size_t M, float* __restrict__ loss)
{
    __shared__ float red[256];
    float s = 0.f;
    for (int i = threadIdx.x; i < n; i += 256) s += block_sums[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int k = 128; k >= 1; k >>= 1) {
        if ((int)threadIdx.x < k) red[threadIdx.x] += red[threadIdx.x + k];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = red[0] / (float)M;
}

}  // namespace ftp
