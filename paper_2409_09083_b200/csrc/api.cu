// C-ABI entry points: argument checks, lazy upload of the plan tables, kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <new>

#include "ftp.h"
#include "kernels.cuh"
#include "kernels_tc.cuh"
#include "plan.hpp"
#include "stationary_args.hpp"
#include "tc_stationary.cuh"

using namespace ftp;

namespace {

inline float* ws_ptr(void* ws, size_t off) { return reinterpret_cast<float*>(static_cast<unsigned char*>(ws) + off); }

// Largest conv window of an executed group (selects the kernel instantiation of the fp32 path).
int max_window(const GroupPlan& g)
{
    int k = 1;
    for (int i = 0; i < g.n_ops; ++i)
        if (g.fwd_ops[i].kind != kOpPool) k = std::max(k, g.fwd_ops[i].k);
    return k;
}

int ensure_device(ftp_plan* p)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return FTP_ERR_CUDA;
    if (p->dev_tables && p->dev_id == dev) return FTP_OK;
    if (p->dev_tables) { cudaFree(p->dev_tables); p->dev_tables = nullptr; }
    if (cudaFuncSetAttribute(fwd_group_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(fwd_group_kernel<7>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(bwd_group_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(bwd_group_kernel<7>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(fwd_group_tc_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(fwd_group_tc_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(bwd_group_tc_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(bwd_group_tc_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(filter_grad_tc_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcFgSmemBudget) != cudaSuccess ||
        cudaFuncSetAttribute(conv_tc_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcConvSmemBudget) != cudaSuccess ||
        !st_prepare_device())
        return FTP_ERR_CUDA;
    if (!p->grad_stream) {
        cudaStream_t gs;
        if (cudaStreamCreateWithFlags(&gs, cudaStreamNonBlocking) != cudaSuccess) return FTP_ERR_CUDA;
        p->grad_stream = gs;
        for (int i = 0; i < 2; ++i) {
            cudaEvent_t a, b;
            if (cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) return FTP_ERR_CUDA;
            p->ev_dz[i] = a; p->ev_fg[i] = b;
        }
    }
    const size_t bytes = p->tables.size() * sizeof(int);
    if (cudaMalloc(&p->dev_tables, bytes) != cudaSuccess) return FTP_ERR_CUDA;
    if (cudaMemcpy(p->dev_tables, p->tables.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess) return FTP_ERR_CUDA;
    p->dev_id = dev;
    return FTP_OK;
}

inline bool launched_ok() { return cudaGetLastError() == cudaSuccess; }

constexpr int kMaxTimed = 512;

// Brackets one kernel launch with events when timing is on, and counts the launch.
struct Timed {
    ftp_plan* p; cudaStream_t st; int slot = -1;
    Timed(ftp_plan* plan, cudaStream_t s, int kind, int group) : p(plan), st(s)
    {
        ++p->launches;
        if (p->timing && p->ev_used < (int)p->ev_begin.size()) {
            slot = p->ev_used++;
            p->ev_kind[slot] = kind; p->ev_group[slot] = group;
            cudaEventRecord(static_cast<cudaEvent_t>(p->ev_begin[slot]), st);
        }
    }
    ~Timed() { if (slot >= 0) cudaEventRecord(static_cast<cudaEvent_t>(p->ev_end[slot]), st); }
};

const float* map_ptr(const ftp_plan* p, const float* x, void* ws, int l /* X_l, 1-based */)
{
    return l == 1 ? x : ws_ptr(ws, p->ws.map_off[l - 1]);
}

void fill_common(const ftp_plan* p, const GroupPlan& g, bool backward, const float* x, const float* params,
                 void* ws, GroupArgs& a)
{
    const PassPlan& pp = backward ? g.bwd : g.fwd;
    std::memset(&a, 0, sizeof(a));
    a.n_ops = g.n_ops; a.R = pp.y.count; a.Q = pp.x.count; a.N = p->N;
    for (int i = 0; i < g.n_ops; ++i) a.op[i] = backward ? g.bwd_ops[i] : g.fwd_ops[i];
    a.map[0] = map_ptr(p, x, ws, g.first);
    for (int i = 0; i < g.n_ops; ++i) {
        const OpDesc& op = a.op[i];
        a.map[i + 1] = map_ptr(p, x, ws, op.out_map);
        a.map_out[i + 1] = const_cast<float*>(a.map[i + 1]);
        a.arg[i] = op.kind == kOpConvPool
                       ? static_cast<unsigned char*>(ws) + p->ws.arg_off[op.out_map - 1] : nullptr;
    }
    a.yspan = p->dev_tables + pp.dev_yspan; a.xspan = p->dev_tables + pp.dev_xspan;
    a.ycell = p->dev_tables + pp.dev_ycell; a.xcell = p->dev_tables + pp.dev_xcell;
    a.yoff = p->dev_tables + pp.dev_yoff;   a.xoff = p->dev_tables + pp.dev_xoff;
    a.ytile = p->dev_tables + pp.dev_ytile; a.xtile = p->dev_tables + pp.dev_xtile;
    a.wpk = ws_ptr(ws, backward ? p->ws.wb_off : p->ws.wf_off);
    a.params = params;
}

int pack_filters(ftp_plan* p, const float* params, void* ws, cudaStream_t st)
{
    PackArgs pa{};
    for (const GroupPlan& g : p->groups)
        for (int i = 0; i < g.n_ops; ++i) {
            const OpDesc& op = g.fwd_ops[i];
            if (op.kind == kOpPool) continue;
            if (pa.n == kMaxOps * 2) {   // flush a full batch
                { Timed t(p, st, 0, -1);
                  pack_filters_kernel<<<dim3(64, pa.n), 256, 0, st>>>(pa, params, ws_ptr(ws, p->ws.wf_off), ws_ptr(ws, p->ws.wb_off)); }
                pa.n = 0;
            }
            pa.l[pa.n++] = PackLayer{op.p_off, op.wf_off, op.wb_off, op.cin, op.cout, op.k, op.cout_pad, op.cin_pad};
        }
    if (pa.n) {
        Timed t(p, st, 0, -1);
        pack_filters_kernel<<<dim3(64, pa.n), 256, 0, st>>>(pa, params, ws_ptr(ws, p->ws.wf_off), ws_ptr(ws, p->ws.wb_off));
    }
    return launched_ok() ? FTP_OK : FTP_ERR_CUDA;
}

inline bool is_tc(const ftp_plan* p) { return p->precision == FTP_BF16_FP32ACC; }
inline int* err_ptr(void* ws, const ftp_plan* p) { return reinterpret_cast<int*>(static_cast<unsigned char*>(ws) + p->ws.err_off); }
// Shared memory requested per block, so that exactly `ctas` blocks share an SM and the tensor memory
// they allocate (512 / ctas columns each) is always available: more than half of the SM's 228 KB for
// one block, more than a third for two.
inline size_t tc_smem(size_t need, int ctas) { return std::max(need, (size_t)(ctas == 2 ? 77 : 120) * 1024); }

// cuTensorMapEncodeTiled, obtained through the runtime (the library does not link against the driver library).
typedef CUresult (*tensor_map_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                         const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                         CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
tensor_map_encode_fn tensor_map_encoder()
{
    static tensor_map_encode_fn fn = []() -> tensor_map_encode_fn {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) return nullptr;
        return reinterpret_cast<tensor_map_encode_fn>(sym);
    }();
    return fn;
}

// Tensor map of a saved bf16 map [N][planes][H][W][8 channels] of THIS GPU's memory, with one tile plane
// (box_h rows x box_w columns x 8 channels) as the box and zeros outside the map.  false: not encodable
// (the kernel then copies the tile with plain loads).
bool encode_plane_map(unsigned char out[128], const void* base, int N, int planes, int H, int W, int box_h, int box_w)
{
    tensor_map_encode_fn enc = tensor_map_encoder();
    if (!enc || box_h > 256 || box_w > 256 || box_h < 1 || box_w < 1) return false;
    static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
    const cuuint64_t dims[4] = {8, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N * planes};
    const cuuint64_t strides[3] = {16, (cuuint64_t)W * 16, (cuuint64_t)H * W * 16};      // bytes, dimensions 1..3
    const cuuint32_t box[4] = {8, (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap m;
    if (enc(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    std::memcpy(out, &m, 128);
    return true;
}

// Tensor map of bf16 planes [N x planes][H][pitch_w][8] of THIS GPU's memory for the banded kernels: columns
// 0 .. W-1 of every row (W < pitch_w: a column range that starts at `base`), seen as rows of 2 W eight-byte elements
// (two per pixel) so that a box row of box_w pixels is one contiguous run; zeros outside.  box_w <= 128.
bool encode_rows_map(unsigned char out[128], const void* base, int N, int planes, int H, int W, int pitch_w, int box_h, int box_w)
{
    tensor_map_encode_fn enc = tensor_map_encoder();
    if (!enc || box_h > 256 || box_w > 128 || box_h < 1 || box_w < 1) return false;
    const cuuint64_t dims[3] = {2 * (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N * planes};
    const cuuint64_t strides[2] = {(cuuint64_t)pitch_w * 16, (cuuint64_t)H * pitch_w * 16};
    const cuuint32_t box[3] = {2 * (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUtensorMap m;
    if (enc(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    std::memcpy(out, &m, 128);
    return true;
}

// One launch of the banded convolution kernel: `in` planes (cin16 channels) -> `out` planes (cout16 channels).
struct PrevLayer { const uint4* y; const unsigned long long* arg; float slope; };   // see TcConvRowsArgs::prev_y

bool launch_tc_conv(ftp_plan* p, const TcConvPlan& c, int kind, int gi, const void* in, const __nv_bfloat16* w, const float* bias,
                    void* out, unsigned char* arg, int K, int cin16, int cout16, int cout, int H, int W, bool pool, float slope,
                    int* error, cudaStream_t st, const PrevLayer* prev = nullptr)
{
    TcConvRowsArgs a{};
    if (!encode_rows_map(a.tmap_x, in, p->N, cin16 / 8, H, W, W, c.R + K - 1, c.Wp)) return false;
    a.w = w;
    if (prev) { a.prev_y = prev->y; a.prev_arg = prev->arg; a.prev_slope = prev->slope; }
    a.bias = bias; a.out = static_cast<uint4*>(out); a.arg = reinterpret_cast<unsigned long long*>(arg);
    a.error = error;
    a.N = p->N; a.K = K; a.cin16 = cin16; a.cout16 = cout16; a.cout = cout; a.H = H; a.W = W; a.pool = pool ? 1 : 0;
    a.slope = slope;
    a.Ns = c.Ns; a.slices = c.slices; a.R = c.R; a.Wp = c.Wp; a.bands_img = c.bands_img; a.nblk = c.nblk; a.kpc = c.kpc;
    a.ncc = c.ncc; a.Cw = c.Cw; a.items = c.items; a.pool_planes = c.pool_planes; a.nbuf = c.nbuf;
    a.x_plane = c.x_plane; a.stage_bytes = c.stage_bytes; a.stages = c.stages;
    { Timed tm(p, st, kind, gi);
      conv_tc_rows_kernel<<<c.blocks, kTcConvThreads, c.smem_bytes, st>>>(a); }
    return launched_ok();
}

void fill_common_tc(const ftp_plan* p, const GroupPlan& g, bool backward, const float* x, const float* params,
                    void* ws, TcGroupArgs& a)
{
    const PassPlan& pp = backward ? g.bwd : g.fwd;
    std::memset(&a, 0, sizeof(a));
    a.n_ops = g.n_ops; a.R = pp.y.count; a.Q = pp.x.count; a.N = p->N;
    for (int i = 0; i < g.n_ops; ++i) a.op[i] = backward ? g.bwd_ops[i] : g.fwd_ops[i];
    a.in_f32 = g.first == 1 ? 1 : 0;
    a.in_C = p->maps[g.first - 1].C;
    a.map[0] = map_ptr(p, x, ws, g.first);
    for (int i = 0; i < g.n_ops; ++i) {
        const OpDesc& op = a.op[i];
        a.map[i + 1] = map_ptr(p, x, ws, op.out_map);
        a.map_out[i + 1] = reinterpret_cast<__nv_bfloat16*>(const_cast<float*>(map_ptr(p, x, ws, op.out_map)));
        a.arg[i] = op.kind == kOpConvPool
                       ? static_cast<unsigned char*>(ws) + p->ws.arg_off[op.out_map - 1] : nullptr;
    }
    a.yspan = p->dev_tables + pp.dev_yspan; a.xspan = p->dev_tables + pp.dev_xspan;
    a.ycell = p->dev_tables + pp.dev_ycell; a.xcell = p->dev_tables + pp.dev_xcell;
    a.yoff = p->dev_tables + pp.dev_yoff;   a.xoff = p->dev_tables + pp.dev_xoff;
    a.ytile = p->dev_tables + pp.dev_ytile; a.xtile = p->dev_tables + pp.dev_xtile;
    a.wpk = reinterpret_cast<const __nv_bfloat16*>(ws_ptr(ws, backward ? p->ws.wb_off : p->ws.wf_off));
    a.params = params;
    a.error = err_ptr(ws, p);
    // tiles of maps stored as bf16 planes arrive by TMA: the group input (forward), every op's input (backward)
    a.use_tma = 0;
    if (p->tc_tma) {
        const int n_maps = backward ? g.n_ops : 1;
        for (int i = 0; i < n_maps; ++i) {
            const OpDesc& op = a.op[i];
            if (i == 0 && a.in_f32) continue;                          // the network input is fp32 NCHW: converted by the threads
            const MapShape& s = p->maps[op.in_map - 1];
            const int planes = (s.C + 15) / 16 * 2;
            const int bh = backward ? op.t_x_Hp : op.t_in_Hp, bw = backward ? op.t_x_Wp : op.t_in_Wp;
            if (planes != op.cin16 / 8) continue;
            if (encode_plane_map(a.tmap[i], a.map[i], p->N, planes, s.H, s.W, bh, bw)) a.use_tma |= 1u << i;
        }
    }
}

int pack_filters_tc(ftp_plan* p, const float* params, void* ws, cudaStream_t st)
{
    __nv_bfloat16* wf = reinterpret_cast<__nv_bfloat16*>(ws_ptr(ws, p->ws.wf_off));
    __nv_bfloat16* wb = reinterpret_cast<__nv_bfloat16*>(ws_ptr(ws, p->ws.wb_off));
    TcPackArgs pa{};
    auto flush = [&]() {
        if (!pa.n) return;
        Timed t(p, st, 0, -1);
        pack_filters_tc_kernel<<<dim3(64, pa.n), 256, 0, st>>>(pa, params, wf, wb);
        pa.n = 0;
    };
    for (const GroupPlan& g : p->groups)
        for (int i = 0; i < g.n_ops; ++i) {
            const OpDesc& op = g.fwd_ops[i];
            if (op.kind == kOpPool) continue;
            if (pa.n == kMaxOps * 2) flush();
            // (first layer on the window-unrolled input: a 1x1 conv with 9 cin input channels, same parameters)
            if (g.col_cin16) pa.l[pa.n++] = TcPackLayer{op.p_off, op.twf_off, g.col_cin, op.cout, 1, g.col_cin16, op.cout16,
                                                        1, g.cf.Ns, g.cf.kpc, g.cd.Ns, g.cd.kpc};
            else pa.l[pa.n++] = TcPackLayer{op.p_off, op.twf_off, op.cin, op.cout, op.k, op.cin16, op.cout16,
                                            g.tfg.on ? 1 : 0, g.cf.Ns, g.cf.kpc, g.cd.Ns, g.cd.kpc};
        }
    flush();
    return launched_ok() ? FTP_OK : FTP_ERR_CUDA;
}

int forward_tc(ftp_plan* p, const float* x, const float* params, float* y, void* ws, cudaStream_t st)
{
    if (cudaMemsetAsync(err_ptr(ws, p), 0, 4, st) != cudaSuccess) return FTP_ERR_CUDA;
    int rc = pack_filters_tc(p, params, ws, st);
    if (rc != FTP_OK) return rc;
    for (size_t gi = 0; gi < p->groups.size(); ++gi) {
        const GroupPlan& g = p->groups[gi];
        TcGroupArgs a;
        fill_common_tc(p, g, false, x, params, ws, a);
        if (g.tfg.on) {                         // one conv: the banded kernel
            const OpDesc& op = g.fwd_ops[0];
            const __nv_bfloat16* wf = reinterpret_cast<const __nv_bfloat16*>(ws_ptr(ws, p->ws.wf_off)) + op.twf_off;
            const void* in = a.map[0];
            if (g.col_cin16) {                  // first layer: a 1x1 conv on the window-unrolled network input
                uint4* col = reinterpret_cast<uint4*>(ws_ptr(ws, p->ws.col_off));
                { Timed t(p, st, 9, (int)gi);
                  launch_unroll_windows(x, col, p->N, op.cin, op.in_H, op.in_W, st); }
                if (!launched_ok()) return FTP_ERR_CUDA;
                in = col;
            }
            if (!launch_tc_conv(p, g.cf, 1, (int)gi, in, wf, params + op.p_off + (size_t)op.cout * op.cin * op.k * op.k,
                                a.map_out[1], a.arg[0], g.tfg.k, g.col_cin16 ? g.col_cin16 : op.cin16, op.cout16, op.cout, op.in_H, op.in_W,
                                op.kind == kOpConvPool, op.slope, a.error, st))
                return FTP_ERR_CUDA;
            continue;
        }
        const int items = a.R * a.Q * p->N;
        { Timed t(p, st, 1, (int)gi);
          const size_t smem = tc_smem(g.fwd.smem_bytes, g.fwd.ctas);
          const int blocks = std::min(items, kSmCount * g.fwd.ctas), tile_bytes = (int)(smem - tc_fixed_bytes(g.fwd.stages));
          // two blocks of 256 threads per SM, or one of 512: the phases around the MMAs want all the warps they can get
          if (g.fwd.ctas == 2) fwd_group_tc_kernel<256><<<blocks, 256, smem, st>>>(a, tile_bytes, kTcTmemCols / 2, g.fwd.stages);
          else fwd_group_tc_kernel<512><<<blocks, 512, smem, st>>>(a, tile_bytes, kTcTmemCols, g.fwd.stages); }
        if (!launched_ok()) return FTP_ERR_CUDA;
    }
    if (y) {
        const MapShape& s = p->maps.back();
        const size_t total = (size_t)p->N * s.C * s.H * s.W;
        const int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)kSmCount * 16);
        ++p->launches;
        planes_to_nchw_kernel<<<blocks, 256, 0, st>>>(
            reinterpret_cast<const __nv_bfloat16*>(map_ptr(p, x, ws, (int)p->layers.size() + 1)), y, p->N, s.C,
            (s.C + 15) / 16 * 16, s.H, s.W);
        if (!launched_ok()) return FTP_ERR_CUDA;
    }
    return FTP_OK;
}

// One-conv group run weight-stationary (stationary.cuh): the convolution with bias, activation and, where a
// pool follows, the 2x2 maximum and its arg-max, written to the group's output map.
bool stationary_forward(ftp_plan* p, const GroupPlan& g, int gi, const float* x, const float* params, void* ws, cudaStream_t st)
{
    const OpDesc& op = g.fwd_ops[0];
    ConvRowsArgs a{};
    a.in = map_ptr(p, x, ws, g.first);
    a.w = ws_ptr(ws, p->ws.wf_off) + op.wf_off;
    a.bias = params + op.p_off + (size_t)op.cout * op.cin * op.k * op.k;
    a.out = const_cast<float*>(map_ptr(p, x, ws, op.out_map));
    a.arg = g.st.pool ? static_cast<unsigned char*>(ws) + p->ws.arg_off[op.out_map - 1] : nullptr;
    a.N = p->N; a.Cin = op.cin; a.Cout = op.cout; a.CoutPad = op.cout_pad; a.H = op.in_H; a.W = op.in_W;
    a.slope = op.slope; a.act = 1; a.pool = g.st.pool;
    { Timed t(p, st, 1, gi);
      st_launch_conv_rows(a, op.k, g.st.fwd_co_tile, g.st.fwd_threads, g.st.fwd_blocks, st); }
    return launched_ok();
}

// Backward of such a group: the delta in front of the activation at the conv's resolution, the partial filter
// and bias gradients (one set per share of the pixels), and the input delta as the convolution of that
// delta with the rotated filters (Section 4.1), written whole to `din` (may be null: not wanted).
bool stationary_backward(ftp_plan* p, const GroupPlan& g, int gi, const float* x, const float* params, const float* dout, float* din,
                         void* ws, cudaStream_t st)
{
    const OpDesc& op = g.bwd_ops[0];
    const int H = op.in_H, W = op.in_W;
    if (g.st.thin) {
        ThinBwdArgs t{};
        t.dyp = dout; t.yp = map_ptr(p, x, ws, op.out_map);
        t.arg = static_cast<unsigned char*>(ws) + p->ws.arg_off[op.out_map - 1];
        t.x = map_ptr(p, x, ws, g.first); t.filter = params + op.p_off; t.dx = din;
        t.partial = ws_ptr(ws, g.partial_off); t.set_floats = (long long)g.param_floats;
        t.filter_off = op.gp_off; t.bias_off = op.gp_off + (long long)op.cout * op.cin * 9;
        t.N = p->N; t.Cin = op.cin; t.Cout = op.cout; t.OH = op.out_H; t.OW = op.out_W;
        t.tiles_y = g.st.thin_tiles_y; t.tiles_x = g.st.thin_tiles_x; t.slope = op.slope;
        { Timed tm(p, st, 3, gi);
          st_launch_thin_bwd(t, g.st.thin_blocks, st); }
        return launched_ok();
    }
    // The filter gradient and the input delta both read dZ and nothing else of each other, so the filter gradient
    // runs on the plan's side stream: the blocks of one kernel fill the SMs that the last, partly filled round of the
    // other leaves idle.  dZ areas are taken in turn; an area is reused only after the filter gradient that read it.
    // (With per-launch timing or per-group notification on, everything stays on the caller's stream.)
    const bool side = !p->timing && !p->group_ready && din != nullptr;
    const int turn = p->dz_turn++ & 1;
    cudaStream_t gs = side ? static_cast<cudaStream_t>(p->grad_stream) : st;
    float* dz = ws_ptr(ws, p->ws.dz_off + (size_t)turn * p->ws.dz_bytes);
    const float* y = map_ptr(p, x, ws, op.out_map);
    const unsigned char* arg = g.st.pool ? static_cast<unsigned char*>(ws) + p->ws.arg_off[op.out_map - 1] : nullptr;
    const size_t count = (size_t)p->N * op.cout * op.out_H * op.out_W;
    if (p->fg_pending[turn]) {
        if (cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(p->ev_fg[turn]), 0) != cudaSuccess) return false;
        p->fg_pending[turn] = false;
    }
    { Timed t(p, st, 6, gi);
      st_launch_delta_act(dout, y, arg, dz, count, op.out_W, op.slope, g.st.pool, st); }
    if (!launched_ok()) return false;
    if (side && (cudaEventRecord(static_cast<cudaEvent_t>(p->ev_dz[turn]), st) != cudaSuccess ||
                 cudaStreamWaitEvent(gs, static_cast<cudaEvent_t>(p->ev_dz[turn]), 0) != cudaSuccess)) return false;
    FilterGradRowsArgs f{};
    f.dz = dz; f.x = map_ptr(p, x, ws, g.first);
    f.partial = ws_ptr(ws, g.partial_off); f.set_floats = (long long)g.param_floats;
    f.filter_off = op.gp_off; f.bias_off = op.gp_off + (long long)op.cout * op.cin * op.k * op.k;
    f.N = p->N; f.Cin = op.cin; f.Cout = op.cout; f.H = H; f.W = W;
    f.stages = g.st.fg_stages; f.splits = g.st.fg_splits;
    { Timed t(p, gs, 7, gi);
      st_launch_filter_grad_rows(f, op.k, g.st.fg_blocks, gs); }
    if (!launched_ok()) return false;
    if (side) {
        if (cudaEventRecord(static_cast<cudaEvent_t>(p->ev_fg[turn]), gs) != cudaSuccess) return false;
        p->fg_pending[turn] = true;
    }
    if (din) {
        ConvRowsArgs a{};
        a.in = dz;
        a.w = ws_ptr(ws, p->ws.wb_off) + op.wb_off;
        a.bias = nullptr; a.out = din; a.arg = nullptr;
        a.N = p->N; a.Cin = op.cout; a.Cout = op.cin; a.CoutPad = op.cin_pad; a.H = H; a.W = W;
        a.slope = 0.f; a.act = 0; a.pool = 0;
        { Timed t(p, st, 8, gi);
          st_launch_conv_rows(a, op.k, g.st.dx_co_tile, g.st.dx_threads, g.st.dx_blocks, st); }
        if (!launched_ok()) return false;
    }
    return true;
}

int forward_impl(ftp_plan* p, const float* x, const float* params, float* y, void* ws, cudaStream_t st)
{
    if (is_tc(p)) return forward_tc(p, x, params, y, ws, st);
    int rc = pack_filters(p, params, ws, st);
    if (rc != FTP_OK) return rc;
    for (size_t gi = 0; gi < p->groups.size(); ++gi) {
        const GroupPlan& g = p->groups[gi];
        if (g.st.on) {
            if (!stationary_forward(p, g, (int)gi, x, params, ws, st)) return FTP_ERR_CUDA;
            continue;
        }
        GroupArgs a;
        fill_common(p, g, false, x, params, ws, a);
        { Timed t(p, st, 1, (int)gi);
          if (max_window(g) <= 3) fwd_group_kernel<3><<<dim3(a.R * a.Q, p->N), kThreads, g.fwd.smem_bytes, st>>>(a);
          else fwd_group_kernel<7><<<dim3(a.R * a.Q, p->N), kThreads, g.fwd.smem_bytes, st>>>(a); }
        if (!launched_ok()) return FTP_ERR_CUDA;
    }
    if (y) {
        const MapShape& s = p->maps.back();
        const size_t bytes = (size_t)p->N * s.C * s.H * s.W * sizeof(float);
        if (cudaMemcpyAsync(y, map_ptr(p, x, ws, (int)p->layers.size() + 1), bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return FTP_ERR_CUDA;
    }
    return FTP_OK;
}

// A layer's entry for the cross-tile reduction: where its slice of the partial sets lies and how it is arranged (the
// first layer on the window-unrolled input: as the 1x1 conv with 9 cin input channels that computed it).
TcReduceLayer reduce_layer(const GroupPlan& g, const OpDesc& op, void* ws)
{
    if (g.col_cin16)
        return TcReduceLayer{op.p_off, ws_ptr(ws, g.partial_off), (long long)g.param_floats, op.tgp_off, g.sets(), g.col_cin, op.cout, 1,
                             g.col_cin16, op.cout16};
    return TcReduceLayer{op.p_off, ws_ptr(ws, g.partial_off), (long long)g.param_floats, op.tgp_off, g.sets(), op.cin, op.cout, op.k,
                         op.cin16, op.cout16};
}

// Backward pass of a one-conv bf16 group: dz planes at the conv's resolution, the filter gradient by the
// weight-stationary tensor-core kernel over bands of the whole batch (one partial set per pixel share), and the delta
// at the group's input.
bool tc_filter_grad(ftp_plan* p, const GroupPlan& g, int gi, const TcGroupArgs& a, void* ws, bool need_dx, float* dx, cudaStream_t st)
{
    const OpDesc& op = g.bwd_ops[0];
    const TcFgPlan& t = g.tfg;
    // the layer's input as bf16 planes: the saved map, or (first layer) the window-unrolled network input of the forward pass
    void* xin = g.col_cin16 ? static_cast<void*>(ws_ptr(ws, p->ws.col_off)) : const_cast<void*>(a.map[0]);
    const int cin16 = g.col_cin16 ? g.col_cin16 : op.cin16;
    // dz planes: the two areas take turns; when the group above is a one-conv group too, its input-delta kernel has
    // already written this group's dz (see below), otherwise delta_act_planes_kernel makes them from the stored delta
    const int G = (int)p->groups.size();
    uint4* dz = reinterpret_cast<uint4*>(ws_ptr(ws, p->ws.dz_off + (size_t)(gi & 1) * p->ws.dz_bytes));
    uint4* dz_below = reinterpret_cast<uint4*>(ws_ptr(ws, p->ws.dz_off + (size_t)((gi + 1) & 1) * p->ws.dz_bytes));
    const bool dz_ready = gi + 1 < G && p->groups[gi + 1].tfg.on;
    const bool feeds_below = gi > 0 && p->groups[gi - 1].tfg.on;
    DeltaActPlanesArgs d{};
    d.dmap = a.dmap_out; d.dmap_planes = a.dmap_planes;
    d.y = static_cast<const uint4*>(a.map[1]);
    d.arg = reinterpret_cast<const unsigned long long*>(a.arg[0]);
    d.dz = dz;
    d.N = p->N; d.cout = op.cout; d.cout16 = op.cout16; d.out_H = op.out_H; d.out_W = op.out_W;
    d.pool = op.kind == kOpConvPool ? 1 : 0;
    d.slope = op.slope;
    const size_t total = (size_t)p->N * (op.cout16 / 8) * op.out_H * op.out_W;
    if (!dz_ready) {
        { Timed tm(p, st, 6, gi);
          delta_act_planes_kernel<<<(int)std::min<size_t>((total + 255) / 256, (size_t)kSmCount * 16), 256, 0, st>>>(d); }
        if (!launched_ok()) return false;
    }

    TcFilterGradArgs f{};
    for (int cc = 0; cc < t.ncc; ++cc)          // one dz map per column chunk: its columns only, zeros behind them
        if (!encode_rows_map(f.tmap_dz[cc], dz + (size_t)cc * t.Cw, p->N, op.cout16 / 8, op.in_H, std::min(t.Cw, op.in_W - cc * t.Cw),
                             op.in_W, t.R, t.Wp))
            return false;
    if (!encode_rows_map(f.tmap_x, xin, p->N, cin16 / 8, op.in_H, op.in_W, op.in_W, t.R + t.k - 1, t.Wp)) return false;
    f.ncc = t.ncc; f.Cw = t.Cw;
    f.partial = a.partial; f.set_floats = a.set_floats; f.tgp_off = op.tgp_off;
    f.error = a.error;
    f.N = p->N; f.K = t.k; f.cout16 = op.cout16; f.cin16 = cin16;
    f.Ms = t.Ms; f.slices = t.slices; f.ncols = t.ncols; f.nci = t.nci;
    f.R = t.R; f.Wp = t.Wp; f.bands_img = t.bands_img; f.bands = t.bands; f.shares = t.shares;
    f.dz_plane = t.dz_plane; f.x_plane = t.x_plane; f.stage_bytes = t.stage_bytes;
    { Timed tm(p, st, 7, gi);
      filter_grad_tc_rows_kernel<<<t.blocks, kTcFgThreads, t.smem_bytes, st>>>(f); }
    if (!launched_ok()) return false;

    // input delta: the convolution of dz with the rotated filters (dz planes in, delta planes out)
    if (!need_dx) return true;
    const __nv_bfloat16* wb = reinterpret_cast<const __nv_bfloat16*>(ws_ptr(ws, p->ws.wb_off)) + op.twb_off;
    if (!g.col_cin16) {
        if (!feeds_below)
            return launch_tc_conv(p, g.cd, 8, gi, dz, wb, nullptr, ws_ptr(ws, p->ws.dmap_off[gi]), nullptr, t.k, op.cout16, cin16, op.cin,
                                  op.in_H, op.in_W, false, 1.0f, a.error, st);
        const OpDesc& below = p->groups[gi - 1].fwd_ops[0];       // its output map is this group's input map
        PrevLayer pv{static_cast<const uint4*>(a.map[0]),
                     below.kind == kOpConvPool ? reinterpret_cast<const unsigned long long*>(static_cast<unsigned char*>(ws) + p->ws.arg_off[below.out_map - 1])
                                               : nullptr,
                     below.slope};
        return launch_tc_conv(p, g.cd, 8, gi, dz, wb, nullptr, dz_below, nullptr, t.k, op.cout16, cin16, op.cin,
                              op.in_H, op.in_W, false, 1.0f, a.error, st, &pv);
    }
    // first layer: the delta of the window-unrolled input (in the dz area that is not in use, sized for it; the unrolled
    // input stays as the forward pass left it), folded back into the caller's fp32 map
    if (!launch_tc_conv(p, g.cd, 8, gi, dz, wb, nullptr, dz_below, nullptr, 1, op.cout16, cin16, g.col_cin, op.in_H, op.in_W, false, 1.0f,
                        a.error, st))
        return false;
    { Timed tm(p, st, 10, gi);
      launch_fold_windows(reinterpret_cast<const __nv_bfloat16*>(dz_below), dx, p->N, op.cin, op.in_H, op.in_W, st); }
    return launched_ok();
}

int backward_tc(ftp_plan* p, const float* x, const float* dy, const float* params, float* dx, float* grad_out,
                float* sgd_params, float lr, void* ws, cudaStream_t st)
{
    const int G = (int)p->groups.size();
    for (int gi = G - 1; gi >= 0; --gi) {
        const GroupPlan& g = p->groups[gi];
        TcGroupArgs a;
        fill_common_tc(p, g, true, x, params, ws, a);
        a.dmap_out = gi == G - 1 ? static_cast<const void*>(dy) : static_cast<const void*>(ws_ptr(ws, p->ws.dmap_off[gi + 1]));
        a.dmap_planes = gi == G - 1 ? 0 : 1;
        a.scratch = ws_ptr(ws, p->ws.scratch_off);
        a.partial = ws_ptr(ws, g.partial_off);
        a.set_floats = (long long)g.param_floats;
        
        a.need_dx = (gi > 0 || dx != nullptr) ? 1 : 0;
        if (g.tfg.on) {
            // one conv behind the first layer: the filter gradient by the weight-stationary kernel, the delta at the group's input as a
            // convolution of dz with the rotated filters (written whole: nothing to sum afterwards)
            if (!tc_filter_grad(p, g, gi, a, ws, a.need_dx != 0, dx, st)) return FTP_ERR_CUDA;
        } else
        { Timed t(p, st, 3, gi);
          const size_t smem = tc_smem(g.bwd.smem_bytes, g.bwd.ctas);
          const int tile_bytes = (int)(smem - tc_fixed_bytes(g.bwd.stages));
          if (g.bwd.ctas == 2) bwd_group_tc_kernel<256><<<g.bwd.blocks, 256, smem, st>>>(a, tile_bytes, kTcTmemCols / 2, g.bwd.stages);
          else bwd_group_tc_kernel<512><<<g.bwd.blocks, 512, smem, st>>>(a, tile_bytes, kTcTmemCols, g.bwd.stages); }
        if (!launched_ok()) return FTP_ERR_CUDA;
        if (p->group_ready && g.param_floats) {       // ftp_step_grad_groups: this group's sets are summed right away
            TcReduceArgs rg{};
            for (int i = 0; i < g.n_ops; ++i) {
                const OpDesc& op = g.bwd_ops[i];
                if (op.kind == kOpPool) continue;
                rg.l[rg.n++] = reduce_layer(g, op, ws);
            }
            { Timed t(p, st, 5, gi);
              reduce_sgd_tc_kernel<<<dim3(1184, rg.n), 128, 0, st>>>(rg, nullptr, 0.f, grad_out); }
            if (!launched_ok()) return FTP_ERR_CUDA;
            long long floats = 0;
            for (int i = 0; i < g.n_ops; ++i)
                if (g.bwd_ops[i].kind != kOpPool) floats += (long long)g.bwd_ops[i].cout * g.bwd_ops[i].cin * g.bwd_ops[i].k * g.bwd_ops[i].k + g.bwd_ops[i].cout;
            p->group_ready(p->group_ready_user, gi, g.param_begin, floats);
        }
        if (a.need_dx && !g.tfg.on) {
            const MapShape& s = p->maps[g.first - 1];
            const bool planes = g.first > 1;          // group input is a saved bf16 map: deltas travel as planes too
            HaloSumArgs h{};
            h.scratch = a.scratch;
            h.out = gi == 0 ? dx : ws_ptr(ws, p->ws.dmap_off[gi]);
            h.yspan = a.yspan; h.xspan = a.xspan; h.yoff = a.yoff; h.xoff = a.xoff;
            h.ycover = p->dev_tables + g.bwd.dev_ycover; h.xcover = p->dev_tables + g.bwd.dev_xcover;
            h.N = p->N; h.C = planes ? (s.C + 15) / 16 * 16 : s.C; h.H = s.H; h.W = s.W; h.R = a.R; h.Q = a.Q;
            h.Htot = g.bwd.y.scratch_off[a.R]; h.Wtot = g.bwd.x.scratch_off[a.Q];
            const size_t rows = (size_t)p->N * (planes ? h.C / 8 : h.C) * s.H;
            const int blocks = (int)std::min<size_t>((rows + 7) / 8, (size_t)kSmCount * 16);
            const size_t tab = (size_t)(2 * h.W + 2 * h.H + 3 * h.Q + 3 * h.R + 2) * sizeof(int);
            { Timed t(p, st, 4, gi);
              if (planes) halo_sum_planes_kernel<<<blocks, 256, tab, st>>>(h);
              else halo_sum_kernel<<<blocks, 256, tab, st>>>(h); }
            if (!launched_ok()) return FTP_ERR_CUDA;
        }
    }
    if (p->group_ready) return launched_ok() ? FTP_OK : FTP_ERR_CUDA;      // summed group by group above
    TcReduceArgs ra{};
    auto flush = [&]() {
        if (!ra.n) return;
        Timed t(p, st, 5, -1);
        reduce_sgd_tc_kernel<<<dim3(1184, ra.n), 128, 0, st>>>(ra, sgd_params, lr, grad_out);
        ra.n = 0;
    };
    for (const GroupPlan& g : p->groups)
        for (int i = 0; i < g.n_ops; ++i) {
            const OpDesc& op = g.bwd_ops[i];
            if (op.kind == kOpPool) continue;
            if (ra.n == kMaxOps * 2) flush();
            ra.l[ra.n++] = reduce_layer(g, op, ws);
        }
    flush();
    return launched_ok() ? FTP_OK : FTP_ERR_CUDA;
}

// ftp_step_grad_groups: the sum of ONE executed group's partial sets, launched as soon as its backward pass is
// queued, and the caller's notification.  Same per-parameter sums as the reduction over all groups.
int reduce_group_and_notify(ftp_plan* p, int gi, float* grad_out, void* ws, cudaStream_t st)
{
    const GroupPlan& g = p->groups[gi];
    if (g.param_floats == 0) return FTP_OK;
    ReduceArgs ra{};
    ra.n = 1;
    ra.g[0] = ReduceGroup{g.param_begin, (long long)g.param_floats, ws_ptr(ws, g.partial_off), g.bwd.blocks};
    const long long first = g.param_begin, total = g.param_begin + (long long)g.param_floats;
    const int blocks = (int)std::min<long long>(((long long)g.param_floats + 255) / 256, (long long)kSmCount * 16);
    { Timed t(p, st, 5, gi);
      reduce_sgd_kernel<<<blocks, 256, 0, st>>>(ra, first, total, nullptr, 0.f, grad_out); }
    if (!launched_ok()) return FTP_ERR_CUDA;
    p->group_ready(p->group_ready_user, gi, first, (long long)g.param_floats);
    return FTP_OK;
}

// Backward of all groups in reverse order, halo sums at the group inputs, then the cross-tile
// reduction; `sgd_params` non-null applies the update in the same kernel.
int backward_impl(ftp_plan* p, const float* x, const float* dy, const float* params, float* dx, float* grad_out,
                  float* sgd_params, float lr, void* ws, cudaStream_t st)
{
    if (is_tc(p)) return backward_tc(p, x, dy, params, dx, grad_out, sgd_params, lr, ws, st);
    const int G = (int)p->groups.size();
    for (int gi = G - 1; gi >= 0; --gi) {
        const GroupPlan& g = p->groups[gi];
        if (g.st.on) {
            const float* dout = gi == G - 1 ? dy : ws_ptr(ws, p->ws.dmap_off[gi + 1]);
            float* din = gi == 0 ? dx : ws_ptr(ws, p->ws.dmap_off[gi]);
            if (!stationary_backward(p, g, gi, x, params, dout, din, ws, st)) return FTP_ERR_CUDA;
            if (p->group_ready) { const int rc = reduce_group_and_notify(p, gi, grad_out, ws, st); if (rc != FTP_OK) return rc; }
            continue;
        }
        GroupArgs a;
        fill_common(p, g, true, x, params, ws, a);
        a.dmap_out = gi == G - 1 ? dy : ws_ptr(ws, p->ws.dmap_off[gi + 1]);
        a.scratch = ws_ptr(ws, p->ws.scratch_off);
        a.partial = ws_ptr(ws, g.partial_off);
        a.param_floats = (long long)g.param_floats;
        
        a.need_dx = (gi > 0 || dx != nullptr) ? 1 : 0;
        { Timed t(p, st, 3, gi);
          if (max_window(g) <= 3) bwd_group_kernel<3><<<g.bwd.blocks, kThreads, g.bwd.smem_bytes, st>>>(a);
          else bwd_group_kernel<7><<<g.bwd.blocks, kThreads, g.bwd.smem_bytes, st>>>(a); }
        if (!launched_ok()) return FTP_ERR_CUDA;
        if (p->group_ready) { const int rc = reduce_group_and_notify(p, gi, grad_out, ws, st); if (rc != FTP_OK) return rc; }
        if (a.need_dx) {
            const MapShape& s = p->maps[g.first - 1];
            HaloSumArgs h{};
            h.scratch = a.scratch;
            h.out = gi == 0 ? dx : ws_ptr(ws, p->ws.dmap_off[gi]);
            h.yspan = a.yspan; h.xspan = a.xspan; h.yoff = a.yoff; h.xoff = a.xoff;
            h.ycover = p->dev_tables + g.bwd.dev_ycover; h.xcover = p->dev_tables + g.bwd.dev_xcover;
            h.N = p->N; h.C = s.C; h.H = s.H; h.W = s.W; h.R = a.R; h.Q = a.Q;
            h.Htot = g.bwd.y.scratch_off[a.R]; h.Wtot = g.bwd.x.scratch_off[a.Q];
            const size_t rows = (size_t)p->N * s.C * s.H;
            const int blocks = (int)std::min<size_t>((rows + 7) / 8, (size_t)kSmCount * 16);
            { Timed t(p, st, 4, gi);
              halo_sum_kernel<<<blocks, 256, (size_t)(2 * h.W + 2 * h.H + 3 * h.Q + 3 * h.R + 2) * sizeof(int), st>>>(h); }
            if (!launched_ok()) return FTP_ERR_CUDA;
        }
    }
    for (int turn = 0; turn < 2; ++turn)     // the filter gradients on the side stream join here
        if (p->fg_pending[turn]) {
            if (cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(p->ev_fg[turn]), 0) != cudaSuccess) return FTP_ERR_CUDA;
            p->fg_pending[turn] = false;
        }
    if (p->group_ready) return FTP_OK;       // every group's sets were summed right after its backward pass
    ReduceArgs ra{};
    for (const GroupPlan& g : p->groups) {
        if (g.param_floats == 0) continue;
        ra.g[ra.n++] = ReduceGroup{g.param_begin, (long long)g.param_floats, ws_ptr(ws, g.partial_off), g.bwd.blocks};
    }
    if (ra.n) {
        const long long total = (long long)p->param_floats;
        const int blocks = (int)std::min<long long>((total + 255) / 256, (long long)kSmCount * 16);
        { Timed t(p, st, 5, -1);
          reduce_sgd_kernel<<<blocks, 256, 0, st>>>(ra, 0, total, sgd_params, lr, grad_out); }
        if (!launched_ok()) return FTP_ERR_CUDA;
    }
    return FTP_OK;
}

bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

}  // namespace

extern "C" {

int ftp_plan_create_opts(const ftp_layer* layers, int n_layers, int N, int C, int H, int W, int grid_y, int grid_x,
                         const ftp_group* groups, int n_groups, int precision, const ftp_plan_opts* opts,
                         ftp_plan** out)
{
    if (!out) return FTP_ERR_ARG;
    *out = nullptr;
    PlanOpts po;
    if (opts) {
        if (opts->struct_size != (int)sizeof(ftp_plan_opts)) return FTP_ERR_ARG;
        if (opts->max_redundancy_pct) po.max_redundancy_pct = opts->max_redundancy_pct;
        if (opts->max_subtile) po.max_subtile = opts->max_subtile;
        if (opts->smem_bytes) po.smem_bytes = opts->smem_bytes;
        po.strict_groups = opts->strict_groups;
        if (opts->tc_blocks_per_sm < 0 || opts->tc_blocks_per_sm > 2) return FTP_ERR_ARG;
        po.tc_ctas = opts->tc_blocks_per_sm;
        if (opts->max_group_convs < -1) return FTP_ERR_ARG;
        if (opts->max_group_convs) po.max_group_convs = opts->max_group_convs < 0 ? 0 : opts->max_group_convs;
        if (opts->cost_model < -1 || opts->cost_model > 1) return FTP_ERR_ARG;
        po.cost_model = opts->cost_model ? (opts->cost_model > 0 ? 1 : 0) : (opts->max_group_convs ? 0 : 1);
        if (opts->stationary < -1 || opts->stationary > 1) return FTP_ERR_ARG;
        po.stationary = opts->stationary;
        if (opts->tc_tma < -1 || opts->tc_tma > 0) return FTP_ERR_ARG;
        po.tc_tma = opts->tc_tma;
    }
    ftp_plan* p = new (std::nothrow) ftp_plan();
    if (!p) return FTP_ERR_ARG;
    int rc = FTP_ERR_ARG;
    try {
        rc = build_plan(*p, layers, n_layers, N, C, H, W, grid_y, grid_x, groups, n_groups, precision, po);
    } catch (...) {
        rc = FTP_ERR_ARG;
    }
    if (rc != FTP_OK) { delete p; return rc; }
    *out = p;
    return FTP_OK;
}

int ftp_plan_create(const ftp_layer* layers, int n_layers, int N, int C, int H, int W, int grid_y, int grid_x,
                    const ftp_group* groups, int n_groups, int precision, ftp_plan** out)
{
    return ftp_plan_create_opts(layers, n_layers, N, C, H, W, grid_y, grid_x, groups, n_groups, precision, nullptr, out);
}

int ftp_plan_exec_groups(const ftp_plan* plan, int* n_groups, ftp_group* groups_out, int capacity)
{
    if (!plan || !n_groups) return FTP_ERR_ARG;
    *n_groups = (int)plan->groups.size();
    if (groups_out)
        for (int i = 0; i < *n_groups && i < capacity; ++i) groups_out[i] = ftp_group{plan->groups[i].first, plan->groups[i].last};
    return FTP_OK;
}

int ftp_plan_group_mode(const ftp_plan* plan, int group, int* stationary, int* partial_sets)
{
    if (!plan || !stationary || group < 0 || group >= (int)plan->groups.size()) return FTP_ERR_ARG;
    *stationary = plan->groups[group].st.on ? 1 : plan->groups[group].tfg.on ? 2 : 0;
    if (partial_sets) *partial_sets = plan->groups[group].sets();
    return FTP_OK;
}

void ftp_plan_destroy(ftp_plan* plan)
{
    if (!plan) return;
    ftp_plan_timing(plan, 0);
    if (plan->dev_tables) cudaFree(plan->dev_tables);
    if (plan->grad_stream) {
        cudaStreamDestroy(static_cast<cudaStream_t>(plan->grad_stream));
        for (int i = 0; i < 2; ++i) {
            cudaEventDestroy(static_cast<cudaEvent_t>(plan->ev_dz[i]));
            cudaEventDestroy(static_cast<cudaEvent_t>(plan->ev_fg[i]));
        }
    }
    if (plan->copy_stream) {
        cudaStreamDestroy(static_cast<cudaStream_t>(plan->copy_stream));
        cudaEventDestroy(static_cast<cudaEvent_t>(plan->ev_fork));
        cudaEventDestroy(static_cast<cudaEvent_t>(plan->ev_join));
        cudaEventDestroy(static_cast<cudaEvent_t>(plan->ev_prefetch));
        cudaEventDestroy(static_cast<cudaEvent_t>(plan->ev_slot_free[0]));
        cudaEventDestroy(static_cast<cudaEvent_t>(plan->ev_slot_free[1]));
    }
    delete plan;
}

int ftp_plan_region(const ftp_plan* plan, int pass, int group, int map_index, int ty, int tx, int span_out[4])
{
    if (!plan) return FTP_ERR_ARG;
    return region(*plan, pass, group, map_index, ty, tx, span_out);
}

int ftp_plan_sizes(const ftp_plan* plan, size_t* param_floats, size_t* workspace_bytes, size_t* out_floats,
                   double* redundancy)
{
    if (!plan) return FTP_ERR_ARG;
    if (param_floats) *param_floats = plan->param_floats;
    if (workspace_bytes) *workspace_bytes = plan->ws.total;
    if (out_floats) {
        const MapShape& s = plan->maps.back();
        *out_floats = (size_t)plan->N * s.C * s.H * s.W;
    }
    if (redundancy) {
        double done = 0, base = 0;
        for (const GroupPlan& g : plan->groups) { done += g.macs_done; base += g.macs_untiled; }
        *redundancy = base > 0 ? done / base : 1.0;
    }
    return FTP_OK;
}

int ftp_plan_subtiles(const ftp_plan* plan, int pass, int group, int* rows, int* cols, size_t* smem_bytes, int* blocks)
{
    if (!plan || group < 0 || group >= (int)plan->groups.size() || pass < 0 || pass > 1) return FTP_ERR_ARG;
    const GroupPlan& gp = plan->groups[group];
    if (gp.st.on) {         // weight-stationary group: row-pair tiles of the whole batch x column tiles, 256-thread blocks
        const OpDesc& op = gp.fwd_ops[0];
        const int per = pass ? kFgRowPairs : st_row_pairs(gp.st.fwd_co_tile, gp.st.fwd_threads);
        if (rows) *rows = (plan->N * ((op.in_H + 1) / 2) + per - 1) / per;
        if (cols) *cols = (op.in_W + kStCols - 1) / kStCols;
        if (smem_bytes) *smem_bytes = pass ? st_filter_grad_smem_bytes(op.k) : st_conv_smem_bytes(op.k, gp.st.fwd_co_tile, gp.st.fwd_threads);
        if (blocks) *blocks = pass ? gp.st.fg_blocks : gp.st.fwd_blocks;
        return FTP_OK;
    }
    const PassPlan& pp = pass ? plan->groups[group].bwd : plan->groups[group].fwd;
    if (rows) *rows = pp.y.count;
    if (cols) *cols = pp.x.count;
    if (smem_bytes) *smem_bytes = pp.smem_bytes;
    if (blocks) *blocks = pp.blocks;
    return FTP_OK;
}

int ftp_plan_delta_staging(const ftp_plan* plan, int group, int* channels)
{
    if (!plan || !channels || group < 0 || group >= (int)plan->groups.size()) return FTP_ERR_ARG;
    *channels = plan->groups[group].bwd.dz_ch;
    return FTP_OK;
}

int ftp_plan_cost(const ftp_plan* plan, int pass, int group, int need_dx, double* terms, double* estimate_us)
{
    if (!plan) return FTP_ERR_ARG;
    double t[kCostTerms];
    const int rc = cost_terms(*plan, pass, group, need_dx, t, estimate_us);
    if (rc == FTP_OK && terms) for (int k = 0; k < kCostTerms; ++k) terms[k] = t[k];
    return rc;
}

int ftp_forward(ftp_plan* plan, const float* x, const float* params, float* y, void* workspace, void* stream)
{
    if (!plan || !x || !params || !workspace || !aligned256(workspace)) return FTP_ERR_ARG;
    int rc = ensure_device(plan);
    if (rc != FTP_OK) return rc;
    return forward_impl(plan, x, params, y, workspace, static_cast<cudaStream_t>(stream));
}

int ftp_backward(ftp_plan* plan, const float* x, const float* dy, const float* params, float* dx, float* dparams,
                 void* workspace, void* stream)
{
    if (!plan || !x || !dy || !params || !dparams || !workspace || !aligned256(workspace)) return FTP_ERR_ARG;
    int rc = ensure_device(plan);
    if (rc != FTP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = is_tc(plan) ? pack_filters_tc(plan, params, workspace, st) : pack_filters(plan, params, workspace, st);
    if (rc != FTP_OK) return rc;
    return backward_impl(plan, x, dy, params, dx, dparams, nullptr, 0.f, workspace, st);
}

static int step_impl(ftp_plan* plan, const float* x, const float* dy, const float* target, const float* params,
                     float* sgd_params, float lr, float* grad_out, float* loss_out, float* dx, void* workspace,
                     void* stream, cudaEvent_t target_ready = nullptr)
{
    if (!plan || !x || !params || !workspace || !aligned256(workspace)) return FTP_ERR_ARG;
    if ((dy == nullptr) == (target == nullptr)) return FTP_ERR_ARG;
    int rc = ensure_device(plan);
    if (rc != FTP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* y32 = (is_tc(plan) && target) ? ws_ptr(workspace, plan->ws.y32_off) : nullptr;
    rc = forward_impl(plan, x, params, y32, workspace, st);
    if (rc != FTP_OK) return rc;
    const float* delta = dy;
    if (target_ready && cudaStreamWaitEvent(st, target_ready, 0) != cudaSuccess) return FTP_ERR_CUDA;
    if (target) {
        const MapShape& s = plan->maps.back();
        const size_t M = (size_t)plan->N * s.C * s.H * s.W;
        float* d = ws_ptr(workspace, plan->ws.dy_off);
        float* sums = ws_ptr(workspace, plan->ws.loss_off);
        { Timed t(plan, st, 2, -1);
          mse_delta_kernel<<<plan->loss_blocks, 256, 0, st>>>(y32 ? y32 : map_ptr(plan, x, workspace, (int)plan->layers.size() + 1),
                                                             target, d, M, sums); }
        if (loss_out) {
            Timed t(plan, st, 2, -1);
            mse_finish_kernel<<<1, 256, 0, st>>>(sums, plan->loss_blocks, M, loss_out);
        }
        if (!launched_ok()) return FTP_ERR_CUDA;
        delta = d;
    }
    return backward_impl(plan, x, delta, params, dx, grad_out, sgd_params, lr, workspace, st);
}

int ftp_loss_mse(ftp_plan* plan, const float* y, const float* target, float* dy, float* loss_out, void* workspace,
                 void* stream)
{
    if (!plan || !y || !target || (!dy && !loss_out) || !workspace || !aligned256(workspace)) return FTP_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const MapShape& s = plan->maps.back();
    const size_t M = (size_t)plan->N * s.C * s.H * s.W;
    float* d = dy ? dy : ws_ptr(workspace, plan->ws.dy_off);
    float* sums = ws_ptr(workspace, plan->ws.loss_off);
    { Timed t(plan, st, 2, -1);
      mse_delta_kernel<<<plan->loss_blocks, 256, 0, st>>>(y, target, d, M, sums); }
    if (loss_out) {
        Timed t(plan, st, 2, -1);
        mse_finish_kernel<<<1, 256, 0, st>>>(sums, plan->loss_blocks, M, loss_out);
    }
    return launched_ok() ? FTP_OK : FTP_ERR_CUDA;
}

int ftp_step(ftp_plan* plan, const float* x, const float* dy, const float* target, float* params, float lr,
             float* loss_out, float* dx, void* workspace, void* stream)
{
    return step_impl(plan, x, dy, target, params, params, lr, nullptr, loss_out, dx, workspace, stream);
}

// Side stream and events of the host-batch entry points, created on first use.
static int ensure_copy_stream(ftp_plan* plan)
{
    if (plan->copy_stream) return FTP_OK;
    cudaStream_t cs;
    cudaEvent_t e[5];
    if (cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) != cudaSuccess) return FTP_ERR_CUDA;
    for (cudaEvent_t& ev : e)
        if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return FTP_ERR_CUDA;
    plan->copy_stream = cs; plan->ev_fork = e[0]; plan->ev_join = e[1]; plan->ev_prefetch = e[2];
    plan->ev_slot_free[0] = e[3]; plan->ev_slot_free[1] = e[4];
    return FTP_OK;
}

int ftp_prefetch_host(ftp_plan* plan, const float* x_host, const float* target_host, void* workspace, void* copy_stream)
{
    if (!plan || !x_host || !target_host || !workspace || !aligned256(workspace)) return FTP_ERR_ARG;
    int rc = ensure_device(plan);
    if (rc == FTP_OK) rc = ensure_copy_stream(plan);
    if (rc != FTP_OK) return rc;
    cudaStream_t cs = copy_stream ? static_cast<cudaStream_t>(copy_stream) : static_cast<cudaStream_t>(plan->copy_stream);
    const MapShape& in = plan->maps.front();
    const MapShape& out = plan->maps.back();
    const int slot = 1 - plan->cur_slot;          // the slot the last (possibly still running) step does not read
    float* xs = ws_ptr(workspace, plan->ws.x_stage_off + slot * plan->ws.x_stage_bytes);
    float* ts = ws_ptr(workspace, plan->ws.t_stage_off + slot * plan->ws.t_stage_bytes);
    // the step that last read this slot must be through with it
    if (plan->slot_used[slot] && cudaStreamWaitEvent(cs, static_cast<cudaEvent_t>(plan->ev_slot_free[slot]), 0) != cudaSuccess)
        return FTP_ERR_CUDA;
    if (cudaMemcpyAsync(xs, x_host, (size_t)plan->N * in.C * in.H * in.W * 4, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaMemcpyAsync(ts, target_host, (size_t)plan->N * out.C * out.H * out.W * 4, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaEventRecord(static_cast<cudaEvent_t>(plan->ev_prefetch), cs) != cudaSuccess)
        return FTP_ERR_CUDA;
    plan->pre_x = x_host; plan->pre_t = target_host; plan->pre_slot = slot;
    return FTP_OK;
}

int ftp_step_host(ftp_plan* plan, const float* x_host, const float* target_host, float* params, float lr,
                  float* loss_host, float* dx, void* workspace, void* stream)
{
    if (!plan || !x_host || !target_host || !params || !workspace || !aligned256(workspace)) return FTP_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const MapShape& in = plan->maps.front();
    const MapShape& out = plan->maps.back();
    float* lv = ws_ptr(workspace, plan->ws.loss_val_off);
    int rc = ensure_copy_stream(plan);
    if (rc != FTP_OK) return rc;
    const bool prefetched = plan->pre_slot >= 0 && plan->pre_x == x_host && plan->pre_t == target_host;
    const int slot = prefetched ? plan->pre_slot : plan->cur_slot;
    float* xs = ws_ptr(workspace, plan->ws.x_stage_off + slot * plan->ws.x_stage_bytes);
    float* ts = ws_ptr(workspace, plan->ws.t_stage_off + slot * plan->ws.t_stage_bytes);
    if (prefetched) {
        // the batch is in (or on its way to) the other staging slot: wait for its copies only
        if (cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(plan->ev_prefetch), 0) != cudaSuccess) return FTP_ERR_CUDA;
        plan->pre_slot = -1;
        plan->cur_slot = slot;
        rc = step_impl(plan, xs, nullptr, ts, params, params, lr, nullptr, lv, dx, workspace, stream);
    } else {
        // The input goes first on the caller's stream; the target is only needed at the loss, so its copy
        // runs on the plan's side stream while the forward pass computes.
        cudaStream_t cs = static_cast<cudaStream_t>(plan->copy_stream);
        cudaEvent_t fork = static_cast<cudaEvent_t>(plan->ev_fork), join = static_cast<cudaEvent_t>(plan->ev_join);
        if (cudaEventRecord(fork, st) != cudaSuccess || cudaStreamWaitEvent(cs, fork, 0) != cudaSuccess ||      // after earlier work on `stream`
            cudaMemcpyAsync(ts, target_host, (size_t)plan->N * out.C * out.H * out.W * 4, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
            cudaEventRecord(join, cs) != cudaSuccess ||
            cudaMemcpyAsync(xs, x_host, (size_t)plan->N * in.C * in.H * in.W * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return FTP_ERR_CUDA;
        rc = step_impl(plan, xs, nullptr, ts, params, params, lr, nullptr, lv, dx, workspace, stream, join);
    }
    if (rc != FTP_OK) return rc;
    if (cudaEventRecord(static_cast<cudaEvent_t>(plan->ev_slot_free[slot]), st) != cudaSuccess) return FTP_ERR_CUDA;
    plan->slot_used[slot] = true;
    if (loss_host && cudaMemcpyAsync(loss_host, lv, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FTP_ERR_CUDA;
    return FTP_OK;
}

int ftp_step_grad(ftp_plan* plan, const float* x, const float* dy, const float* target, const float* params,
                  float* dparams, float* loss_out, float* dx, void* workspace, void* stream)
{
    if (!dparams) return FTP_ERR_ARG;
    return step_impl(plan, x, dy, target, params, nullptr, 0.f, dparams, loss_out, dx, workspace, stream);
}

int ftp_step_grad_groups(ftp_plan* plan, const float* x, const float* dy, const float* target, const float* params,
                         float* dparams, float* loss_out, float* dx, void* workspace, void* stream,
                         ftp_group_ready_fn ready, void* user)
{
    if (!plan || !dparams) return FTP_ERR_ARG;
    plan->group_ready = ready; plan->group_ready_user = user;
    const int rc = step_impl(plan, x, dy, target, params, nullptr, 0.f, dparams, loss_out, dx, workspace, stream);
    plan->group_ready = nullptr; plan->group_ready_user = nullptr;
    return rc;
}

int ftp_sgd(float* params, const float* grad, size_t count, float lr, void* stream)
{
    if (!params || !grad) return FTP_ERR_ARG;
    if (count == 0) return FTP_OK;
    const int blocks = (int)std::min<size_t>((count + 255) / 256, (size_t)kSmCount * 16);
    sgd_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(params, grad, count, lr);
    return launched_ok() ? FTP_OK : FTP_ERR_CUDA;
}

int ftp_plan_timing(ftp_plan* plan, int enable)
{
    if (!plan) return FTP_ERR_ARG;
    for (void* e : plan->ev_begin) cudaEventDestroy(static_cast<cudaEvent_t>(e));
    for (void* e : plan->ev_end) cudaEventDestroy(static_cast<cudaEvent_t>(e));
    plan->ev_begin.clear(); plan->ev_end.clear(); plan->ev_kind.clear(); plan->ev_group.clear();
    plan->ev_used = 0;
    plan->timing = false;
    if (!enable) return FTP_OK;
    for (int i = 0; i < kMaxTimed; ++i) {
        cudaEvent_t a, b;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return FTP_ERR_CUDA;
        plan->ev_begin.push_back(a); plan->ev_end.push_back(b);
    }
    plan->ev_kind.assign(kMaxTimed, 0); plan->ev_group.assign(kMaxTimed, -1);
    plan->timing = true;
    return FTP_OK;
}

int ftp_plan_timing_read(ftp_plan* plan, int* n, ftp_launch_time* out, int capacity)
{
    if (!plan || !n) return FTP_ERR_ARG;
    *n = plan->ev_used;
    for (int i = 0; i < plan->ev_used && i < capacity && out; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, static_cast<cudaEvent_t>(plan->ev_begin[i]), static_cast<cudaEvent_t>(plan->ev_end[i])) != cudaSuccess)
            return FTP_ERR_CUDA;
        out[i] = ftp_launch_time{plan->ev_kind[i], plan->ev_group[i], ms};
    }
    plan->ev_used = 0;
    return FTP_OK;
}

long long ftp_plan_launch_count(const ftp_plan* plan) { return plan ? plan->launches : 0; }

int ftp_plan_check(ftp_plan* plan, void* workspace, void* stream)
{
    if (!plan || !workspace) return FTP_ERR_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return FTP_ERR_CUDA;
    if (!is_tc(plan)) return FTP_OK;
    int word = 0;
    if (cudaMemcpy(&word, err_ptr(workspace, plan), 4, cudaMemcpyDeviceToHost) != cudaSuccess) return FTP_ERR_CUDA;
    return word ? FTP_ERR_TIMEOUT : FTP_OK;
}

int ftp_plan_wait_probe(ftp_plan* plan, void* workspace, int limit_us, void* stream)
{
    if (!plan || !workspace || !aligned256(workspace) || limit_us <= 0 || limit_us > 100000) return FTP_ERR_ARG;
    if (!is_tc(plan)) return FTP_ERR_PRECISION;
    ++plan->launches;
    tcd::wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(err_ptr(workspace, plan), (long long)limit_us * 2000);
    return launched_ok() ? FTP_OK : FTP_ERR_CUDA;
}

const char* ftp_strerror(int code)
{
    switch (code) {
    case FTP_OK: return "ok";
    case FTP_ERR_ARG: return "invalid argument (null pointer, bad size or index, unaligned workspace)";
    case FTP_ERR_LAYERS: return "unsupported layer (conv: odd k<=7, stride 1, pad k/2; maxpool: 2x2/2 on even extents; bf16 fused stacks: at most 512 channels) or channel mismatch";
    case FTP_ERR_GRID: return "tile grid has more tiles than pixels in a group's output map";
    case FTP_ERR_GROUPS: return "groups must be contiguous, cover layers 1..L, and hold at most 16 layers each";
    case FTP_ERR_WORKSPACE: return "no sub-tile of a group fits in shared memory; use smaller groups";
    case FTP_ERR_CUDA: return "a CUDA runtime call failed";
    case FTP_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case FTP_ERR_PRECISION: return "requested arithmetic is not built into this library";
    case FTP_ERR_TOO_LARGE: return "size exceeds the fixed capacity of this no-allocation entry point";
    default: return "unknown error";
    }
}

}  // extern "C"
