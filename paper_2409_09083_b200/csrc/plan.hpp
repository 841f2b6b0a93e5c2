// Internal plan structures shared by the host planner and the kernel launchers.
// Host-only logic lives in plan.cpp; nothing here depends on the CUDA runtime.
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "ftp.h"

namespace ftp {

constexpr int kMaxOps      = 16;      // layers per group
constexpr int kThreads     = 512;     // threads per block of the fused kernels
constexpr int kSmCount     = 148;     // B200
constexpr int kSmemBudget  = 225 * 1024;  // dynamic shared memory a block may use
constexpr int kSmemHeader  = 1024;    // bytes reserved at the start for per-block tables
constexpr int kCoutTile    = 8;       // output channels per thread task (packed weights are padded to it)
constexpr int kMinFilterStage = 2048;   // fp32 path: smallest half (floats) of a filter staging area worth its barriers
constexpr int kDeltaStageChannels = 16; // fp32 backward: channels of the output delta staged at a time for the input-delta convolution

// Tensor-core (bf16) tile kernels: one block of 512 threads per SM with all 512 tensor-memory columns, or two
// blocks of 256 threads with 256 columns each.
constexpr int kTcMaxStages  = 4;          // weight ring: 2 stages of kTcStageBytes, 4 where that costs no sub-tile size
constexpr int kTcStageBytes = 16384;
constexpr int kTcTmemCols   = 512;        // tensor-memory columns of an SM; a block takes all of them, or half with two blocks per SM
constexpr int kTcHeader     = 4096;       // per-block tables, barriers, bias staging
constexpr int tc_fixed_bytes(int stages) { return kTcHeader + stages * kTcStageBytes; }   // shared memory before the activation area
constexpr int kTcSmemBudget = 227 * 1024; // dynamic shared memory a tensor-core block may use (one block per SM)
constexpr int kTcSmemBudget2 = 113 * 1024;// ... with two blocks per SM
constexpr int kTcIssuers = 4;             // threads (lane 0 of warps 0..3) that issue MMAs, each for its own accumulators
constexpr int kTcMaxUnits = 32;           // filter-gradient accumulators per pass (at least 16 columns each)
constexpr int kTcTailEntries = 16;        // 16-byte entries appended to every tile plane
// Bytes from one 8-channel plane of a shared-memory tile to the next: Hp x Wp entries of 16 bytes and the tail, rounded to
// 128 bytes so that every plane can be the destination of a tensor (TMA) copy.
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr size_t tc_plane_bytes(int Hp, int Wp) { return ((((size_t)Hp * Wp + kTcTailEntries) * 16) + 127) / 128 * 128; }
// Weight-stationary kernels of one-conv groups (stationary.cuh): 256 threads, two blocks per SM.
constexpr int kStThreads = 256;
// convolution: 64 output channels x 16 row pairs per block (8 channels x 2 rows x 4 columns per thread), or 32 x 32 for layers
// with at most 32 output channels
// with at most 32 output channels or with so few blocks that the last round of 64-channel blocks would leave SMs idle
constexpr int st_row_pairs(int co_tile, int threads = kStThreads) { return threads * 4 / co_tile; }
constexpr int kStCols    = 8;             // columns per block, both kernels
constexpr int kFgCo = 64, kFgCi = 32;     // filter gradient: (output, input) channel slice of a block (8 x 1 per thread)
constexpr int kFgRowPairs = 4;            // filter gradient: row pairs per pixel stage
constexpr int kFg1Co = 64, kFg1Ci = 128, kFg1Px = 32;   // filter gradient of a 1 x 1 conv: channel slice of a block, pixels per stage
constexpr int kThinTileH = 8, kThinTileW = 32;   // thin-input backward: pooled pixels per tile
constexpr int kStatMinCin = 32;           // fewest input channels for which a one-conv group runs weight-stationary by default
constexpr double kStatTflops = 45.0;      // measured rate of the weight-stationary kernels on B200 (3x3 layers), for the planner's estimates
constexpr double kStatTflops1x1 = 25.0;   // ... of the 1x1 kernels and of the thin first layer (dense-equivalent)
constexpr int kCostTerms = 8;             // terms of the planner's time estimate of one pass of a group

struct Span { int a, b; };            // inclusive interval on one axis

// One layer inside a group, as the kernels see it.
enum { kOpConv = 0, kOpPool = 1, kOpConvPool = 2 };   // an op is one layer, or a conv fused with the pool after it

struct OpDesc {
    int   kind;                 // kOpConv / kOpPool / kOpConvPool
    int   cin, cout, k, pad;    // conv part (pool: cin == cout, k = 2, pad = 0)
    int   S, keff;              // output -> input coordinate scale and effective window (conv K; pool 2; fused K+1)
    float slope;
    int   prev_has_act;         // the producer of this op's input, inside the same group, ends in a leaky ReLU
    int   in_map, out_map;      // 1-based indices l of the maps X_l this op reads / writes
    int   in_H, in_W;           // extents of the input map
    int   out_H, out_W;         // extents of the output map
    // shared-memory geometry (float offsets from the start of the dynamic area after the header)
    int   in_off, in_pitch, in_cs;     // forward input buffer / backward copy of the op's input
    int   d_off, d_pitch, d_cs;        // backward: delta at this op's output (no apron)
    int   d_arg_off;                   // backward, fused op: byte offset of the arg-max copy (same geometry as d)
    int   dz_off, dz_ch;               // backward: staging area of the zero-extended output delta, dz_ch channels at a time (0: none)
    int   w_off, w_ch;                 // filter staging area (two halves of w_ch input channels each; 0: filters are read from global memory)
    int   cout_pad, cin_pad;           // channel counts padded to kCoutTile in the packed filters
    long long wf_off, wb_off;          // float offsets into the packed forward / rotated filters
    long long p_off;                   // float offset of the filter in params (bias follows it)
    long long gp_off;                  // float offset of the filter inside the group's partial set
    // --- bf16 tensor-core path: shared-memory tiles are [channel/8][row][col][8] bf16 planes ---
    int   cin16, cout16;               // channel counts padded to 16 (pool: both = padded channels of the map)
    int   t_in_off, t_in_Hp, t_in_Wp;  // forward input tile: byte offset in the activation area, padded rows / cols
    int   t_x_off, t_x_Hp, t_x_Wp;     // backward: copy of the op's input
    int   t_dz_off, t_dz_Hp, t_dz_Wp;  // backward: delta at the conv output (before the pool), zero apron of k-1 around it
    int   t_dz_planes;                 // planes reserved for it (8, or a multiple of 16: the M = 64 / 128 operand stays inside)
    long long twf_off, twb_off;        // bf16 element offsets of the packed forward / rotated filters
    long long tgp_off;                 // float offset inside the group's partial set in the tensor-core layout
};

// Axis tables of one (group, pass): for sub-tile index r and map m (0 = group input ... n_ops = output)
//   span[(m * count + r) * 2 + {0,1}]   clamped span the sub-tile touches at map m
//   cell[(m * count + r) * 2 + {0,1}]   the part of map m this sub-tile owns (disjoint, covering)
struct AxisTables {
    int count = 0;                        // sub-tiles along this axis over the whole map
    std::vector<int> span, cell;
    std::vector<int> tile_begin;          // per user tile: first sub-tile index; size tiles + 1
    std::vector<int> scratch_off;         // prefix sum of span extents at map 0; size count + 1
    std::vector<int> cover;               // per position of map 0: first and last sub-tile covering it
    std::vector<int> maxext;              // per map m: max span extent
};

struct PassPlan {
    AxisTables y, x;
    size_t smem_bytes = 0;
    int blocks = 0;                 // forward: R*Q*N ; backward: min(R*Q*N, blocks that run at once), each with its own partial set
    int dz_ch = 0;                  // backward, fp32 path: channels of the delta staging area (see layout_backward)
    int stages = 2;                 // tensor-core path: stages of the filter ring
    int ctas = 1;                   // tensor-core path: blocks per SM (2 = each block takes half of the tensor memory)
    size_t scratch_floats = 0;      // backward: floats of per-sub-tile group-input deltas (all images)
    // offsets (in ints) of the tables inside the plan's device table blob
    int dev_yspan = 0, dev_xspan = 0, dev_ycell = 0, dev_xcell = 0;
    int dev_yoff = 0, dev_xoff = 0, dev_ycover = 0, dev_xcover = 0;
    int dev_ytile = 0, dev_xtile = 0;
};

// Weight-stationary execution of an executed group that holds one conv layer (stationary.cuh).
struct StatPlan {
    int on = 0;
    int thin = 0;                           // conv3x3 + pool with at most 4 input and 32 output channels: backward by thin_bwd_kernel
    int thin_blocks = 0, thin_tiles_y = 0, thin_tiles_x = 0;
    int k = 0, pool = 0;
    int fwd_blocks = 0, dx_blocks = 0;      // convolution launches: (row-pair tiles) x (column tiles) x (channel slices)
    int fwd_co_tile = 64, dx_co_tile = 64;  // output channels per block of the two convolutions (64 or 32)
    int fwd_threads = kStThreads, dx_threads = kStThreads;   // threads per block (256, or 128 where whole blocks would leave SMs idle)
    int fg_stages = 0, fg_splits = 0;       // filter gradient: pixel stages over the batch, and the shares they are dealt out in
    int fg_blocks = 0;                      // (64 x 32 channel slices) x shares; a share is one partial gradient set
};

// bf16 path, one-conv groups: the filter gradient by the weight-stationary tensor-core kernel (tc_stationary.cuh);
// the forward pass and the input delta (a plain convolution of dz with the rotated filters) by the banded
// convolution kernel, which writes every cell once, so there are no overlapping parts to sum.
struct TcFgPlan {
    int on = 0;
    int k = 0, Ms = 0, slices = 0;          // output channels per block (64 or 128), number of slices
    int ncols = 0, nci = 0;                 // input channels per block (multiple of 16), number of slices
    int R = 0, Wp = 0;                      // rows of a band, pitch of its tiles (Cw + k - 1)
    int ncc = 1, Cw = 0;                    // column chunks of a row band (maps wider than 126 pixels) and their width
    int bands_img = 0, bands = 0;           // bands per image and in the batch
    int shares = 0;                         // pixel shares = partial gradient sets of the group
    int blocks = 0;                         // slices * nci * shares
    int dz_plane = 0, x_plane = 0;          // bytes between the planes of the two tiles
    int stage_bytes = 0, smem_bytes = 0;
};
// Banded tensor-core convolution of a one-conv bf16 group (conv_tc_rows_kernel): forward pass and input delta.
struct TcConvPlan {
    int on = 0;
    int Ns = 0, slices = 0;                 // output channels per block, number of slices
    int R = 0, Wp = 0, bands_img = 0;       // rows per band, tile pitch, bands (row bands x column chunks) per image
    int ncc = 1, Cw = 0;                    // column chunks of a row band (maps wider than 126 pixels) and their width
    int nblk = 0;                           // accumulator blocks (128 tile entries each) of a full band
    int kpc = 0;                            // 8-channel input planes per chunk
    int x_plane = 0, stage_bytes = 0, stages = 0, smem_bytes = 0;
    int items = 0;                          // N * bands_img * slices
    int blocks = 0;                         // persistent blocks: min(items, SMs)
    int pool_planes = 0;                    // fused pool: 8-channel planes the staging area holds
    int pool_stage_bytes = 0;               //             and its size
    int nbuf = 1;                           // accumulator buffers (2 for slices of at most 64 channels)
};
constexpr int kTcPoolStageBytes = 32 * 1024;  // least staging area of the fused pool in the banded convolution (more where it fits)
constexpr int kTcConvSmemBudget = 224 * 1024; // banded convolution: header + stages + pool staging
constexpr int kTcMaxColChunks = 8;            // a band spans at most 126 columns (a TMA box row of 128 pixels with the halo): wider maps are cut into chunks
constexpr int kTcFgHeader = 1024;             // barriers, tensor-memory slot, a core matrix of ones
constexpr int kTcFgSmemBudget = 200 * 1024;   // header + two stages

struct GroupPlan {
    int first = 0, last = 0;        // 1-based layers
    StatPlan st;
    TcFgPlan tfg;
    TcConvPlan cf, cd;              // tfg.on: the forward convolution and the input-delta convolution (dz planes in, delta planes
                                    //   out: the conv with the channel counts exchanged and the filters rotated) as banded kernels
    // First layer of the bf16 path: a 3x3 conv with few input channels runs as a 1x1 conv with 9 cin input channels
    // on a window-unrolled copy of the network input (channel ci * 9 + ky * 3 + kx of a pixel = the input of channel ci
    // at window position (ky, kx)); the parameters keep their places, since W[co][ci][ky][kx] IS W'[co][ci * 9 + ky * 3 + kx].
    int col_cin = 0, col_cin16 = 0;     // 9 cin and its padding to 16 (0: not this route)
    int sets() const { return tfg.on ? tfg.shares : bwd.blocks; }   // partial gradient sets the reduction sums
    int n_ops = 0;
    OpDesc fwd_ops[kMaxOps];
    OpDesc bwd_ops[kMaxOps];
    PassPlan fwd, bwd;
    std::vector<Span> tile_y, tile_x;   // user-tile partition of the group's output map
    size_t param_floats = 0;            // floats of this group's partial gradient set (tensor-core path: padded layout)
    long long param_begin = 0;          // offset of the group's first parameter in params
    size_t partial_off = 0;             // float offset of the group's partial sets in the workspace
    double macs_done = 0, macs_untiled = 0;
};

struct MapShape { int C, H, W; };

struct Workspace {                 // byte offsets, all 256-aligned
    std::vector<size_t> map_off;   // X_2 .. X_{L+1}  (index l-1; entry 0 unused; maps inside a fused op have none)
    std::vector<size_t> arg_off;   // arg-max bytes of the pooled map X_l written by a fused op (index l-1)
    std::vector<size_t> dmap_off;  // delta maps at group inputs of groups 1.. (index = group), and slot for dY
    size_t dy_off = 0;             // loss delta at the last map (ftp_step with target)
    size_t scratch_off = 0;
    size_t col_off = 0;                // first layer of the bf16 path: the window-unrolled network input (bf16 planes)
    size_t dz_off = 0, dz_bytes = 0;   // one-conv groups: two areas (taken in turn, the second dz_bytes behind the first) for the
                                       // delta in front of the activation at the conv's resolution
    size_t wf_off = 0, wb_off = 0; // packed filters
    size_t partial_off = 0;
    size_t grad_off = 0;           // summed gradient (ftp_step keeps it internal)
    size_t loss_off = 0;           // per-block partial sums of the MSE
    size_t loss_val_off = 0;       // the loss value (ftp_step_host)
    size_t x_stage_off = 0, t_stage_off = 0;   // device copies of a host batch (ftp_step_host): two slots each, x_stage_bytes / t_stage_bytes apart
    size_t x_stage_bytes = 0, t_stage_bytes = 0;
    size_t y32_off = 0;            // tensor-core path: fp32 NCHW copy of the last map for the loss (ftp_step with target)
    size_t err_off = 0;            // device error word of the tensor-core kernels (a bounded wait ran out)
    size_t total = 0;
};

}  // namespace ftp

struct ftp_plan {
    std::vector<ftp_layer> layers;
    std::vector<ftp::MapShape> maps;        // X_1 .. X_{L+1}; index l-1
    std::vector<ftp_group> user_groups;     // the requested grouping profile
    std::vector<ftp::GroupPlan> groups;     // the executed groups (a requested group may be cut, see build_plan)
    int N = 0, grid_y = 0, grid_x = 0, precision = 0;
    int tc_tma = 1;                         // bf16 path: tiles of saved bf16 maps are copied by TMA (0: by the threads)
    size_t param_floats = 0;
    size_t wf_floats = 0, wb_floats = 0;    // packed filters (tensor-core path: counted in bf16 elements)
    ftp::Workspace ws;
    std::vector<int> tables;                // host copy of all device tables
    int*  dev_tables = nullptr;             // uploaded lazily by the first launch
    int   dev_id = -1;
    long long launches = 0;
    // optional per-launch timing (see ftp_plan_timing)
    bool timing = false;
    std::vector<void*> ev_begin, ev_end;    // cudaEvent_t, pre-created
    std::vector<int> ev_kind, ev_group;
    int ev_used = 0;
    int loss_blocks = 0;
    // ftp_step_host: side stream and events that let the target's host-to-device copy overlap the forward pass
    void* copy_stream = nullptr; void* ev_fork = nullptr; void* ev_join = nullptr;
    // ftp_prefetch_host: the batch copied ahead of its step into the staging slot the running step does not use
    void* ev_prefetch = nullptr; void* ev_slot_free[2] = {nullptr, nullptr};
    bool slot_used[2] = {false, false};
    int cur_slot = 0, pre_slot = -1;
    const float* pre_x = nullptr; const float* pre_t = nullptr;
    // weight-stationary groups: the filter gradients run on a side stream beside the input-delta convolutions
    void* grad_stream = nullptr; void* ev_dz[2] = {nullptr, nullptr}; void* ev_fg[2] = {nullptr, nullptr};
    bool fg_pending[2] = {false, false};
    int dz_turn = 0;
    // ftp_step_grad_groups: called on the host right after the launches that complete an executed group's summed gradient
    ftp_group_ready_fn group_ready = nullptr; void* group_ready_user = nullptr;
};

namespace ftp {
struct PlanOpts {
    int max_redundancy_pct = 150;   // a requested group is cut when its halo recomputation exceeds this (percent of untiled MACs)
    int max_subtile = 0;            // 0 = as large as fits; else an upper bound (tests use it to force sub-tiling)
    int smem_bytes = kSmemBudget;   // dynamic shared memory a block may use
    int strict_groups = 0;          // 1 = never cut a requested group
    int max_group_convs = 2;        // executed groups hold at most this many conv layers (0 = no limit)
    int cost_model = 1;             // 1 = the time model (pass_cost_terms) may replace the fixed rule's cuts, see build_plan
    int refine_backward = 1;        // 1 = the time model may take a finer backward split that balances the blocks (refine_backward_split)
    int tc_ctas = 0;                // tensor-core path: blocks per SM, 1 or 2 (0 = two where every layer of the group allows it)
    int tc_tma = 0;                 // bf16 path: 0 = tiles of saved maps arrive by TMA (cp.async.bulk.tensor), -1 = copied by the threads
    int stationary = 0;             // one-conv groups run weight-stationary: 0 = with at least kStatMinCin input channels, 1 = all, -1 = none
    int tensor_cores = 0;           // set by build_plan from the precision: shared-memory layouts of the bf16 path
};
// Builds everything but the device upload.  Returns FTP_OK or an error code.
int build_plan(ftp_plan& p, const ftp_layer* layers, int n_layers, int N, int C, int H, int W,
               int gy, int gx, const ftp_group* groups, int n_groups, int precision, const PlanOpts& opts);
int region(const ftp_plan& p, int pass, int group, int map_index, int ty, int tx, int out[4]);
// Cost terms of one pass of executed group `group` (see plan.cpp) and the estimate in microseconds built from them.
int cost_terms(const ftp_plan& p, int pass, int group, int need_dx, double terms[kCostTerms], double* est_us);
}  // namespace ftp
