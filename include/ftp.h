/*
 * ftp -- fused tile-partitioned CNN training step for NVIDIA B200 (sm_100a).
 *
 * C-ABI of the library.  It implements the training cycle of "Distributed
 * Convolutional Neural Network Training on Mobile and Edge Clusters"
 * (arXiv 2409.09083): feature maps (forward) and delta maps (backward) are cut
 * into a grid of tiles, matching tiles of consecutive conv / max-pool layers are
 * fused into independent stacks, layers are combined into groups that exchange
 * boundary data only at group inputs (Section 3, Section 4.2), every tile
 * produces a partial filter-gradient set, and the sets are summed once per
 * batch and used to update the filters (Section 4.1).  Here a tile stack runs
 * in a thread block of one GPU instead of on an edge device.
 *
 * Conventions
 *  - Every tensor pointer is CALLER-OWNED DEVICE memory, dense fp32, NCHW.
 *  - `params` is one flat vector: for each conv layer in order the filter
 *    [cout][cin][k][k] followed by the bias [cout].
 *  - `workspace` is caller-allocated device memory of at least the size
 *    ftp_plan_sizes reports, 256-byte aligned.  It holds the maps at group
 *    boundaries, the saved layer outputs the backward pass reads, the per-tile
 *    partial gradient sets and small tables.  Its contents carry state from
 *    ftp_forward to ftp_backward and are otherwise scratch.
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *    return without synchronising.  The first launch on a plan uploads the
 *    plan's tables to the device with a blocking copy (a few KB, one
 *    cudaMalloc); make that first call outside any stream capture.
 *  - Return value: 0 on success, a negative FTP_ERR_* code otherwise.  Invalid
 *    arguments are detected on the host before anything is launched.  The
 *    library never aborts, throws or traps.
 *  - A plan is immutable after creation; using one plan from several host
 *    threads at once, or on overlapping streams with the same workspace, races.
 */
#ifndef FTP_H
#define FTP_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    FTP_OK            =  0,
    FTP_ERR_ARG       = -1,  /* null pointer, non-positive size, bad index        */
    FTP_ERR_LAYERS    = -2,  /* unsupported layer or channel mismatch             */
    FTP_ERR_GRID      = -3,  /* more tiles than pixels in a group's output map    */
    FTP_ERR_GROUPS    = -4,  /* groups not contiguous or not covering 1..L        */
    FTP_ERR_WORKSPACE = -5,  /* no sub-tile of a group fits in shared memory      */
    FTP_ERR_CUDA      = -6,  /* a CUDA runtime call failed                        */
    FTP_ERR_TIMEOUT   = -7,  /* a bounded device-side wait ran out (ftp_plan_check) */
    FTP_ERR_PRECISION = -8,  /* requested arithmetic is not built                 */
    FTP_ERR_TOO_LARGE = -9   /* size beyond the fixed capacity of a no-allocation entry point */
};

enum { FTP_CONV = 0, FTP_MAXPOOL = 1 };
enum { FTP_FP32 = 0, FTP_BF16_FP32ACC = 1 };

/* Layer descriptor: kernel K_l x K_l and stride S_l in the paper's notation
 * (Section 4.2).  Supported: conv with odd k <= 7, stride 1, pad = k / 2,
 * followed by bias and leaky ReLU with negative slope `leaky` (derivative
 * `leaky` at exactly 0); max-pool with k = 2, stride 2, pad 0 on even extents
 * (first maximum in row-major window order receives the gradient). */
typedef struct {
    int   kind;          /* FTP_CONV or FTP_MAXPOOL */
    int   cin, cout;     /* conv only */
    int   k, stride, pad;
    float leaky;         /* conv only */
} ftp_layer;

/* A group as an inclusive 1-based layer range.  The paper's tuple (s, e)
 * spans the maps from the input of layer s to the input of layer e
 * (Section 4.2); here that is (first, last + 1).  Boundary data is exchanged
 * only at the input map of `first`. */
typedef struct { int first, last; } ftp_group;

typedef struct ftp_plan ftp_plan;   /* opaque, host-owned */

/*
 * Tile-region planner (Section 4.2).  For every group the group's output map
 * is partitioned equally among the grid_y x grid_x tiles (tile i of g owns
 * [floor(i*E/g), floor((i+1)*E/g) - 1] along an axis of extent E), and each
 * tile's span at every earlier map of the group follows from the receptive
 * field recursion, Eq. (1), generalised with explicit padding so that it also
 * covers the 2x2/2 pool (in1 = out1*S - P, in2 = out2*S - P + K - 1), clamped
 * to the map at every step.  Tiles are further cut into sub-tiles whose whole
 * layer stack fits the shared memory of one thread block; results do not
 * depend on that cut.  A requested group whose stack can be held in shared
 * memory only with sub-tiles so small that halo recomputation explodes (deep
 * stacks at high resolution, or layers with many channels) is executed as
 * several consecutive groups, i.e. with the
 * finer grouping profile ftp_plan_exec_groups reports; the method's result does
 * not depend on the profile (Section 3), only its cost does.
 * N, C, H, W: shape of the network input X_1.  `layers`/`groups` are copied.
 * Errors: FTP_ERR_ARG, _LAYERS, _GRID, _GROUPS, _WORKSPACE, _PRECISION.
 * Needs no GPU.
 */
int ftp_plan_create(const ftp_layer* layers, int n_layers,
                    int N, int C, int H, int W,
                    int grid_y, int grid_x,
                    const ftp_group* groups, int n_groups,
                    int precision, ftp_plan** out);

/* Planner options; zero-initialise, set struct_size = sizeof(ftp_plan_opts),
 * and leave a field 0 for its default. */
typedef struct {
    int struct_size;
    int max_redundancy_pct; /* a requested group is cut into shorter groups when the multiply-accumulates
                           of its sub-tile stacks (halo recomputation included) exceed this percentage of
                           the untiled ones in either pass (default 150, minimum 100) */
    int max_subtile;    /* upper bound on the sub-tile extent (default: none) */
    int smem_bytes;     /* dynamic shared memory a block may use (default and maximum 230400) */
    int strict_groups;  /* 1: never cut a requested group; FTP_ERR_WORKSPACE if it cannot fit at all */
    int tc_blocks_per_sm; /* bf16 path: thread blocks per SM, 1 or 2, for both passes of every group whose layers have at
                           most 256 channels (two blocks hide each other's latencies but each gets half of the shared
                           and tensor memory, i.e. smaller sub-tiles).  Default: 2 only in the forward pass of groups
                           with at most 64 channels */
    int max_group_convs;  /* executed groups hold at most this many conv layers, with the pools that follow them
                           (default 2; -1: no limit).  A requested group with more is executed as consecutive
                           shorter groups: measured on B200, on the 8- and 16-layer stacks and both precisions,
                           conv(+pool) pairs beat longer fused runs (halo recomputation and small sub-tiles cost
                           more than the extra boundary traffic) and single layers (launches, boundary traffic) */
    int cost_model;       /* 1: compare all cuts of each requested group into executed groups of one to three conv
                           layers by the planner's time model (ftp_plan_cost) and take the best one instead of the
                           max_group_convs rule's cuts when the model puts it at least 3 % ahead; -1: never.
                           Default: 1, unless max_group_convs is given (then only that rule applies) */
    int stationary;       /* fp32 path: executed groups that hold ONE conv layer (with the pool after it, if any;
                           1x1 or 3x3 window) can run weight-stationary instead of as fused sub-tile stacks: blocks
                           keep a 64-channel slice of the filter, or a 64 x 32 slice of the filter gradient, on chip
                           and stream pixel tiles through it, and the layer's maps cross the group boundary in
                           global memory as at any group boundary (the paper's weight-dominated layers, Section 6).
                           Default (0): groups whose conv has at least 32 input channels; 1: every such group
                           whatever its channel count; -1: never.
                           bf16 path: a conv layer with a 1x1 or 3x3 window on a map of at most 1008 columns (the first
                           layer: a 3x3 window and at most 7 input channels) becomes an executed group of its own (with
                           its pool).  Forward pass and input delta run as banded tensor-core convolutions (a band of
                           rows x a slice of output channels stays in tensor memory while the input channels stream
                           past; the delta is the convolution of dz with the rotated filters and writes every cell
                           once), the filter gradient by a weight-stationary kernel that keeps a slice of the gradient
                           in tensor memory while the batch streams past; the first layer runs as a 1x1 conv on a
                           window-unrolled bf16 copy of the network input, with the same parameters.
                           0 and 1: every such layer; -1: never (fused stacks only).  Conv layers with more than 512
                           input or output channels run this way only (the fused kernels keep all output channels of
                           an op in the 512 tensor-memory columns): a bf16 plan that would put such a layer into a
                           fused stack is refused with FTP_ERR_LAYERS */
    int tc_tma;           /* bf16 path, fused sub-tile kernels: how the tiles of maps saved as bf16 planes reach shared memory.  Default (0): tensor
                           copies by the TMA engine (cp.async.bulk.tensor, one box per 8-channel plane, zeros outside the map;
                           the tensor maps cover the calling GPU's own memory only and no copy is multicast); -1: plain
                           loads by the threads */
} ftp_plan_opts;

/* ftp_plan_create with explicit planner options (NULL = defaults). */
int ftp_plan_create_opts(const ftp_layer* layers, int n_layers,
                         int N, int C, int H, int W,
                         int grid_y, int grid_x,
                         const ftp_group* groups, int n_groups,
                         int precision, const ftp_plan_opts* opts, ftp_plan** out);

/* The grouping profile that is executed (see ftp_plan_create): writes up to
 * `capacity` groups to groups_out (may be NULL) and the count to *n_groups. */
int ftp_plan_exec_groups(const ftp_plan* plan, int* n_groups, ftp_group* groups_out, int capacity);

/* How executed group `group` (0-based index into ftp_plan_exec_groups) runs: *stationary = 1 if it is a one-conv
 * group run by the weight-stationary kernels of the fp32 path (see ftp_plan_opts.stationary), 2 if by the banded
 * tensor-core kernels of the bf16 path, 0 if as fused sub-tile stacks;
 * *partial_sets (may be NULL) = the partial gradient sets of the group that the cross-tile reduction sums
 * (Section 4.1).  FTP_ERR_ARG on a bad index or NULL. */
int ftp_plan_group_mode(const ftp_plan* plan, int group, int* stationary, int* partial_sets);

void ftp_plan_destroy(ftp_plan* plan);

/*
 * Span of user tile (ty, tx) at map X_{map_index} (1-based; must lie in
 * first..last+1 of `group`, 0-based group index): span_out = {x1, y1, x2, y2},
 * inclusive, the paper's (x1, y1), (x2, y2) (Section 4.2).
 * pass 0: feature-map span of the forward pass, Eq. (1).
 * pass 1: delta-map span the tile back-propagates.  The backward pass runs in
 *   adjoint form: a tile pushes the delta of its owned part of the group's
 *   output map back through its own forward stack, so these spans equal the
 *   forward spans, and overlapping contributions are summed at the group
 *   input.
 * pass 2: Eq. (2) gather-form span, for reference: the delta span at
 *   X_{map_index} needed to produce the tile's equal share of the group's
 *   INPUT delta map.
 */
int ftp_plan_region(const ftp_plan* plan, int pass, int group, int map_index,
                    int ty, int tx, int span_out[4]);

/*
 * Sizes: number of parameter floats, workspace bytes, floats of the network
 * output X_{L+1} (N*C*H*W of the last map), and the forward redundancy factor
 * (multiply-accumulates executed with halo recomputation / untiled ones).
 * Any out pointer may be NULL.
 */
int ftp_plan_sizes(const ftp_plan* plan, size_t* param_floats,
                   size_t* workspace_bytes, size_t* out_floats,
                   double* redundancy);

/*
 * Sub-tiling chosen for an EXECUTED group (0-based index into the profile of
 * ftp_plan_exec_groups) and pass (0 forward, 1 backward):
 * number of sub-tile rows and columns over the whole map, dynamic shared
 * memory per block in bytes, and blocks launched.  Any out pointer may be NULL.
 */
int ftp_plan_subtiles(const ftp_plan* plan, int pass, int group,
                      int* rows, int* cols, size_t* smem_bytes, int* blocks);

/*
 * fp32 path, backward pass of an EXECUTED group: channels of the shared-memory staging area in
 * which the delta at the output of a fused conv+pool layer is laid out, routed through the
 * arg-max and zero-extended, for the input-delta convolution (the back-propagation of Section 3
 * through a max-pool and a conv in one go).  The planner grants the area where it costs no
 * sub-tile size; 0 means the convolution expands the pooled delta on the fly instead.  Both forms
 * compute the same sums in the same order.  FTP_ERR_ARG on a bad index.
 */
int ftp_plan_delta_staging(const ftp_plan* plan, int group, int* channels);

/*
 * The planner's time model of one pass (0 forward, 1 backward) of an EXECUTED
 * group.  The paper chooses its grouping profile by weighing halo
 * recomputation against boundary exchanges (Sections 4.2 and 5.3) but does not
 * print the procedure; this library estimates the time of a pass as a
 * weighted sum of FTP_COST_TERMS work terms taken on the pass's critical path
 * (multiply-accumulates or tensor-core cycles incl. halo recomputation, filter
 * bytes streamed, partial-set bytes updated, map bytes moved, per-layer
 * synchronisations, one launch), with weights fitted to measurements on B200.
 * need_dx: whether the delta at the group's input is produced (it is for every
 * group but the first of a training step).  terms (host, FTP_COST_TERMS
 * doubles, may be NULL) receives the terms, estimate_us (host, may be NULL)
 * the estimate in microseconds.  FTP_ERR_ARG on a bad index.
 */
#define FTP_COST_TERMS 8
int ftp_plan_cost(const ftp_plan* plan, int pass, int group, int need_dx,
                  double* terms, double* estimate_us);

/*
 * Forward pass (Section 3; Section 4.1 forward; Section 4.2 groups): one fused
 * launch per group, halo exchange through the group's input map in HBM.
 *   x [N,C,H,W] in, params in, y [N,C_out,H_out,W_out] out (may be NULL).
 * Layer outputs are kept in `workspace` for ftp_backward.
 */
int ftp_forward(ftp_plan* plan, const float* x, const float* params, float* y,
                void* workspace, void* stream);

/*
 * Backward pass (Section 4.1 back-propagation and filter gradients; Section
 * 4.2): needs a preceding ftp_forward with the same plan, x, params and
 * workspace.  dy = dLoss/dX_{L+1} in.  dx = dLoss/dX_1 out, may be NULL (then
 * it is not computed).  dparams out, same layout as params: the sum over all
 * tiles of the partial filter and bias gradients, in a fixed order.
 */
int ftp_backward(ftp_plan* plan, const float* x, const float* dy,
                 const float* params, float* dx, float* dparams,
                 void* workspace, void* stream);

/*
 * One training cycle (Section 3: forward, backward, sum of the partial
 * filter-gradient sets once per batch, update): params <- params - lr * grad
 * in place (plain SGD).  Give exactly one of
 *   dy      the loss delta at the last map, or
 *   target  [same shape as the output] for the mean-squared-error loss
 *           L = mean((X_{L+1} - target)^2).
 * loss_out (device, 1 float, may be NULL) receives L when `target` is given.
 * dx (may be NULL) receives dLoss/dX_1.
 */
int ftp_step(ftp_plan* plan, const float* x, const float* dy,
             const float* target, float* params, float lr, float* loss_out,
             float* dx, void* workspace, void* stream);

/*
 * The loss-delta injection of the training cycle on its own (Section 3: the initial delta of the
 * loss enters at the last layer), for callers that drive ftp_forward and ftp_backward themselves:
 * mean-squared error L = mean((y - target)^2) over the plan's output map X_{L+1}
 * ([N,C_out,H_out,W_out], y and target), dy = dL/dy = 2 (y - target) / M with M the element count.
 * dy (device, same shape) and loss_out (device, 1 float) may each be NULL but not both.
 * Uses a few KB of `workspace` as scratch for per-block partial sums; the sum order is fixed.
 */
int ftp_loss_mse(ftp_plan* plan, const float* y, const float* target, float* dy, float* loss_out,
                 void* workspace, void* stream);

/*
 * ftp_loss_mse for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for the environments named below, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a CUDA stream capture,
 * under a framework or allocator that owns all device memory and forbids side allocations, in a
 * real-time loop that must not take the driver's allocation lock, or in a process whose memory
 * budget is fixed at start-up.  ftp_loss_mse needs a plan (whose first use allocates its tables)
 * and a workspace; this call needs neither.  It calls no cudaMalloc, no cudaFree and no
 * allocating library routine.
 *
 * Same arithmetic as ftp_loss_mse: L = mean((y - target)^2) over `count` elements,
 * dy[i] = 2 (y[i] - target[i]) / count.  y, target: device, `count` floats.  dy (device, `count`
 * floats) and loss_out (device, 1 float) may each be NULL but not both.  The partial sums are
 * added in a fixed order, which is not ftp_loss_mse's order: the two losses agree to rounding.
 *
 * Scratch: the per-block partial sums sit in a fixed 16 KB array inside the library image (every
 * GPU that loads the library holds it until the process exits).  That fixes the capacity:
 * count <= FTP_LOSS_STATIC_MAX_COUNT, else FTP_ERR_TOO_LARGE and nothing is launched.
 *
 * All calls on one GPU share that array.  Nothing in it has to start at zero (each call overwrites
 * every slot it later reads), so calls one after the other on a stream need no clearing; two calls
 * whose kernels overlap on the GPU (different streams, no ordering) race on it and may both return
 * a wrong loss.  Order them, or use ftp_loss_mse with separate workspaces.
 *
 * The first call on each device looks up the array's device address (once, with that device
 * current, under a host lock); make that first call before any stream capture begins.
 * Errors: FTP_ERR_ARG (null pointer, count 0, device ordinal >= 64), FTP_ERR_TOO_LARGE,
 * FTP_ERR_CUDA.
 */
#define FTP_LOSS_STATIC_MAX_COUNT (1u << 26)   /* 67 108 864 elements (256 MiB per fp32 tensor) */
int ftp_loss_mse_static(const float* y, const float* target, float* dy, float* loss_out,
                        size_t count, void* stream);

/*
 * ftp_step for callers whose batch lives in HOST memory: copies x_host and target_host
 * (pinned memory recommended; shapes as in ftp_step) into staging areas of the workspace,
 * runs the training cycle with the mean-squared-error loss and copies the loss (1 float) to
 * loss_host, all ordered on `stream` (the target's copy runs on a side stream of the plan, created on
 * the first call, and joins before the loss); loss_host is valid once the stream is synchronised.
 * params stays in device memory and is updated in place.  dx (device, may be NULL) receives
 * dLoss/dX_1 as in ftp_step.
 */
int ftp_step_host(ftp_plan* plan, const float* x_host, const float* target_host, float* params,
                  float lr, float* loss_host, float* dx, void* workspace, void* stream);

/*
 * Input pipeline for ftp_step_host (the paper's devices receive their tiles of the next image over the
 * network while they compute, Section 5; here the next batch crosses PCIe while the current step runs).
 * Copies x_host and target_host (pinned memory, shapes as in ftp_step_host) into the staging slot of the
 * workspace that the last ftp_step_host call does not read, asynchronously on `copy_stream` (a
 * cudaStream_t; NULL = the plan's own side stream), after the step that last read that slot.  The next
 * ftp_step_host call that is given the SAME two host pointers waits for these copies on its stream
 * instead of copying; a call with other pointers copies as usual and leaves the prefetched batch in
 * place.  The host buffers must stay unchanged until that step's stream has been synchronised.  One
 * batch can be in flight at a time: a second prefetch before the step overwrites the first.
 * Returns FTP_ERR_ARG on a null or unaligned pointer, FTP_ERR_CUDA if a runtime call fails.
 */
int ftp_prefetch_host(ftp_plan* plan, const float* x_host, const float* target_host,
                      void* workspace, void* copy_stream);

/*
 * The two halves of ftp_step for data-parallel replicas (one process per GPU, the batch split
 * across them; Section 4.1 sums the partial gradient sets one time for each batch, which across GPUs
 * is an all-reduce the caller runs between these two calls):
 * ftp_step_grad = ftp_step without the update: forward, loss delta, backward, and the fixed-order
 *   sum of this GPU's partial sets written to dparams (device, same layout as params).
 * ftp_sgd = params[i] -= lr * grad[i] for i < count (device pointers).
 */
int ftp_step_grad(ftp_plan* plan, const float* x, const float* dy, const float* target,
                  const float* params, float* dparams, float* loss_out, float* dx,
                  void* workspace, void* stream);
int ftp_sgd(float* params, const float* grad, size_t count, float lr, void* stream);

/*
 * ftp_step_grad that tells the caller when the gradient of each executed group is complete, so that its
 * all-reduce can run while the groups before it are still being back-propagated (the paper's devices send
 * their partial sets to the common device at the end of the batch, Section 4.1; between GPUs the sets of the
 * last layers can travel while the first layers still compute).  Groups finish in reverse order.  Right
 * after the launches that write parameters [param_begin, param_begin + param_floats) of dparams have been
 * put on `stream`, `ready` is called ON THE HOST, in the calling thread: the work is queued, not done, so the
 * callee orders its own work behind it (record an event on `stream`, make the communication stream wait for
 * it).  Every parameter is reported exactly once.  The sums are the same, in the same order, as
 * ftp_step_grad's: dparams is bit-identical.  `ready` may be NULL (then this is ftp_step_grad).
 */
typedef void (*ftp_group_ready_fn)(void* user, int group, long long param_begin, long long param_floats);
int ftp_step_grad_groups(ftp_plan* plan, const float* x, const float* dy, const float* target,
                         const float* params, float* dparams, float* loss_out, float* dx,
                         void* workspace, void* stream, ftp_group_ready_fn ready, void* user);

/*
 * Per-launch device timing for benchmarks.  ftp_plan_timing(plan, 1) makes every later call on
 * this plan record a CUDA event before and after each kernel it launches, on the stream it
 * launches on (events are created here, not in the hot path); 0 switches it off and frees them.
 * After synchronising the stream, ftp_plan_timing_read returns, for the launches of the most
 * recent ftp_forward / ftp_backward / ftp_step* call(s) since the last read, up to `capacity`
 * records {kind, group, milliseconds}: kind 0 filter packing, 1 fused forward, 2 loss delta,
 * 3 fused backward, 4 halo sum, 5 reduction (+SGD); group = executed-group index or -1.
 */
typedef struct { int kind; int group; float ms; } ftp_launch_time;
int ftp_plan_timing(ftp_plan* plan, int enable);
int ftp_plan_timing_read(ftp_plan* plan, int* n, ftp_launch_time* out, int capacity);

/*
 * Measurement aid for the roofline of the fp32 (CUDA-core) kernels, which are bound by the fp32
 * multiply-add rate and not by memory (the fused stacks move about 9 MB per image for 15.8 GFLOP,
 * Section 5 workload): launches a register-only loop of independent fp32 FMAs on every
 * multiprocessor (two blocks of 512 threads each) on `stream`.  The caller times the launch with
 * events; *flops receives the floating-point operations it performs (2 per FMA).
 *   out        DEVICE, at least 1024 x (number of multiprocessors) floats, overwritten
 *   iters      loop count per thread (128 FMAs per iteration)
 * Returns FTP_ERR_ARG on a null pointer, iters <= 0 or a too-small `out`, FTP_ERR_CUDA if a runtime
 * call fails.  The paper has no counterpart; it is here so that the fraction of peak is quoted
 * against a number measured on the same device in the same run.
 */
int ftp_fma_peak(float* out, size_t out_count, long long iters, double* flops, void* stream);

/* Number of kernels the library launched on the calling thread's behalf since
 * the plan was created (for launch accounting in benchmarks). */
long long ftp_plan_launch_count(const ftp_plan* plan);

/*
 * Synchronises `stream` and reports whether a kernel of the bf16 tensor-core path gave up on one
 * of its bounded waits (for a filter stage to arrive or for the tensor core to finish) since the
 * last ftp_forward / ftp_step* call on this plan and workspace: FTP_ERR_TIMEOUT if so -- the results
 * of that call are then invalid -- else FTP_OK.  Kernels never wait without a limit; after a
 * failed wait they skip the remaining waits, release their tensor memory and return.  Always
 * FTP_OK for the fp32 path, which has no device-side waits.
 */
int ftp_plan_check(ftp_plan* plan, void* workspace, void* stream);

/*
 * Diagnostic for the error path above (the paper has no counterpart): launches, on `stream`, one small
 * kernel whose only thread waits on a barrier that nothing arrives on, through the same bounded-wait
 * routine as the bf16 tile kernels but with a limit of about `limit_us` microseconds (1 .. 100000, counted
 * in SM clock cycles at a nominal 2 GHz).  The wait runs out, the kernel sets the workspace's error word
 * and returns; nothing faults and the context stays usable.  The next ftp_plan_check then reports
 * FTP_ERR_TIMEOUT; the next ftp_forward / ftp_step* clears the word again.  bf16 plans only
 * (FTP_ERR_PRECISION otherwise); FTP_ERR_ARG on a null or unaligned pointer or a limit out of range.
 */
int ftp_plan_wait_probe(ftp_plan* plan, void* workspace, int limit_us, void* stream);

const char* ftp_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* FTP_H */
